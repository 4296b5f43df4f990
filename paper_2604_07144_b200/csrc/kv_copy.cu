// KV page copy: whole pages (every kv head, every slot, K and V) from one pool
// to another pool of the same shape, or to other pages of the same pool.  A
// pure 16-byte-vector copy, bit-exact by construction, bound by HBM (each byte
// is read once and written once).
#include "internal.h"
#include "ptx.cuh"

namespace ap {

namespace {

constexpr int kCopyThreads = 256;
constexpr int kVecPerThread = 4;                                  // 64 bytes per thread and plane in flight
constexpr int kVecPerBlock = kCopyThreads * kVecPerThread;        // 16 KB of one plane per CTA

// CTA (x, y): chunk x of page pair y.  A page of one plane is `page_vecs` contiguous 16-byte
// vectors; the CTA moves vectors [x * kVecPerBlock, ...) of the K page and of the V page.  All loads
// are issued before the first store.
__global__ void __launch_bounds__(kCopyThreads)
kv_copy_pages_kernel(uint4 *__restrict__ k_dst, uint4 *__restrict__ v_dst, const uint4 *__restrict__ k_src,
                     const uint4 *__restrict__ v_src, const int32_t *__restrict__ pairs, int page_vecs,
                     int num_pages_dst, int num_pages_src, int *status) {
    ptx::griddep_launch_dependents();
    ptx::griddep_wait();                          // the pools may still be in use by the kernel before
    const int32_t dst = __ldg(pairs + 2 * blockIdx.y), src = __ldg(pairs + 2 * blockIdx.y + 1);
    if (dst < 0 || dst >= num_pages_dst || src < 0 || src >= num_pages_src) {
        if (threadIdx.x == 0) ptx::record_status(status, AP_ERR_BAD_BLOCK_TABLE);
        return;
    }
    const int64_t so = (int64_t)src * page_vecs, dof = (int64_t)dst * page_vecs;
    const int v0 = blockIdx.x * kVecPerBlock + threadIdx.x;
    uint4 a[kVecPerThread], b[kVecPerThread];
#pragma unroll
    for (int i = 0; i < kVecPerThread; ++i) {
        const int v = v0 + i * kCopyThreads;
        if (v < page_vecs) {
            a[i] = __ldcs(k_src + so + v);
            b[i] = __ldcs(v_src + so + v);
        }
    }
#pragma unroll
    for (int i = 0; i < kVecPerThread; ++i) {
        const int v = v0 + i * kCopyThreads;
        if (v < page_vecs) {
            __stcs(k_dst + dof + v, a[i]);
            __stcs(v_dst + dof + v, b[i]);
        }
    }
}

}  // namespace

cudaError_t launch_kv_copy_pages(const ap_kv_pool *dst_pool, const ap_kv_pool *src_pool, const int32_t *d_pairs,
                                 int n_pairs, cudaStream_t stream) {
    const int page_vecs = dst_pool->desc.num_kv_heads * kPageSize * dst_pool->desc.head_dim * 2 / 16;
    const unsigned chunks = (unsigned)((page_vecs + kVecPerBlock - 1) / kVecPerBlock);
    cudaError_t e = cudaSuccess;
    // gridDim.y is limited to 65535: larger requests go out in slices
    for (int done = 0; done < n_pairs && e == cudaSuccess; done += 65535) {
        const int n = n_pairs - done < 65535 ? n_pairs - done : 65535;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(chunks, (unsigned)n);
        cfg.blockDim = dim3(kCopyThreads);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kv_copy_pages_kernel, (uint4 *)dst_pool->desc.k_base,
                               (uint4 *)dst_pool->desc.v_base, (const uint4 *)src_pool->desc.k_base,
                               (const uint4 *)src_pool->desc.v_base, d_pairs + 2 * (size_t)done, page_vecs,
                               (int)dst_pool->desc.num_pages, (int)src_pool->desc.num_pages, dst_pool->status_dev);
    }
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ap
