// KV append: scatter the new tokens' K/V rows into their (page, slot) of the
// pool.  A pure 16-byte-vector copy, so the result is bit-exact by
// construction.  HBM-bound and small next to attention.
#include "internal.h"
#include "ptx.cuh"

namespace ap {

namespace {

// One thread moves one 16-byte vector of K and the matching vector of V.
// vec index v -> (row, kv head, chunk) with chunk fastest, so a warp reads
// 512 contiguous bytes of k_new and writes 256-byte runs of the pool.
__global__ void __launch_bounds__(256) kv_append_kernel(uint4 *__restrict__ k_pool, uint4 *__restrict__ v_pool,
                                                        const uint4 *__restrict__ k_new,
                                                        const uint4 *__restrict__ v_new,
                                                        const int32_t *__restrict__ append_dst, int64_t n_vec,
                                                        int num_kv_heads, int chunks_per_row, int num_pages,
                                                        int *status) {
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n_vec) return;
    const int c = (int)(v % chunks_per_row);
    const int64_t rh = v / chunks_per_row;
    const int g = (int)(rh % num_kv_heads);
    const int64_t row = rh / num_kv_heads;
    const int32_t dst = __ldg(append_dst + row);      // plan data: uploaded before any kernel of the step
    ptx::griddep_launch_dependents();
    ptx::griddep_wait();                              // the pool may still be read by the kernel before
    const int32_t page = dst >> 4, slot = dst & 15;
    if (page < 0 || page >= num_pages) {
        ptx::record_status(status, AP_ERR_BAD_BLOCK_TABLE);
        return;
    }
    const int64_t o = (((int64_t)page * num_kv_heads + g) * kPageSize + slot) * chunks_per_row + c;
    k_pool[o] = __ldg(k_new + v);
    v_pool[o] = __ldg(v_new + v);
}

}  // namespace

cudaError_t launch_kv_append(const ap_kv_pool *pool, const ap_plan *plan, const void *k_new, const void *v_new,
                             cudaStream_t stream) {
    const int chunks = pool->desc.head_dim / 8;
    const int64_t n_vec = plan->info.n_new * pool->desc.num_kv_heads * chunks;
    const int threads = 256;
    const int64_t blocks = (n_vec + threads - 1) / threads;
    cudaError_t e = launch_overlapped(kv_append_kernel, (unsigned)blocks, (unsigned)threads, 0, stream,
                                      (uint4 *)pool->desc.k_base, (uint4 *)pool->desc.v_base, (const uint4 *)k_new,
                                      (const uint4 *)v_new, plan->d_append_dst, n_vec, pool->desc.num_kv_heads, chunks,
                                      pool->desc.num_pages, pool->status_dev);
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ap
