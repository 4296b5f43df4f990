// Prefill-chunk attention kernel (tcgen05 / tensor memory) and its launcher; the device code is in
// prefill_tcgen05.cuh.
#include "prefill_tcgen05.cuh"

namespace ap {

namespace {

using namespace prefill;

template <int D>
__global__ void __launch_bounds__(kPrefillThreads, 1)
prefill_tcgen05_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                       const __grid_constant__ CUtensorMap v_map, const PrefillTile *__restrict__ tiles,
                       const int32_t *__restrict__ bt_flat, __nv_bfloat16 *__restrict__ out,
                       float *__restrict__ lse_out, int Hq, int Hkv, int num_pages, float scale_log2, int *status,
                       uint64_t wait_limit_ns) {
    prefill_unit<D>(q_map, k_map, v_map, tiles, bt_flat, out, lse_out, Hq, Hkv, num_pages, scale_log2, status, wait_limit_ns,
                    (int)blockIdx.x);
}

template <int D>
cudaError_t launch_prefill_t(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                             cudaStream_t stream) {
    using Cfg = PrefillCfg<D>;
    static bool configured[64] = {};
    const int dev = pool->desc.device & 63;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tcgen05_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    CUtensorMap q_map;
    if (encode_q_tensor_map(&q_map, q, plan->info.n_new, plan->num_q_heads, D) != AP_OK) return cudaErrorInvalidValue;
    const float scale_log2 = plan->scale * 1.4426950408889634f;
    cudaError_t e = launch_overlapped(
        prefill_tcgen05_kernel<D>, (unsigned)plan->info.prefill_tiles, (unsigned)kPrefillThreads,
        (size_t)Cfg::kSmemBytes, stream, q_map, pool->k_map, pool->v_map, plan->d_tiles, plan->d_bt_flat,
        (__nv_bfloat16 *)out, lse, plan->num_q_heads, pool->desc.num_kv_heads, pool->desc.num_pages, scale_log2,
        pool->status_dev, pool->wait_limit_ns);
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefill(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                           cudaStream_t stream) {
    if (pool->desc.head_dim == 128) return launch_prefill_t<128>(pool, plan, q, out, lse, stream);
    return launch_prefill_t<64>(pool, plan, q, out, lse, stream);
}

}  // namespace ap
