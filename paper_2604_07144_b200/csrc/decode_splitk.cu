// Decode attention kernel (split-K flash-decoding over paged KV) and its launcher; the device code is
// in decode_splitk.cuh.
#include "decode_splitk.cuh"

namespace ap {

namespace {

using namespace decode;

template <int D>
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_splitk_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
                     const __nv_bfloat16 *__restrict__ q, const DecodeItem *__restrict__ items,
                     const int32_t *__restrict__ cta_begin, const int32_t *__restrict__ bt_flat,
                     const MergeEntry *__restrict__ merges, float *o_part, float *lse_part,
                     __nv_bfloat16 *__restrict__ out, float *__restrict__ lse_out, int Hq, int Hkv, int G, int HB,
                     int n_stages, int n_bufs, int num_pages, float scale_log2, int *status, int *merge_counters,
                     uint64_t wait_limit_ns) {
    decode_cta<D>(k_map, v_map, q, items, cta_begin, bt_flat, merges, o_part, lse_part, out, lse_out, Hq, Hkv, G, HB, n_stages,
                  n_bufs, num_pages, scale_log2, status, merge_counters, wait_limit_ns, (int)blockIdx.x);
}

template <int D>
cudaError_t launch_decode_t(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                            float *o_part, float *lse_part, cudaStream_t stream) {
    using Cfg = DecodeCfg<D>;
    static bool configured[64] = {};
    const int dev = pool->desc.device & 63;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(decode_splitk_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    const float scale_log2 = plan->scale * 1.4426950408889634f;
    cudaError_t e = launch_overlapped(
        decode_splitk_kernel<D>, (unsigned)plan->info.decode_ctas, (unsigned)kDecodeThreads, (size_t)Cfg::kSmemBytes,
        stream, plan->head_block > 1 ? pool->k_map_blk : pool->k_map, plan->head_block > 1 ? pool->v_map_blk : pool->v_map,
        (const __nv_bfloat16 *)q, plan->d_items, plan->d_cta_begin, plan->d_bt_flat,
        plan->d_merge, o_part, lse_part, (__nv_bfloat16 *)out, lse, plan->num_q_heads, pool->desc.num_kv_heads,
        plan->group, plan->head_block, plan->head_block > 1 ? Cfg::kStagesMax : Cfg::kStagesWide,
        plan->head_block > 1 ? 1 : 2, pool->desc.num_pages, scale_log2, pool->status_dev, pool->d_counters, pool->wait_limit_ns);
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

int decode_ctas_per_sm(int head_dim) {
    (void)head_dim;
    return 1;
}

cudaError_t launch_decode_splitk(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out,
                                 float *lse, float *o_part, float *lse_part, cudaStream_t stream) {
    if (pool->desc.head_dim == 128) return launch_decode_t<128>(pool, plan, q, out, lse, o_part, lse_part, stream);
    return launch_decode_t<64>(pool, plan, q, out, lse, o_part, lse_part, stream);
}

}  // namespace ap
