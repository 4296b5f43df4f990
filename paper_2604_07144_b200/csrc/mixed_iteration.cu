// One launch for a mixed iteration: the plan's decode CTAs and its prefill units in a single grid.
// Blocks 0 .. n_decode_ctas - 1 take the decode role (each walks its item list, confined to as many
// SMs); every later block is one prefill unit.  The hardware hands blocks out in index order, so the
// decode CTAs are resident first, the prefill units fill the other SMs, and as decode CTAs retire
// their SMs go over to prefill units: the schedule of the two-stream dispatch without its second
// stream, fork / join events and priorities.  No block waits for another one.
#include "decode_splitk.cuh"
#include "prefill_tcgen05.cuh"

namespace ap {

namespace {

template <int D>
constexpr int mixed_smem_bytes() {
    return decode::DecodeCfg<D>::kSmemBytes > prefill::PrefillCfg<D>::kSmemBytes ? decode::DecodeCfg<D>::kSmemBytes
                                                                                  : prefill::PrefillCfg<D>::kSmemBytes;
}

template <int D>
__global__ void __launch_bounds__(prefill::kPrefillThreads, 1)
mixed_iteration_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                       const __grid_constant__ CUtensorMap v_map, const __grid_constant__ CUtensorMap k_map_blk,
                       const __grid_constant__ CUtensorMap v_map_blk, const __nv_bfloat16 *__restrict__ q,
                       const DecodeItem *__restrict__ items, const int32_t *__restrict__ cta_begin,
                       const int32_t *__restrict__ bt_flat, const MergeEntry *__restrict__ merges, float *o_part,
                       float *lse_part, __nv_bfloat16 *__restrict__ out, float *__restrict__ lse_out,
                       const PrefillTile *__restrict__ tiles, int Hq, int Hkv, int G, int HB, int n_stages, int n_bufs,
                       int num_pages, float scale_log2, int *status, int *merge_counters, uint64_t wait_limit_ns,
                       int n_decode_ctas) {
    static_assert(decode::kDecodeThreads <= prefill::kPrefillThreads, "the block is sized for the larger role");
    if ((int)blockIdx.x < n_decode_ctas) {
        if (threadIdx.x < decode::kDecodeThreads)
            decode::decode_cta<D>(HB > 1 ? k_map_blk : k_map, HB > 1 ? v_map_blk : v_map, q, items, cta_begin, bt_flat, merges,
                                  o_part, lse_part, out, lse_out, Hq, Hkv, G, HB, n_stages, n_bufs, num_pages, scale_log2,
                                  status, merge_counters, wait_limit_ns, (int)blockIdx.x);
    } else {
        prefill::prefill_unit<D>(q_map, k_map, v_map, tiles, bt_flat, out, lse_out, Hq, Hkv, num_pages, scale_log2, status,
                                 wait_limit_ns, (int)blockIdx.x - n_decode_ctas);
    }
}

template <int D>
cudaError_t launch_mixed_t(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse, float *o_part,
                           float *lse_part, cudaStream_t stream) {
    static bool configured[64] = {};
    const int dev = pool->desc.device & 63;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(mixed_iteration_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             mixed_smem_bytes<D>());
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    CUtensorMap q_map;
    if (encode_q_tensor_map(&q_map, q, plan->info.n_new, plan->num_q_heads, D) != AP_OK) return cudaErrorInvalidValue;
    const float scale_log2 = plan->scale * 1.4426950408889634f;
    using DCfg = decode::DecodeCfg<D>;
    const unsigned grid = (unsigned)(plan->info.decode_ctas + plan->info.prefill_tiles);
    cudaError_t e = launch_overlapped(
        mixed_iteration_kernel<D>, grid, (unsigned)prefill::kPrefillThreads, (size_t)mixed_smem_bytes<D>(), stream, q_map,
        pool->k_map, pool->v_map, pool->k_map_blk, pool->v_map_blk, (const __nv_bfloat16 *)q, plan->d_items,
        plan->d_cta_begin, plan->d_bt_flat, plan->d_merge, o_part, lse_part, (__nv_bfloat16 *)out, lse, plan->d_tiles,
        plan->num_q_heads, pool->desc.num_kv_heads, plan->group, plan->head_block,
        plan->head_block > 1 ? DCfg::kStagesMax : DCfg::kStagesWide, plan->head_block > 1 ? 1 : 2, pool->desc.num_pages,
        scale_log2, pool->status_dev, pool->d_counters, pool->wait_limit_ns, (int)plan->info.decode_ctas);
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

cudaError_t launch_mixed_iteration(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                                   float *o_part, float *lse_part, cudaStream_t stream) {
    if (pool->desc.head_dim == 128) return launch_mixed_t<128>(pool, plan, q, out, lse, o_part, lse_part, stream);
    return launch_mixed_t<64>(pool, plan, q, out, lse, o_part, lse_part, stream);
}

}  // namespace ap
