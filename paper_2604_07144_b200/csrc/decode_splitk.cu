// Decode attention: split-K flash-decoding over paged KV (HBM-bound).
//
// A persistent CTA walks its list of work items; an item is the G query heads
// of one kv head of one decode row over a contiguous range of the sequence's
// pages.  One producer warp streams (page, kv head) tiles of K and V -- 4 KB
// each, contiguous in HBM -- into a multi-stage shared-memory ring with TMA
// (128-byte swizzle, completion on mbarriers) and runs ahead across item
// boundaries, so the pipeline never drains while consumers finish an item.
// Eight consumer warps work as two groups of four that take alternate stages of
// the ring (two warps per scheduler hide each other's MMA and shuffle latency);
// within its group's stage a warp owns one page:
//     S^T = K_page Q^T      (mma.sync m16n8k16: M = 16 tokens, N = 8 heads)
//     online softmax over tokens (fp32, warp shuffles across the token lanes)
//     O^T += V_page^T P^T   (M = 16 columns of d per tile, N = 8 heads)
// so every MMA row is a real token and no accumulator register is padding.
// At the end of an item the four warps drop their (m, l, O) into one of two
// shared-memory buffers and move on; a combine warp folds them and writes either
// the final bf16 output (item covers the whole context) or an fp32 partial
// (o normalised, lse), off the consumers' critical path.  A further warp counts the
// CTA's partials in on a device-wide arrival counter per cut stream; the last
// one to arrive merges the stream's partials by log-sum-exp and writes the final
// output while producer and consumers carry on, so no second kernel is needed.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace ap {

namespace {

using namespace ptx;

constexpr int kConsumerWarps = 8;           // two groups of four; a group takes every other stage of the ring
constexpr int kDecodeThreads = (kConsumerWarps + 3) * 32;   // consumers, producer, LSE-merge warp, combine warp
constexpr int kPPS = kDecodePagesPerStage;
// A stream is only ever cut at a CTA boundary, so a CTA holds at most two items
// that produce partials (the planner puts them first in the CTA's list).
constexpr int kMaxPartialItems = 2;
constexpr int kSmemItems = 64;           // item descriptors of a CTA kept in shared memory
static_assert(2 * kPPS == kConsumerWarps, "one page of a stage per warp of a consumer group");

template <int D>
struct DecodeCfg {
    static constexpr int kTileBytes = kPageSize * D * 2;            // one (page, head) tile of one plane
    static constexpr int kQBytes = 8 * D * 2;                       // up to 8 query heads
    static constexpr int kStageBytes = 2 * kPPS * kTileBytes + kQBytes;
    static constexpr int kStages = D == 128 ? 4 : 8;
    static constexpr int kORow = D + 4;                             // padded fp32 row of the merge buffer
    static constexpr int kMergeWarpFloats = 8 * kORow + 16;         // O[8][D+4], m[8], l[8]
    static constexpr int kMergeBytes = 2 * kConsumerWarps * kMergeWarpFloats * 4;   // two buffers
    static constexpr int kBarrierBytes = (2 * kStages + kMaxPartialItems + 4) * 8 + 16 + kSmemItems * 32;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kMergeBytes + kBarrierBytes;
    static_assert(kStageBytes % 1024 == 0, "stages keep the 1024-byte swizzle alignment");
    static_assert(kStages % 2 == 0, "consumer groups own alternate ring slots");
};

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

// byte offset of the 16-byte chunk `chunk` (0 .. D/8-1) of token `tok` (0..15)
// inside a swizzled (page, head) tile: [token/8][half][token%8][64 elements]
template <int D>
__device__ __forceinline__ uint32_t tile_off(int tok, int chunk) {
    return (uint32_t)((tok >> 3) * (1024 * (D / 64)) + (chunk >> 3) * 1024 + (tok & 7) * 128 +
                      (((chunk & 7) ^ (tok & 7)) << 4));
}

// One warp merges the partials of a cut stream,
//   lse = m* + ln sum_k exp(lse_k - m*),  o = sum_k exp(lse_k - lse) o_k,  m* = max_k lse_k,
// and writes the bf16 result.  The merge often sits in the kernel's tail, so it is laid out for
// latency: lane k holds the lse of partial k for all heads (one batch of loads), the weights then
// travel by shuffle, and the o rows are fetched a batch of up to 16 independent 16-byte loads per lane at
// a time (lane = 4 columns of d).  Streams of more than 32 partials take the same path in chunks,
// re-reading the lse values from L2 instead of keeping them in registers.
template <int D, int G>
__device__ __forceinline__ void merge_stream(const MergeEntry me, const float *o_part, const float *lse_part,
                                             __nv_bfloat16 *out, float *lse_out, int Hq, int lane) {
    const int n = me.part_count;
    const float *lse_base = lse_part + (size_t)me.part_begin * G;
    // ---- lse of the whole stream, per head
    float v[G], mx[G], sm[G], lse_tot[G];
#pragma unroll
    for (int h = 0; h < G; ++h) mx[h] = -INFINITY;
    for (int k0 = 0; k0 < n; k0 += 32) {
#pragma unroll
        for (int h = 0; h < G; ++h) v[h] = k0 + lane < n ? __ldcg(lse_base + (size_t)(k0 + lane) * G + h) : -INFINITY;
#pragma unroll
        for (int h = 0; h < G; ++h) mx[h] = fmaxf(mx[h], v[h]);
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
#pragma unroll
        for (int sh = 16; sh >= 1; sh >>= 1) mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], sh));
        sm[h] = 0.f;
    }
    for (int k0 = 0; k0 < n; k0 += 32) {
        if (n > 32) {
#pragma unroll
            for (int h = 0; h < G; ++h)
                v[h] = k0 + lane < n ? __ldcg(lse_base + (size_t)(k0 + lane) * G + h) : -INFINITY;
        }
#pragma unroll
        for (int h = 0; h < G; ++h) sm[h] += __expf(v[h] - mx[h]);
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
#pragma unroll
        for (int sh = 16; sh >= 1; sh >>= 1) sm[h] += __shfl_xor_sync(0xffffffffu, sm[h], sh);
        lse_tot[h] = mx[h] + __logf(sm[h]);
    }
    // ---- weighted sum of the partial outputs
    constexpr int kBatch = G <= 4 ? 16 / G : 1;       // partials fetched per batch (up to 16 loads in flight per lane)
    float4 acc[G];
#pragma unroll
    for (int h = 0; h < G; ++h) acc[h] = make_float4(0.f, 0.f, 0.f, 0.f);
    const bool col_ok = lane * 4 < D;
    const float4 *o_base = reinterpret_cast<const float4 *>(o_part + (size_t)me.part_begin * G * D) + lane;
    for (int c0 = 0; c0 < n; c0 += 32) {
        float w[G];                                    // this lane's partial (c0 + lane): weight per head
        if (n > 32) {
#pragma unroll
            for (int h = 0; h < G; ++h)
                v[h] = c0 + lane < n ? __ldcg(lse_base + (size_t)(c0 + lane) * G + h) : -INFINITY;
        }
#pragma unroll
        for (int h = 0; h < G; ++h) w[h] = __expf(v[h] - lse_tot[h]);
        const int cn = min(32, n - c0);
        for (int k0 = 0; k0 < cn; k0 += kBatch) {
            float4 o[kBatch][G];
#pragma unroll
            for (int kk = 0; kk < kBatch; ++kk)
#pragma unroll
                for (int h = 0; h < G; ++h)
                    o[kk][h] = (k0 + kk < cn && col_ok)
                                   ? __ldcg(o_base + ((size_t)(c0 + k0 + kk) * G + h) * (D / 4))
                                   : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int kk = 0; kk < kBatch; ++kk)
#pragma unroll
                for (int h = 0; h < G; ++h) {
                    const float wk = __shfl_sync(0xffffffffu, w[h], (k0 + kk) & 31);
                    acc[h].x += wk * o[kk][h].x; acc[h].y += wk * o[kk][h].y;
                    acc[h].z += wk * o[kk][h].z; acc[h].w += wk * o[kk][h].w;
                }
        }
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
        if (col_ok) {
            const size_t orow = (size_t)me.q_row * Hq + (size_t)me.kv_head * G + h;
            *reinterpret_cast<uint2 *>(out + orow * D + lane * 4) =
                make_uint2(pack_bf16x2(acc[h].x, acc[h].y), pack_bf16x2(acc[h].z, acc[h].w));
            if (lane == 0 && lse_out) lse_out[orow] = lse_tot[h];
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_splitk_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
                     const __nv_bfloat16 *__restrict__ q, const DecodeItem *__restrict__ items,
                     const int32_t *__restrict__ cta_begin, const int32_t *__restrict__ bt_flat,
                     const MergeEntry *__restrict__ merges, float *o_part, float *lse_part,
                     __nv_bfloat16 *__restrict__ out, float *__restrict__ lse_out, int Hq, int Hkv, int G,
                     int num_pages, float scale_log2, int *status, uint64_t wait_limit_ns) {
    using Cfg = DecodeCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *stages = smem;
    float *merge = (float *)(smem + Cfg::kStages * Cfg::kStageBytes);
    uint64_t *full = (uint64_t *)((uint8_t *)merge + Cfg::kMergeBytes);
    uint64_t *empty = full + Cfg::kStages;
    uint64_t *part_done = empty + Cfg::kStages;      // [kMaxPartialItems], each completes once
    uint64_t *item_done = part_done + kMaxPartialItems;   // [2] consumers -> combine warp, per merge buffer
    uint64_t *buf_free = item_done + 2;                    // [2] combine warp -> consumers
    volatile int *abort_flag = (volatile int *)(buf_free + 2);
    DecodeItem *s_items = (DecodeItem *)(buf_free + 4);
    int *merge_counters = status + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int item_begin = cta_begin[blockIdx.x], item_end = cta_begin[blockIdx.x + 1];

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kConsumerWarps);
        }
        for (int i = 0; i < kMaxPartialItems; ++i) mbar_init(&part_done[i], 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&item_done[i], kConsumerWarps);
            mbar_init(&buf_free[i], 1);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    // The CTA's item descriptors go to shared memory once, so that neither the producer nor the
    // consumers pay a global-memory round trip at every item boundary.
    {
        const int n_ints = min(item_end - item_begin, kSmemItems) * (int)(sizeof(DecodeItem) / 4);
        const int32_t *src = reinterpret_cast<const int32_t *>(items + item_begin);
        for (int i = threadIdx.x; i < n_ints; i += kDecodeThreads) reinterpret_cast<int32_t *>(s_items)[i] = __ldg(src + i);
    }
    __syncthreads();
    auto get_item = [&](int it) -> DecodeItem { return it - item_begin < kSmemItems ? s_items[it - item_begin] : items[it]; };
    // Everything up to here reads only the plan (uploaded before the step's kernels), so it may
    // overlap the tail of the kernel before this one; the pool, q, the partial buffers and the
    // counters may not be touched before that kernel is done.
    griddep_launch_dependents();
    if (warp != kConsumerWarps) griddep_wait();

    int stage = 0;
    uint32_t phase = 0;

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------ producer --
        if (lane == 0) {
            prefetch_tensormap(&k_map);
            prefetch_tensormap(&v_map);
        }
        DecodeItem item = get_item(item_begin);
        int32_t cur = lane < item.page_count ? __ldg(bt_flat + item.bt_offset + item.page_begin + lane) : 0;
        griddep_wait();      // after the first block-table entries are on their way
        for (int it = item_begin; it < item_end; ++it) {
            const int32_t *bt = bt_flat + item.bt_offset + item.page_begin;
            const int npages = item.page_count;
            // block-table entries of the next item's first pages are fetched one item ahead
            DecodeItem next_item = item;
            int32_t next_cur = 0;
            if (it + 1 < item_end) {
                next_item = get_item(it + 1);
                next_cur = lane < next_item.page_count
                               ? __ldg(bt_flat + next_item.bt_offset + next_item.page_begin + lane) : 0;
            }
            for (int p0 = 0; p0 < npages; p0 += 32) {
                const int32_t nxt = p0 + 32 + lane < npages ? __ldg(bt + p0 + 32 + lane) : 0;
                const int ngroup = min(32, npages - p0);
                for (int s0 = 0; s0 < ngroup; s0 += kPPS) {
                    const int n = min(kPPS, ngroup - s0);
                    if (!wait_or_abort(&empty[stage], phase ^ 1, abort_flag, wait_limit_ns)) {
                        atomicCAS(status, 0, AP_ERR_TIMEOUT);
                        *abort_flag = 1;
                        return;
                    }
                    int32_t page = __shfl_sync(0xffffffffu, cur, s0 + (lane & (kPPS - 1)));
                    const bool first = p0 == 0 && s0 < 2 * kPPS;   // each consumer group reads Q from its first stage
                    uint8_t *st = stages + stage * Cfg::kStageBytes;
                    if (lane == 0)
                        mbar_arrive_expect_tx(&full[stage], (uint32_t)(n * 2 * Cfg::kTileBytes +
                                                                      (first ? G * D * 2 : 0)));
                    __syncwarp();
                    if (lane < n) {
                        if (page < 0 || page >= num_pages) {
                            atomicCAS(status, 0, AP_ERR_BAD_BLOCK_TABLE);
                            page = 0;
                        }
                        const int group = (page * Hkv + item.kv_head) * 2;
                        tma_load_4d(st + lane * Cfg::kTileBytes, &k_map, &full[stage], 0, 0, 0, group);
                        tma_load_4d(st + (kPPS + lane) * Cfg::kTileBytes, &v_map, &full[stage], 0, 0, 0, group);
                    } else if (lane == kPPS && first) {
                        bulk_load(st + 2 * kPPS * Cfg::kTileBytes,
                                  q + ((size_t)item.q_row * Hq + (size_t)item.kv_head * G) * D,
                                  (uint32_t)(G * D * 2), &full[stage]);
                    }
                    if (++stage == Cfg::kStages) { stage = 0; phase ^= 1; }
                }
                cur = nxt;
            }
            item = next_item;
            cur = next_cur;
        }
        return;
    }

    if (warp == kConsumerWarps + 1) {
        // ---- LSE merge warp, off the critical path.  For each of this CTA's partial items, once the
        // consumers have written it: count it in on the stream's device-wide arrival counter; the
        // item that completes the count merges all partials of the stream,
        //   lse = m* + ln sum_k exp(lse_k - m*),  o = sum_k exp(lse_k - lse) o_k,  m* = max_k lse_k,
        // and writes the bf16 result.  mbarrier arrive/wait carry the consumers' stores to this
        // warp (release/acquire at CTA scope); the acq_rel atomic publishes them device-wide and
        // acquires the other items' partials.
        for (int pi = 0; pi < kMaxPartialItems && item_begin + pi < item_end; ++pi) {
            const DecodeItem item = get_item(item_begin + pi);
            if (item.part_slot < 0) break;
            const MergeEntry me = merges[item.merge_index];
            if (!wait_or_abort(&part_done[pi], 0, abort_flag, wait_limit_ns)) {
                atomicCAS(status, 0, AP_ERR_TIMEOUT);
                *abort_flag = 1;
                return;
            }
            int last = 0;
            if (lane == 0) {
                int old;
                asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;"
                             : "=r"(old) : "l"(merge_counters + item.merge_index) : "memory");
                last = old == me.part_count - 1;
                if (last) merge_counters[item.merge_index] = 0;      // ready for the next launch
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (!last) continue;
            switch (G) {
                case 1: merge_stream<D, 1>(me, o_part, lse_part, out, lse_out, Hq, lane); break;
                case 2: merge_stream<D, 2>(me, o_part, lse_part, out, lse_out, Hq, lane); break;
                case 3: merge_stream<D, 3>(me, o_part, lse_part, out, lse_out, Hq, lane); break;
                case 4: merge_stream<D, 4>(me, o_part, lse_part, out, lse_out, Hq, lane); break;
                case 5: merge_stream<D, 5>(me, o_part, lse_part, out, lse_out, Hq, lane); break;
                case 6: merge_stream<D, 6>(me, o_part, lse_part, out, lse_out, Hq, lane); break;
                case 7: merge_stream<D, 7>(me, o_part, lse_part, out, lse_out, Hq, lane); break;
                default: merge_stream<D, 8>(me, o_part, lse_part, out, lse_out, Hq, lane); break;
            }
        }
        return;
    }

    if (warp == kConsumerWarps + 2) {
        // ---- combine warp: per item, folds the four consumer warps' (m, l, O) into one result,
        //   m* = max_w m_w,  L = sum_w 2^((m_w - m*) c) l_w,  o = sum_w 2^((m_w - m*) c) O_w / L,
        // and writes the final bf16 output (item covers the whole context) or the fp32 partial.
        const float kLn2 = 0.6931471805599453f;
        const bool col_ok = lane * 4 < D;
        for (int it = item_begin; it < item_end; ++it) {
            const DecodeItem item = get_item(it);
            const int ti = it - item_begin, buf = ti & 1;
            if (!wait_or_abort(&item_done[buf], (uint32_t)(ti >> 1) & 1u, abort_flag, wait_limit_ns)) {
                atomicCAS(status, 0, AP_ERR_TIMEOUT);
                *abort_flag = 1;
                return;
            }
            const float *mb = merge + buf * kConsumerWarps * Cfg::kMergeWarpFloats;
#pragma unroll
            for (int h = 0; h < 8; ++h) {
                if (h >= G) break;
                float mw[kConsumerWarps], mstar = -INFINITY;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    mw[w] = mb[w * Cfg::kMergeWarpFloats + 8 * Cfg::kORow + h];
                    mstar = fmaxf(mstar, mw[w]);
                }
                float L = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float wt = exp2_approx((mw[w] - mstar) * scale_log2);
                    L += wt * mb[w * Cfg::kMergeWarpFloats + 8 * Cfg::kORow + 8 + h];
                    if (col_ok) {
                        const float4 o = *reinterpret_cast<const float4 *>(mb + w * Cfg::kMergeWarpFloats +
                                                                            h * Cfg::kORow + lane * 4);
                        acc.x += wt * o.x; acc.y += wt * o.y; acc.z += wt * o.z; acc.w += wt * o.w;
                    }
                }
                const float inv = 1.f / L;
                const float lse = (mstar * scale_log2 + log2f(L)) * kLn2;
                acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
                if (item.part_slot < 0) {
                    const size_t row = (size_t)item.q_row * Hq + (size_t)item.kv_head * G + h;
                    if (col_ok)
                        *reinterpret_cast<uint2 *>(out + row * D + lane * 4) =
                            make_uint2(pack_bf16x2(acc.x, acc.y), pack_bf16x2(acc.z, acc.w));
                    if (lane == 0 && lse_out) lse_out[row] = lse;
                } else {
                    const size_t row = (size_t)item.part_slot * G + h;
                    if (col_ok) *reinterpret_cast<float4 *>(o_part + row * D + lane * 4) = acc;
                    if (lane == 0) lse_part[row] = lse;
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&buf_free[buf]);
                // the partial is complete: hand it to the merge warp
                if (item.part_slot >= 0 && ti < kMaxPartialItems) mbar_arrive(&part_done[ti]);
            }
        }
        return;
    }

    // ---------------------------------------------------------- consumers --
    const int g = lane >> 2, t = lane & 3;
    const int grp = warp / kPPS, slot = warp % kPPS;

    for (int it = item_begin; it < item_end; ++it) {
        const DecodeItem item = get_item(it);
        const int npages = item.page_count;
        const int valid = min(item.kv_len, (item.page_begin + npages) * kPageSize) - item.page_begin * kPageSize;

        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[D / 16][4];
#pragma unroll
        for (int i = 0; i < D / 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        uint32_t qf[D / 16][2];
        bool have_q = false;

        for (int p0 = 0; p0 < npages; p0 += kPPS) {
            // Every warp passes through every stage, also the other group's: it sees the stage
            // arrive and signs it off.  A stage is refilled only after all eight warps are past it,
            // which keeps every waiter within one phase of each barrier (a parity wait is ambiguous
            // beyond that).
            if (!wait_or_abort(&full[stage], phase, abort_flag, wait_limit_ns)) {
                atomicCAS(status, 0, AP_ERR_TIMEOUT);
                *abort_flag = 1;
                return;
            }
            if ((stage & 1) != grp) {                    // the other group's stage (ring slots alternate)
                if (lane == 0) mbar_arrive(&empty[stage]);
                if (++stage == Cfg::kStages) { stage = 0; phase ^= 1; }
                continue;
            }
            uint8_t *st = stages + stage * Cfg::kStageBytes;
            if (!have_q) {                               // this group's first stage of the item (it carries Q)
                have_q = true;
                // Q^T as the B operand: b0 = Q[head g][16ks + 2t, +1], b1 = Q[head g][16ks + 8 + 2t, +1]
                const uint32_t *qs = (const uint32_t *)(st + 2 * kPPS * Cfg::kTileBytes);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    qf[ks][0] = g < G ? qs[(g * D + ks * 16 + 2 * t) >> 1] : 0u;
                    qf[ks][1] = g < G ? qs[(g * D + ks * 16 + 8 + 2 * t) >> 1] : 0u;
                }
            }
            const int my_page = p0 + slot;
            if (my_page < npages) {
                const int tv = min(kPageSize, valid - my_page * kPageSize);   // valid tokens in this page (>= 1)
                const uint32_t k_tile = smem_u32(st + slot * Cfg::kTileBytes);
                uint8_t *v_ptr = st + (kPPS + slot) * Cfg::kTileBytes;
                const uint32_t v_tile = smem_u32(v_ptr);
                if (tv < kPageSize) {
                    // slots past the context hold no token: clear their V rows so 0 * garbage cannot poison O
                    for (int idx = lane; idx < (kPageSize - tv) * (D / 8); idx += 32) {
                        const int tok = tv + idx / (D / 8), ch = idx % (D / 8);
                        *(uint4 *)(v_ptr + tile_off<D>(tok, ch)) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                }
                // ---- S^T = K Q^T : tokens (g, g+8) x heads (2t, 2t+1)
                float s[4] = {0.f, 0.f, 0.f, 0.f};
                {
                    const int mat = lane >> 3, r = lane & 7;
                    const int tok = (mat & 1) * 8 + r;
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        uint32_t a[4];
                        ldmatrix_x4(a, k_tile + tile_off<D>(tok, 2 * ks + (mat >> 1)));
                        mma_bf16_16816(s, a[0], a[1], a[2], a[3], qf[ks][0], qf[ks][1]);
                    }
                }
                if (g >= tv) s[0] = s[1] = -INFINITY;
                if (g + 8 >= tv) s[2] = s[3] = -INFINITY;
                float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
                for (int sh = 4; sh <= 16; sh <<= 1) {
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
                }
                const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                const float al0 = exp2_approx((m0 - mn0) * scale_log2), al1 = exp2_approx((m1 - mn1) * scale_log2);
                const float ms0 = mn0 * scale_log2, ms1 = mn1 * scale_log2;
                const float p0_ = exp2_approx(s[0] * scale_log2 - ms0), p1_ = exp2_approx(s[1] * scale_log2 - ms1);
                const float p2_ = exp2_approx(s[2] * scale_log2 - ms0), p3_ = exp2_approx(s[3] * scale_log2 - ms1);
                l0 = l0 * al0 + p0_ + p2_;
                l1 = l1 * al1 + p1_ + p3_;
                m0 = mn0;
                m1 = mn1;
#pragma unroll
                for (int i = 0; i < D / 16; ++i) {
                    o[i][0] *= al0; o[i][1] *= al1; o[i][2] *= al0; o[i][3] *= al1;
                }
                // P^T as the B operand: transpose the two 8x8 (token x head) blocks across the warp
                const uint32_t b0 = movmatrix_trans(pack_bf16x2(p0_, p1_));
                const uint32_t b1 = movmatrix_trans(pack_bf16x2(p2_, p3_));
                // ---- O^T += V^T P^T : columns of d (16mt + g, + 8) x heads (2t, 2t+1)
                {
                    const int mat = lane >> 3, r = lane & 7;
                    const int tok = (mat >> 1) * 8 + r;
#pragma unroll
                    for (int mt = 0; mt < D / 16; ++mt) {
                        uint32_t a[4];
                        ldmatrix_x4_trans(a, v_tile + tile_off<D>(tok, 2 * mt + (mat & 1)));
                        mma_bf16_16816(o[mt], a[0], a[1], a[2], a[3], b0, b1);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[stage]);
            if (++stage == Cfg::kStages) { stage = 0; phase ^= 1; }
        }

        // ---- hand (m, l, O) to the combine warp through one of two shared-memory buffers and go on
        // with the next item; the buffer is reused two items later, once the combine warp has freed it
        const int ti = it - item_begin, buf = ti & 1;
        if (!wait_or_abort(&buf_free[buf], ((uint32_t)(ti >> 1) & 1u) ^ 1u, abort_flag, wait_limit_ns)) {
            atomicCAS(status, 0, AP_ERR_TIMEOUT);
            *abort_flag = 1;
            return;
        }
        float *my_merge = merge + (buf * kConsumerWarps + warp) * Cfg::kMergeWarpFloats;
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
            l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
        }
#pragma unroll
        for (int mt = 0; mt < D / 16; ++mt) {
            my_merge[(2 * t) * Cfg::kORow + mt * 16 + g] = o[mt][0];
            my_merge[(2 * t + 1) * Cfg::kORow + mt * 16 + g] = o[mt][1];
            my_merge[(2 * t) * Cfg::kORow + mt * 16 + g + 8] = o[mt][2];
            my_merge[(2 * t + 1) * Cfg::kORow + mt * 16 + g + 8] = o[mt][3];
        }
        if (g == 0) {
            my_merge[8 * Cfg::kORow + 2 * t] = m0;
            my_merge[8 * Cfg::kORow + 2 * t + 1] = m1;
            my_merge[8 * Cfg::kORow + 8 + 2 * t] = l0;
            my_merge[8 * Cfg::kORow + 8 + 2 * t + 1] = l1;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&item_done[buf]);
    }
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
        stream, pool->k_map, pool->v_map, (const __nv_bfloat16 *)q, plan->d_items, plan->d_cta_begin, plan->d_bt_flat,
        plan->d_merge, o_part, lse_part, (__nv_bfloat16 *)out, lse, plan->num_q_heads, pool->desc.num_kv_heads,
        plan->group, pool->desc.num_pages, scale_log2, pool->d_status, pool->wait_limit_ns);
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
