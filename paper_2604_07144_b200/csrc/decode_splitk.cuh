// Decode attention: split-K flash-decoding over paged KV (HBM-bound).
//
// A persistent CTA walks its list of work items; an item is the query heads of a
// block of HB consecutive kv heads (HB = 4, 2 or 1) of one decode row over a
// contiguous range of the sequence's pages.  One producer warp streams K and V
// into a multi-stage shared-memory ring with TMA (128-byte swizzle, completion on
// mbarriers), one request per page and plane for the HB (page, kv head) tiles
// that lie together in HBM (16 KB at HB = 4, d = 128: the TMA unit of an SM
// sustains ~58 GB/s in 4 KB requests but over 100 GB/s in 16 KB ones), and runs
// ahead across item boundaries, so the pipeline never drains while consumers
// finish an item.  Eight consumer warps work as two groups of four that take
// alternate stages of the ring (two warps per scheduler hide each other's MMA and
// shuffle latency); a stage holds four tiles per plane (4 / HB pages of HB heads)
// and within its group's stage a warp owns one (page, kv head) tile:
//     S^T = K_page Q^T      (mma.sync m16n8k16: M = 16 tokens, N = 8 heads)
//     online softmax over tokens (fp32, warp shuffles across the token lanes)
//     O^T += V_page^T P^T   (M = 16 columns of d per tile, N = 8 heads)
// so every MMA row is a real token and no accumulator register is padding.
// At the end of an item the eight warps drop their (m, l, O) into a
// shared-memory buffer and move on; a combine warp folds those of the same kv head and writes either
// the final bf16 output (item covers the whole context) or an fp32 partial
// (o normalised, lse), off the consumers' critical path.  A further warp counts the
// CTA's partials in on a device-wide arrival counter per cut stream; the last
// one to arrive merges the stream's partials by log-sum-exp and writes the final
// output while producer and consumers carry on, so no second kernel is needed.
#pragma once

#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace ap {
namespace decode {

using namespace ptx;

constexpr int kConsumerWarps = 8;           // two groups of four; a group takes every other stage of the ring
constexpr int kDecodeThreads = (kConsumerWarps + 3) * 32;   // consumers, producer, LSE-merge warp, combine warp
constexpr int kTPS = kDecodeTilesPerStage;   // tiles of one plane per stage
constexpr int kSmemItems = 32;           // item descriptors of a CTA kept in shared memory
constexpr int kMaxItemHeads = 32;        // query heads of an item: at most 4 kv heads x 8 query heads each
static_assert(2 * kTPS == kConsumerWarps, "one tile of a stage per warp of a consumer group");

template <int D>
struct DecodeCfg {
    static constexpr int kTileBytes = kPageSize * D * 2;            // one (page, head) tile of one plane
    static constexpr int kStageBytes = 2 * kTPS * kTileBytes;       // K tiles, then V tiles
    static constexpr int kORow = D + 4;                             // padded fp32 row of the merge buffer
    static constexpr int kMergeWarpFloats = 8 * kORow + 16;         // O[8][D+4], m[8], l[8]
    static constexpr int kMergeBytes = kConsumerWarps * kMergeWarpFloats * 4 + 32; // one hand-over buffer: the warps' data, then the item
    static constexpr int kQBytes = kMaxItemHeads * D * 2;           // the query heads of one item; two buffers
    // Two ways to spend the same shared memory (the kernel takes the pair as arguments):
    //   whole-GPU decode, one kv head per item: many short items, so two hand-over buffers keep the
    //     consumers from waiting on the combine warp; 4 stages of 32 KB are plenty at ~41 GB/s per SM;
    //   decode confined to k SMs, a block of kv heads per item: few long items, one buffer will do; the
    //     ring gets a 5th stage, because an SM's rate is (bytes in flight) / (memory latency) and two
    //     stages are always held by the consumer groups.
    static constexpr int kStagesMax = (D == 128 ? 5 : 10);
    static constexpr int kStagesWide = (D == 128 ? 4 : 8);
    static constexpr int kBarrierBytes = (2 * kStagesMax + 8 + 2) * 8 + 16 + kSmemItems * 32;
    static constexpr int kRingAndBuffers = kStagesMax * kStageBytes + kMergeBytes > kStagesWide * kStageBytes + 2 * kMergeBytes
                                               ? kStagesMax * kStageBytes + kMergeBytes
                                               : kStagesWide * kStageBytes + 2 * kMergeBytes;
    static constexpr int kSmemBytes = 1024 + kRingAndBuffers + 2 * kQBytes + kBarrierBytes;
    static_assert(kSmemBytes <= 227 * 1024, "fits the shared memory of an SM");
    static_assert(kStageBytes % 1024 == 0, "stages keep the 1024-byte swizzle alignment");
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
// A partial holds PH heads (those of the item's kv head block); one call merges G of them, heads
// h0 .. h0 + G - 1 of the partial, which are query heads first_q_head + h0 ... of the row.
template <int D, int G>
__device__ __forceinline__ void merge_stream(const MergeEntry me, const float *o_part, const float *lse_part,
                                             __nv_bfloat16 *out, float *lse_out, int Hq, int lane, int PH, int h0,
                                             int first_q_head) {
    const int n = me.part_count;
    const float *lse_base = lse_part + (size_t)me.part_begin * PH + h0;
    // ---- lse of the whole stream, per head
    float v[G], mx[G], sm[G], lse_tot[G];
#pragma unroll
    for (int h = 0; h < G; ++h) mx[h] = -INFINITY;
    for (int k0 = 0; k0 < n; k0 += 32) {
#pragma unroll
        for (int h = 0; h < G; ++h) v[h] = k0 + lane < n ? __ldcg(lse_base + (size_t)(k0 + lane) * PH + h) : -INFINITY;
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
                v[h] = k0 + lane < n ? __ldcg(lse_base + (size_t)(k0 + lane) * PH + h) : -INFINITY;
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
    const float4 *o_base = reinterpret_cast<const float4 *>(o_part + ((size_t)me.part_begin * PH + h0) * D) + lane;
    for (int c0 = 0; c0 < n; c0 += 32) {
        float w[G];                                    // this lane's partial (c0 + lane): weight per head
        if (n > 32) {
#pragma unroll
            for (int h = 0; h < G; ++h)
                v[h] = c0 + lane < n ? __ldcg(lse_base + (size_t)(c0 + lane) * PH + h) : -INFINITY;
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
                                   ? __ldcg(o_base + ((size_t)(c0 + k0 + kk) * PH + h) * (D / 4))
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
            const size_t orow = (size_t)me.q_row * Hq + (size_t)(first_q_head + h0 + h);
            *reinterpret_cast<uint2 *>(out + orow * D + lane * 4) =
                make_uint2(pack_bf16x2(acc[h].x, acc[h].y), pack_bf16x2(acc[h].z, acc[h].w));
            if (lane == 0 && lse_out) lse_out[orow] = lse_tot[h];
        }
    }
}

// Folds, for one item, the consumer warps' (m, l, O) per kv head of the item's block (HB heads; the
// 8 / HB warps hh, hh + HB, ... worked on head hh) and writes the bf16 output or the fp32 partial.
template <int D, int HB>
__device__ __forceinline__ void combine_item(const DecodeItem item, const float *mb, int G, int Hq, float scale_log2,
                                             __nv_bfloat16 *out, float *lse_out, float *o_part, float *lse_part, int lane) {
    using Cfg = DecodeCfg<D>;
    constexpr int kWarpsPerHead = kConsumerWarps / HB;
    const float kLn2 = 0.6931471805599453f;
    const bool col_ok = lane * 4 < D;
    const int PH = HB * G;
#pragma unroll
    for (int hh = 0; hh < HB; ++hh) {
#pragma unroll
        for (int h = 0; h < 8; ++h) {
            if (h >= G) break;
            float mw[kWarpsPerHead], mstar = -INFINITY;
#pragma unroll
            for (int i = 0; i < kWarpsPerHead; ++i) {
                mw[i] = mb[(hh + i * HB) * Cfg::kMergeWarpFloats + 8 * Cfg::kORow + h];
                mstar = fmaxf(mstar, mw[i]);
            }
            float L = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int i = 0; i < kWarpsPerHead; ++i) {
                const float *wb = mb + (hh + i * HB) * Cfg::kMergeWarpFloats;
                const float wt = exp2_approx((mw[i] - mstar) * scale_log2);
                L += wt * wb[8 * Cfg::kORow + 8 + h];
                if (col_ok) {
                    const float4 o = *reinterpret_cast<const float4 *>(wb + h * Cfg::kORow + lane * 4);
                    acc.x += wt * o.x; acc.y += wt * o.y; acc.z += wt * o.z; acc.w += wt * o.w;
                }
            }
            const float inv = 1.f / L;
            const float lse = (mstar * scale_log2 + log2f(L)) * kLn2;
            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
            if (item.part_slot < 0) {
                const size_t row = (size_t)item.q_row * Hq + (size_t)(item.kv_head + hh) * G + h;
                if (col_ok)
                    *reinterpret_cast<uint2 *>(out + row * D + lane * 4) =
                        make_uint2(pack_bf16x2(acc.x, acc.y), pack_bf16x2(acc.z, acc.w));
                if (lane == 0 && lse_out) lse_out[row] = lse;
            } else {
                const size_t row = (size_t)item.part_slot * PH + hh * G + h;
                if (col_ok) *reinterpret_cast<float4 *>(o_part + row * D + lane * 4) = acc;
                if (lane == 0) lse_part[row] = lse;
            }
        }
    }
}

// The work of one decode CTA: list number `cta` of the plan.  Called by kDecodeThreads threads of a CTA
// (any further threads of the block must not call it).
template <int D>
__device__ __forceinline__ void decode_cta(const CUtensorMap &k_map, const CUtensorMap &v_map, const __nv_bfloat16 *__restrict__ q,
                                           const DecodeItem *__restrict__ items, const int32_t *__restrict__ cta_begin,
                                           const int32_t *__restrict__ bt_flat, const MergeEntry *__restrict__ merges,
                                           float *o_part, float *lse_part, __nv_bfloat16 *__restrict__ out,
                                           float *__restrict__ lse_out, int Hq, int Hkv, int G, int HB, int n_stages, int n_bufs,
                                           int num_pages, float scale_log2, int *status, int *merge_counters,
                                           uint64_t wait_limit_ns, int cta) {
    using Cfg = DecodeCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *stages = smem;
    float *merge = (float *)(smem + n_stages * Cfg::kStageBytes);    // [n_bufs] hand-over buffers
    uint8_t *q_buf = (uint8_t *)merge + n_bufs * Cfg::kMergeBytes;   // [2][kQBytes]
    uint64_t *full = (uint64_t *)(q_buf + 2 * Cfg::kQBytes);
    uint64_t *empty = full + Cfg::kStagesMax;
    uint64_t *item_done = empty + Cfg::kStagesMax;         // [2] consumers -> combine warp, per hand-over buffer
    uint64_t *buf_free = item_done + 2;                    // [2] combine warp -> consumers
    uint64_t *q_full = buf_free + 2;                       // [2] an item's query heads have landed
    uint64_t *q_empty = q_full + 2;                        // [2] all consumer warps have taken their fragments
    uint64_t *merge_req = q_empty + 2;                     // combine warp -> merge warp: a stream is complete
    uint64_t *merge_ack = merge_req + 1;                   // merge warp -> combine warp: request taken care of
    volatile int *abort_flag = (volatile int *)(merge_ack + 1);
    volatile int *merge_idx = abort_flag + 1;              // the request: index of the merge entry, or -1: no more
    DecodeItem *s_items = (DecodeItem *)(merge_ack + 3);   // [kSmemItems] the head of the CTA's list

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int item_begin = cta_begin[cta], n_items = cta_begin[cta + 1] - item_begin;
    const int PS = kTPS / HB;        // pages of an item per stage
    const int PH = HB * G;           // query heads of an item (and of a partial)

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kConsumerWarps);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&item_done[i], kConsumerWarps);
            mbar_init(&buf_free[i], 1);
            mbar_init(&q_full[i], 1);
            mbar_init(&q_empty[i], kConsumerWarps);
        }
        mbar_init(merge_req, 1);
        mbar_init(merge_ack, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    // The CTA's item descriptors go to shared memory once, so that neither the producer nor the
    // consumers pay a global-memory round trip at every item boundary.
    {
        const int n_ints = min(n_items, kSmemItems) * (int)(sizeof(DecodeItem) / 4);
        const int32_t *src = reinterpret_cast<const int32_t *>(items + item_begin);
        for (int i = threadIdx.x; i < n_ints; i += kDecodeThreads) reinterpret_cast<int32_t *>(s_items)[i] = __ldg(src + i);
    }
    named_barrier_sync(1, kDecodeThreads);      // the threads of this role only (the block may hold more)
    // Item number n of this CTA's list; page_count 0 past its end.
    auto get_item = [&](int n) {
        DecodeItem item{};
        if (n < n_items) item = n < kSmemItems ? s_items[n] : items[item_begin + n];
        return item;
    };
    // Everything up to here reads only the plan (uploaded before the step's kernels), so it may
    // overlap the tail of the kernel before this one; the pool, q, the partial buffers and the
    // counters may not be touched before that kernel is done.
    griddep_launch_dependents();
    if (warp != kConsumerWarps) griddep_wait();

    // Ring position: stage slot, phase of its barriers, and which consumer group the stage belongs to
    // (the stages of an item go to the two groups in turn, whatever the number of slots).
    int stage = 0, turn = 0;
    uint32_t phase = 0;
    auto advance = [&]() {
        if (++stage == n_stages) { stage = 0; phase ^= 1; }
        turn ^= 1;
    };

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------ producer --
        if (lane == 0) {
            prefetch_tensormap(&k_map);
            prefetch_tensormap(&v_map);
        }
        DecodeItem item = get_item(0);
        int32_t cur = lane < item.page_count ? __ldg(bt_flat + item.bt_offset + item.page_begin + lane) : 0;
        griddep_wait();      // after the first block-table entries are on their way
        const uint32_t page_bytes = (uint32_t)(2 * HB * Cfg::kTileBytes);   // K and V tiles of one page of the block
        // a decode stream is read once: its lines should be the first to leave the L2 (next to a prefill
        // kernel, whose units read the same K/V tiles again and again, they would otherwise push those out)
        const uint64_t stream_once = l2_policy_evict_first();
        for (int n = 0; item.page_count > 0; ++n) {
            const int32_t *bt = bt_flat + item.bt_offset + item.page_begin;
            const int npages = item.page_count;
            // the first block-table entries of the next item are fetched one item ahead
            const DecodeItem next = get_item(n + 1);
            const int32_t next_cur = lane < next.page_count ? __ldg(bt_flat + next.bt_offset + next.page_begin + lane) : 0;
            {
                // the item's query heads (PH * D contiguous bf16) go ahead of its first stage, into the
                // buffer the item before last used
                const int qb = n & 1;
                if (!wait_or_abort(&q_empty[qb], (((uint32_t)n >> 1) & 1u) ^ 1u, abort_flag, wait_limit_ns)) {
                    record_status(status, AP_ERR_TIMEOUT);
                    *abort_flag = 1;
                    return;
                }
                if (lane == 0) {
                    mbar_arrive_expect_tx(&q_full[qb], (uint32_t)(PH * D * 2));
                    bulk_load(q_buf + qb * Cfg::kQBytes, q + ((size_t)item.q_row * Hq + (size_t)item.kv_head * G) * D,
                              (uint32_t)(PH * D * 2), &q_full[qb]);
                }
                __syncwarp();
            }
            for (int p0 = 0; p0 < npages; p0 += 32) {
                const int32_t nxt = p0 + 32 + lane < npages ? __ldg(bt + p0 + 32 + lane) : 0;
                const int ngroup = min(32, npages - p0);
                for (int s0 = 0; s0 < ngroup; s0 += PS) {
                    const int np = min(PS, ngroup - s0);
                    if (!wait_or_abort(&empty[stage], phase ^ 1, abort_flag, wait_limit_ns)) {
                        record_status(status, AP_ERR_TIMEOUT);
                        *abort_flag = 1;
                        return;
                    }
                    int32_t page = __shfl_sync(0xffffffffu, cur, s0 + (lane & (PS - 1)));
                    uint8_t *st = stages + stage * Cfg::kStageBytes;
                    if (lane == 0) mbar_arrive_expect_tx(&full[stage], (uint32_t)np * page_bytes);
                    __syncwarp();
                    if (lane < np) {
                        if (page < 0 || page >= num_pages) {
                            record_status(status, AP_ERR_BAD_BLOCK_TABLE);
                            page = 0;
                        }
                        // one request per plane: the HB tiles of this page that belong to the item's kv heads
                        const int group = (page * Hkv + item.kv_head) * 2;
                        tma_load_4d_hint(st + lane * HB * Cfg::kTileBytes, &k_map, &full[stage], 0, 0, 0, group, stream_once);
                        tma_load_4d_hint(st + (kTPS + lane * HB) * Cfg::kTileBytes, &v_map, &full[stage], 0, 0, 0, group, stream_once);
                    }
                    advance();
                }
                cur = nxt;
            }
            item = next;
            cur = next_cur;
        }
        return;
    }

    if (warp == kConsumerWarps + 1) {
        // ---- LSE merge warp, off everybody's path: when the combine warp has counted in the last
        // partial of a stream it asks this warp to merge the stream's partials,
        //   lse = m* + ln sum_k exp(lse_k - m*),  o = sum_k exp(lse_k - lse) o_k,  m* = max_k lse_k,
        // and to write the bf16 result.  (The counting atomic is acq_rel at device scope: it publishes
        // this CTA's partial and acquires the others'; the request barrier carries that on to this warp.)
        for (uint32_t r = 0;; ++r) {
            if (!wait_or_abort(merge_req, r & 1u, abort_flag, wait_limit_ns)) {
                record_status(status, AP_ERR_TIMEOUT);
                *abort_flag = 1;
                return;
            }
            const int idx = *merge_idx;
            if (idx < 0) return;
            const MergeEntry me = merges[idx];
            __syncwarp();
            if (lane == 0) mbar_arrive(merge_ack);         // the request word may be reused
            // the PH heads of the stream, up to eight per pass (what one warp can keep in registers)
            const int fq = me.kv_head * G;
            int h0 = 0;
            for (; h0 + 8 <= PH; h0 += 8) merge_stream<D, 8>(me, o_part, lse_part, out, lse_out, Hq, lane, PH, h0, fq);
            switch (PH - h0) {
                case 1: merge_stream<D, 1>(me, o_part, lse_part, out, lse_out, Hq, lane, PH, h0, fq); break;
                case 2: merge_stream<D, 2>(me, o_part, lse_part, out, lse_out, Hq, lane, PH, h0, fq); break;
                case 3: merge_stream<D, 3>(me, o_part, lse_part, out, lse_out, Hq, lane, PH, h0, fq); break;
                case 4: merge_stream<D, 4>(me, o_part, lse_part, out, lse_out, Hq, lane, PH, h0, fq); break;
                case 5: merge_stream<D, 5>(me, o_part, lse_part, out, lse_out, Hq, lane, PH, h0, fq); break;
                case 6: merge_stream<D, 6>(me, o_part, lse_part, out, lse_out, Hq, lane, PH, h0, fq); break;
                case 7: merge_stream<D, 7>(me, o_part, lse_part, out, lse_out, Hq, lane, PH, h0, fq); break;
                default: break;
            }
        }
    }

    if (warp == kConsumerWarps + 2) {
        // ---- combine warp: per item and kv head of its block, folds the (m, l, O) of the consumer
        // warps that worked on that head (warps hh, hh + HB, ...) into one result,
        //   m* = max_w m_w,  L = sum_w 2^((m_w - m*) c) l_w,  o = sum_w 2^((m_w - m*) c) O_w / L,
        // and writes the final bf16 output (item covers the whole context) or the fp32 partial.  A
        // partial is then counted in on its stream's device-wide arrival counter; the one that
        // completes the count has the merge warp merge the stream.  The item's description comes with
        // the consumers' data (this warp may be an item or two behind them).
        uint32_t requests = 0;
        auto post = [&](int idx) {                // to the merge warp; waits for the request before to be taken
            if (requests > 0 && !wait_or_abort(merge_ack, (requests - 1) & 1u, abort_flag, wait_limit_ns)) return false;
            if (lane == 0) {
                *merge_idx = idx;
                mbar_arrive(merge_req);
            }
            ++requests;
            return true;
        };
        for (int n = 0;; ++n) {
            const int buf = n % n_bufs;
            if (!wait_or_abort(&item_done[buf], (uint32_t)(n / n_bufs) & 1u, abort_flag, wait_limit_ns)) {
                record_status(status, AP_ERR_TIMEOUT);
                *abort_flag = 1;
                return;
            }
            const float *mb = merge + buf * (Cfg::kMergeBytes / 4);
            const DecodeItem item = *reinterpret_cast<const DecodeItem *>(mb + kConsumerWarps * Cfg::kMergeWarpFloats);
            if (item.page_count == 0) break;                       // the consumers are through
            switch (HB) {
                case 4: combine_item<D, 4>(item, mb, G, Hq, scale_log2, out, lse_out, o_part, lse_part, lane); break;
                case 2: combine_item<D, 2>(item, mb, G, Hq, scale_log2, out, lse_out, o_part, lse_part, lane); break;
                default: combine_item<D, 1>(item, mb, G, Hq, scale_log2, out, lse_out, o_part, lse_part, lane); break;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&buf_free[buf]);
            if (item.part_slot >= 0) {
                int last = 0;
                if (lane == 0) {
                    int old;
                    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;"
                                 : "=r"(old) : "l"(merge_counters + item.merge_index) : "memory");
                    last = old == __ldg(&merges[item.merge_index].part_count) - 1;
                    if (last) merge_counters[item.merge_index] = 0;      // ready for the next launch
                }
                last = __shfl_sync(0xffffffffu, last, 0);
                if (last && !post(item.merge_index)) {
                    record_status(status, AP_ERR_TIMEOUT);
                    *abort_flag = 1;
                    return;
                }
            }
        }
        if (!post(-1)) {
            record_status(status, AP_ERR_TIMEOUT);
            *abort_flag = 1;
        }
        return;
    }

    // ---------------------------------------------------------- consumers --
    const int g = lane >> 2, t = lane & 3;
    const int grp = warp / kTPS, slot = warp % kTPS;
    const int my_head = slot % HB, my_pg = slot / HB;      // this warp's tile in a stage: kv head of the block, page of the stage

    for (int n = 0;; ++n) {
        const DecodeItem item = get_item(n);
        const int buf = n % n_bufs;
        float *hand_over = merge + buf * (Cfg::kMergeBytes / 4);
        if (item.page_count == 0) {
            // no more items: tell the combine warp through the hand-over buffer
            if (!wait_or_abort(&buf_free[buf], ((uint32_t)(n / n_bufs) & 1u) ^ 1u, abort_flag, wait_limit_ns)) {
                record_status(status, AP_ERR_TIMEOUT);
                *abort_flag = 1;
                return;
            }
            if (warp == 0 && lane == 0) *reinterpret_cast<DecodeItem *>(hand_over + kConsumerWarps * Cfg::kMergeWarpFloats) = item;
            __syncwarp();
            if (lane == 0) mbar_arrive(&item_done[buf]);
            return;
        }
        const int npages = item.page_count;
        const int valid = min(item.kv_len, (item.page_begin + npages) * kPageSize) - item.page_begin * kPageSize;
        turn = 0;    // an item's first stage goes to group 0 whatever came before

        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[D / 16][4];
#pragma unroll
        for (int i = 0; i < D / 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        // Q^T as the B operand: b0 = Q[head g][16ks + 2t, +1], b1 = Q[head g][16ks + 8 + 2t, +1], for the G query
        // heads of this warp's kv head; taken once per item from the buffer the producer filled
        uint32_t qf[D / 16][2];
        {
            const int qb = n & 1;
            if (!wait_or_abort(&q_full[qb], ((uint32_t)n >> 1) & 1u, abort_flag, wait_limit_ns)) {
                record_status(status, AP_ERR_TIMEOUT);
                *abort_flag = 1;
                return;
            }
            const uint32_t *qs = reinterpret_cast<const uint32_t *>(q_buf + qb * Cfg::kQBytes) + ((my_head * G * D) >> 1);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                qf[ks][0] = g < G ? qs[(g * D + ks * 16 + 2 * t) >> 1] : 0u;
                qf[ks][1] = g < G ? qs[(g * D + ks * 16 + 8 + 2 * t) >> 1] : 0u;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&q_empty[qb]);
        }

        for (int p0 = 0; p0 < npages; p0 += PS) {
            // Every warp passes through every stage, also the other group's: it sees the stage
            // arrive and signs it off.  A stage is refilled only after all eight warps are past it,
            // which keeps every waiter within one phase of each barrier (a parity wait is ambiguous
            // beyond that).
            if (!wait_or_abort(&full[stage], phase, abort_flag, wait_limit_ns)) {
                record_status(status, AP_ERR_TIMEOUT);
                *abort_flag = 1;
                return;
            }
            if (turn != grp) {                           // the other group's stage
                if (lane == 0) mbar_arrive(&empty[stage]);
                advance();
                continue;
            }
            uint8_t *st = stages + stage * Cfg::kStageBytes;
            const int my_page = p0 + my_pg;
            if (my_page < npages) {
                const int tv = min(kPageSize, valid - my_page * kPageSize);   // valid tokens in this page (>= 1)
                const uint32_t k_tile = smem_u32(st + slot * Cfg::kTileBytes);
                uint8_t *v_ptr = st + (kTPS + slot) * Cfg::kTileBytes;
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
            advance();
        }

        // ---- hand (m, l, O) and the item's description to the combine warp through a shared-memory
        // buffer and go on with the next item; a buffer is free again once the combine warp has folded
        // the item that used it
        if (!wait_or_abort(&buf_free[buf], ((uint32_t)(n / n_bufs) & 1u) ^ 1u, abort_flag, wait_limit_ns)) {
            record_status(status, AP_ERR_TIMEOUT);
            *abort_flag = 1;
            return;
        }
        float *my_merge = hand_over + warp * Cfg::kMergeWarpFloats;
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
        if (warp == 0 && lane == 0) *reinterpret_cast<DecodeItem *>(hand_over + kConsumerWarps * Cfg::kMergeWarpFloats) = item;
        __syncwarp();
        if (lane == 0) mbar_arrive(&item_done[buf]);
    }
}

}  // namespace decode
}  // namespace ap
