// Prefill-chunk attention: causal tiled attention on tcgen05 tensor cores with
// accumulators in tensor memory (TMEM).
//
// One CTA handles one work unit: 128 consecutive query rows of one sequence for
// TWO q heads of the same kv head (tiles A and B; B may be absent), over keys
// 0 .. (position of the last row).  Both tiles consume the same K/V stream, which
// comes through the block table, one TMA per (page, kv head) tile, straight into
// the 128-byte-swizzled operand layout tcgen05.mma reads.
//
//   warps 0-3   softmax group A: thread r owns query row r of tile A (= TMEM lane r)
//   warps 4-7   softmax group B: same for tile B
//               per step of 128 keys: read S from TMEM, mask, running max / sum in
//               fp32, write P (bf16) back into the S columns of TMEM as the A operand
//               of the second product, rescale O in TMEM when the running max has
//               moved enough, and write the normalised output at the end
//   warp 8      producer: Q tiles once, then K and V tiles into one 5-slot ring
//   warps 9, 10 MMA issuers, one per tile (converged warp, one elected lane issues): S = Q_x K^T, O_x += P_x V;
//               the tensor pipe works on one tile while the other tile's softmax runs
//   warp 11     idle (it only completes the third warpgroup for the register split)
//
// TMEM columns: S 0-127 (ONE score region that tiles A and B use in turn), P_A 128-191, P_B 192-255,
// O_A 256-.., O_B 384-.. (512 allocated).  A softmax group copies its S tile into registers at once and
// hands the region back (s_out), and P has columns of its own, so the next scores of a tile,
// S_x(j+1), do not have to wait for O_x += P_x(j) V: they are issued ahead of it.  The order on the
// tensor pipe is  S_A(j+1), P_A(j) V, S_B(j+1), P_B(j) V;  per tile only softmax(j) -> softmax(j+1)
// remains as a chain, instead of softmax -> P V -> Q K^T -> softmax.
// Registers: the block is launched with 168 registers per thread; the third
// warpgroup drops to 72 and the two softmax groups raise themselves to 216
// (128 * 72 + 256 * 216 = 384 * 168), so a whole S row fits in registers.
//
// Every wait is bounded; a wait that runs out records AP_ERR_TIMEOUT, raises the
// CTA's abort flag, and all roles fall through to the common exit where TMEM is
// released.
#pragma once

#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace ap {
namespace prefill {

using namespace ptx;

constexpr int kTileM = 128;                 // query rows per tile
constexpr int kTileN = 128;                 // keys per step (8 pages)
constexpr int kPagesPerTile = kTileN / kPageSize;
// K and V tiles share one ring of 32 KB slots, filled in the order K_0, K_1, V_0, K_2, V_1, ...
// (K one step ahead: S(j+1) is issued right after P V of step j).  While one K and one V tile are
// being consumed, three slots (96 KB) are in flight, which covers the L2 latency at full MMA rate;
// separate 3 + 2 rings left only one V tile in flight and made the V arrival the period.
constexpr int kKvSlots = 5;
__host__ __device__ constexpr int kv_seq_k(int j) { return j == 0 ? 0 : 2 * j - 1; }
__host__ __device__ inline int kv_seq_v(int j, int n_steps) { return min(2 * j + 2, 2 * n_steps - 1); }
constexpr int kPrefillThreads = 384;
constexpr int kProducerWarp = 8, kMmaWarp = 9;
constexpr float kRescaleThreshold = 8.0f;   // in log2 units: P stays below 2^8

template <int D>
struct PrefillCfg {
    static constexpr int kHalves = D / 64;
    static constexpr int kPageTileBytes = kPageSize * D * 2;
    static constexpr int kQBytes = kTileM * D * 2;
    static constexpr int kKvTileBytes = kTileN * D * 2;
    static constexpr int kOffQ = 0;                                   // [2] tiles A, B
    static constexpr int kOffK = kOffQ + 2 * kQBytes;
    static constexpr int kOffBar = kOffK + kKvSlots * kKvTileBytes;
    static constexpr int kSmemBytes = 1024 + kOffBar + 256;
    static constexpr uint32_t kTmemCols = 512;
    static constexpr uint32_t kColS = 0;      // shared by both tiles
    static constexpr uint32_t kColP = 128;    // + 64 * tile (bf16 pairs)
    static constexpr uint32_t kColO = 256;    // + 128 * tile
};

// three-input maximum (one instruction on sm_100)
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// 2^x for two values on the FMA pipe (relieves the special-function unit, which would otherwise
// bound the softmax): x = n + f with n = round(x), f in [-0.5, 0.5]; 2^f by a cubic fitted for
// relative error (7.7e-5, well inside the bf16 rounding P gets anyway); 2^n by adding n to the
// exponent field.  x is clamped at -125 so the exponent cannot wrap (2^-125 is zero for our purposes).
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
    const float kMagic = 12582912.f;                       // 1.5 * 2^23: x + kMagic holds round(x) in its low bits
    x.x = fmaxf(x.x, -125.f);
    x.y = fmaxf(x.y, -125.f);
    const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
    const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
    const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
    float2 p = __ffma2_rn(f, make_float2(0.05508868f, 0.05508868f), make_float2(0.24260405f, 0.24260405f));
    p = __ffma2_rn(p, f, make_float2(0.69327624f, 0.69327624f));
    p = __ffma2_rn(p, f, make_float2(0.99992894f, 0.99992894f));
    p.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
    p.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
    return p;
}

// Shared-memory matrix descriptor for tcgen05.mma, 128-byte swizzle:
// start address, leading / stride byte offsets (all >> 4), descriptor version 1
// (bits 46-47), layout type SWIZZLE_128B = 2 (bits 61-63).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor, kind::f16: D = fp32 (bits 4-5 = 1), A = B = bf16
// (bits 7-9, 10-12 = 1), B major-ness in bit 16 (0 = K-major, 1 = MN-major),
// N >> 3 in bits 17-22, M >> 4 in bits 24-28.
__host__ __device__ constexpr uint32_t instr_desc(int m, int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(m >> 4) << 24);
}

// O (this thread's row, D fp32 columns in tensor memory) *= alpha.  Rare (the reference maximum moves
// by more than the threshold only in a row's first steps), so it is kept out of line: the softmax loop
// stays short and its registers are not shared with this path.
template <int D>
__device__ __noinline__ void rescale_o(uint32_t taddr, float alpha) {
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        uint32_t oreg[32];
        tmem_ld_32x32b_x32(taddr + c * 32, oreg);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) oreg[i] = __float_as_uint(__uint_as_float(oreg[i]) * alpha);
        tmem_st_32x32b_x32(taddr + c * 32, oreg);
    }
}

// One work unit: entry `unit` of the plan's list.  Called by all kPrefillThreads threads of a CTA.
template <int D>
__device__ __forceinline__ void prefill_unit(const CUtensorMap &q_map, const CUtensorMap &k_map, const CUtensorMap &v_map,
                                             const PrefillTile *__restrict__ tiles, const int32_t *__restrict__ bt_flat,
                                             __nv_bfloat16 *__restrict__ out, float *__restrict__ lse_out, int Hq, int Hkv,
                                             int num_pages, float scale_log2, int *status, uint64_t wait_limit_ns, int unit) {
    using Cfg = PrefillCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + Cfg::kOffBar);
    uint64_t *q_full = bars + 0;
    uint64_t *kv_full = bars + 1;                // [kKvSlots]
    uint64_t *kv_empty = kv_full + kKvSlots;     // [kKvSlots]
    uint64_t *s_full = kv_empty + kKvSlots;      // [2] per tile
    uint64_t *p_full = s_full + 2;               // [2]
    uint64_t *pv_done = p_full + 2;              // [2] O_x += P_x V of a step has completed
    uint64_t *s_out = pv_done + 2;               // [2] tile x's scores have been copied out of the shared region
    uint32_t *tmem_slot = (uint32_t *)(s_out + 2);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const PrefillTile tile = tiles[unit];
    const int n_tiles = tile.q_head_b >= 0 ? 2 : 1;
    const int kv_len = tile.pos0 + tile.rows;                       // keys the last valid row attends
    const int n_steps = (kv_len + kTileN - 1) / kTileN;
    const int total_pages = (tile.ctx_len + kPageSize - 1) / kPageSize;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < kKvSlots; ++s) {
            mbar_init(&kv_full[s], 1);
            mbar_init(&kv_empty[s], n_tiles);    // one commit per issuing warp
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(&s_full[x], 1);
            mbar_init(&p_full[x], 4);            // one arrival per softmax warp
            mbar_init(&pv_done[x], 1);
            mbar_init(&s_out[x], 4);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(tmem_slot, Cfg::kTmemCols);
        tmem_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem = *tmem_slot;
    // The preamble above reads only the plan; q, the pool and the outputs wait for the kernel
    // before this one in the stream.
    griddep_launch_dependents();
    griddep_wait();

    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
        if (warp == kProducerWarp) {
            // -------------------------------------------------- producer --
            if (lane == 0) {
                prefetch_tensormap(&q_map);
                prefetch_tensormap(&k_map);
                prefetch_tensormap(&v_map);
                mbar_arrive_expect_tx(q_full, (uint32_t)(n_tiles * Cfg::kQBytes));
                tma_load_3d(smem + Cfg::kOffQ, &q_map, q_full, 0, tile.q_row0, tile.q_head * Cfg::kHalves);
                if (n_tiles == 2)
                    tma_load_3d(smem + Cfg::kOffQ + Cfg::kQBytes, &q_map, q_full, 0, tile.q_row0,
                                tile.q_head_b * Cfg::kHalves);
            }
            const int32_t *bt = bt_flat + tile.bt_offset;
            // ring order K_0, K_1, V_0, K_2, V_1, ...: entry n goes to slot n % kKvSlots
            const int n_entries = 2 * n_steps;
            for (int n = 0; n < n_entries; ++n) {
                // entry n: K_j for n = 0 or odd n < 2 n_steps - 1, else V_j
                const bool is_k = n == 0 || ((n & 1) && n < n_entries - 1);
                const int j = is_k ? (n + 1) / 2 : (n == n_entries - 1 ? n_steps - 1 : n / 2 - 1);
                const int s = n % kKvSlots;
                const uint32_t ph = (uint32_t)(n / kKvSlots) & 1u;
                const int np = min(kPagesPerTile, total_pages - j * kPagesPerTile);
                int32_t page = lane < np ? __ldg(bt + j * kPagesPerTile + lane) : 0;
                if (!wait_or_abort(&kv_empty[s], ph ^ 1u, abort_flag, wait_limit_ns)) {
                    record_status(status, AP_ERR_TIMEOUT);
                    *abort_flag = 1;
                    break;
                }
                if (lane == 0) mbar_arrive_expect_tx(&kv_full[s], (uint32_t)(np * Cfg::kPageTileBytes));
                __syncwarp();
                if (lane < np) {
                    if (page < 0 || page >= num_pages) {
                        record_status(status, AP_ERR_BAD_BLOCK_TABLE);
                        page = 0;
                    }
                    const int group = (page * Hkv + tile.kv_head) * 2;
                    tma_load_4d(smem + Cfg::kOffK + s * Cfg::kKvTileBytes + lane * Cfg::kPageTileBytes,
                                is_k ? &k_map : &v_map, &kv_full[s], 0, 0, 0, group);
                }
            }
        } else if (warp == kMmaWarp || (warp == kMmaWarp + 1 && n_tiles == 2)) {
            // ----------------------------------------------- MMA issuers --
            // One issuing warp per tile (warp 9: tile A, warp 10: tile B), so that one tile's wait for
            // its P does not hold up the other tile's instructions.  Each warp runs this block
            // converged; `leader` selects the lane that issues.  The two meet only in barriers: the
            // score region passes from one tile to the other through s_free, and a K/V slot is
            // released when both have committed their last product on it.
            {
                const int x = warp - kMmaWarp;
                const uint32_t leader = elect_one();
                constexpr uint32_t kIdescQK = instr_desc(kTileM, kTileN, false);
                constexpr uint32_t kIdescPV = instr_desc(kTileM, D, true);
                bool ok = wait_or_abort(q_full, 0, abort_flag, wait_limit_ns);
                // Descriptors are built once; per MMA only a constant is added to the address field
                // (addresses are below 256 KB, so the 14-bit field cannot carry out).
                // Q: [half][128 rows][64], 8-row groups 1024 B apart.  K: [16 groups of 8 keys][half][8][64].
                // V (MN-major): 64-column halves 1024 B apart (LBO), 8-key groups 1024 * halves apart (SBO).
                const uint64_t q_desc0 = smem_desc(smem_u32(smem + Cfg::kOffQ + x * Cfg::kQBytes), 16, 1024);
                const uint64_t k_desc0 = smem_desc(smem_u32(smem + Cfg::kOffK), 16, 1024 * Cfg::kHalves);
                const uint64_t v_desc0 = smem_desc(smem_u32(smem + Cfg::kOffK), 1024, 1024 * Cfg::kHalves);
                const uint32_t q_lo = (uint32_t)q_desc0, q_hi = (uint32_t)(q_desc0 >> 32);
                const uint32_t k_lo = (uint32_t)k_desc0, k_hi = (uint32_t)(k_desc0 >> 32);
                const uint32_t v_lo = (uint32_t)v_desc0, v_hi = (uint32_t)(v_desc0 >> 32);
                const uint32_t t_s = tmem + Cfg::kColS, t_p = tmem + Cfg::kColP + x * 64, t_o = tmem + Cfg::kColO + x * 128;
                // S = Q_x K^T with K in ring slot `slot`, into the shared score region
                auto issue_qk = [&](int slot) {
                    const uint32_t b0 = k_lo + (uint32_t)((slot * Cfg::kKvTileBytes) >> 4);
                    // 16 elements of d per MMA: 32 bytes further inside the 64-element half, next half every four
#pragma unroll
                    for (int kh = 0; kh < D / 64; ++kh)
                        umma_ss_x4(leader, t_s, q_lo + (uint32_t)((kh * (kTileM * 128)) >> 4), q_hi,
                                   b0 + (uint32_t)((kh * 1024) >> 4), k_hi, kIdescQK, kh > 0 ? 1u : 0u, 32u >> 4, 32u >> 4);
                    umma_commit(leader, &s_full[x]);
                    umma_commit(leader, &kv_empty[slot]);
                };
                // O_x += P_x V with V in ring slot `slot`.  P_x: bf16 pairs in 64 columns of its own
                // (A operand from TMEM, 8 columns per 16 keys); 16 keys of V = 2 groups of 8.
                auto issue_pv = [&](int slot, bool first_step) {
                    const uint32_t b0 = v_lo + (uint32_t)((slot * Cfg::kKvTileBytes) >> 4);
                    constexpr uint32_t kVStep = (uint32_t)((2 * 1024 * Cfg::kHalves) >> 4);   // 16 keys of V
#pragma unroll
                    for (int kq = 0; kq < kTileN / 64; ++kq)
                        umma_ts_x4(leader, t_o, t_p + kq * 32, b0 + kq * 4 * kVStep, v_hi, kIdescPV,
                                   (first_step && kq == 0) ? 0u : 1u, 8u, kVStep);
                    umma_commit(leader, &pv_done[x]);
                    umma_commit(leader, &kv_empty[slot]);
                };
                // The score region is used by one tile after the other: use number u = step * tiles + x
                // may be issued once the softmax group of use u - 1 has copied its scores out.
                // S_x(step) may be issued once the scores written before it have been copied out: with two
                // tiles, S_B(step - 1) before S_A(step) and S_A(step) before S_B(step); with one, S_A(step - 1).
                // Each of the two barriers has one waiter that follows it phase by phase (a parity wait can
                // only tell the current phase from the one before).
                auto wait_s_free = [&](int step) {
                    if (n_tiles == 2 && x == 1) return wait_or_abort(&s_out[0], (uint32_t)step & 1u, abort_flag, wait_limit_ns);
                    if (step == 0) return true;
                    return wait_or_abort(&s_out[n_tiles - 1], (uint32_t)(step - 1) & 1u, abort_flag, wait_limit_ns);
                };
                if (ok) ok = wait_or_abort(&kv_full[0], 0, abort_flag, wait_limit_ns);
                if (ok) ok = wait_s_free(0);
                if (ok) {
                    tcgen05_fence_after();
                    issue_qk(0);                                        // K_0 is ring entry 0, slot 0
                }
                for (int j = 0; ok && j < n_steps; ++j) {
                    const int nv = kv_seq_v(j, n_steps), nk = kv_seq_k(j + 1);
                    if (j + 1 < n_steps) {
                        // the next scores of the tile go ahead of this step's P V
                        if (!wait_or_abort(&kv_full[nk % kKvSlots], (uint32_t)(nk / kKvSlots) & 1u, abort_flag,
                                           wait_limit_ns) || !wait_s_free(j + 1)) { ok = false; break; }
                        tcgen05_fence_after();
                        issue_qk(nk % kKvSlots);
                    }
                    if (!wait_or_abort(&kv_full[nv % kKvSlots], (uint32_t)(nv / kKvSlots) & 1u, abort_flag, wait_limit_ns) ||
                        !wait_or_abort(&p_full[x], (uint32_t)j & 1u, abort_flag, wait_limit_ns)) { ok = false; break; }
                    // In the last step tile A's softmax group clears the V rows past the context before it
                    // hands P_A over; tile B's product reads the same V tile and has to see that too.
                    if (x == 1 && j == n_steps - 1 && tile.ctx_len < n_steps * kTileN &&
                        !wait_or_abort(&p_full[0], (uint32_t)j & 1u, abort_flag, wait_limit_ns)) { ok = false; break; }
                    tcgen05_fence_after();
                    issue_pv(nv % kKvSlots, j == 0);
                }
                if (!ok && leader) {
                    record_status(status, AP_ERR_TIMEOUT);
                    *abort_flag = 1;
                }
            }
            __syncwarp();
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // ------------------------------------------------------- softmax --
        const int x = warp >> 2;                                     // tile A or B
        if (x < n_tiles) {
            const int r = threadIdx.x & 127;                         // query row = TMEM lane
            const int q_head = x == 0 ? tile.q_head : tile.q_head_b;
            const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
            const uint32_t col_s = Cfg::kColS, col_p = Cfg::kColP + x * 64, col_o = Cfg::kColO + x * 128;
            const int my_pos = min(tile.pos0 + r, tile.ctx_len - 1); // last key this row attends
            float m_used = -INFINITY, l = 0.f;
            bool ok = true;
            for (int j = 0; j < n_steps; ++j) {
                // S_x(j) complete: copy this row's 128 scores out and give the region back at once
                if (!wait_or_abort(&s_full[x], (uint32_t)j & 1u, abort_flag, wait_limit_ns)) { ok = false; break; }
                tcgen05_fence_after();
                uint32_t sreg[4][32];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x32(lane_addr + col_s + c * 32, sreg[c]);
                tmem_ld_wait();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_out[x]);
                const int tok0 = j * kTileN;
                float mx = -INFINITY;
                if (tok0 + kTileN - 1 > tile.pos0) {
                    // diagonal or last step: keys past the row's position (or past the context) are masked
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            float v = __uint_as_float(sreg[c][i]);
                            if (tok0 + c * 32 + i > my_pos) v = -INFINITY;
                            sreg[c][i] = __float_as_uint(v);
                            mx = fmaxf(mx, v);
                        }
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int i = 0; i < 32; i += 2)
                            mx = max3(mx, __uint_as_float(sreg[c][i]), __uint_as_float(sreg[c][i + 1]));
                }
                // Keep the old reference max unless some row of the warp moved by more than the
                // threshold: P stays bounded by 2^threshold and O needs no rescale most steps.
                // P_x and O_x belong to the tensor pipe until O_x += P_x V of the step before is done
                if (j > 0) {
                    if (!wait_or_abort(&pv_done[x], (uint32_t)(j - 1) & 1u, abort_flag, wait_limit_ns)) { ok = false; break; }
                    tcgen05_fence_after();
                }
                const float m_new = fmaxf(m_used, mx);
                const bool moved = (m_new - m_used) * scale_log2 > kRescaleThreshold;   // true while m_used = -inf
                const bool rescale = __any_sync(0xffffffffu, moved);
                float alpha = 1.f;
                if (rescale) {
                    alpha = exp2_approx((m_used - m_new) * scale_log2);   // 0 on the first step
                    m_used = m_new;
                    if (j > 0) rescale_o<D>(lane_addr + col_o, alpha);
                }
                const float ms = m_used * scale_log2;
                const float2 sc2 = make_float2(scale_log2, scale_log2), nms2 = make_float2(-ms, -ms);
                float2 sum2 = make_float2(0.f, 0.f), sum2b = make_float2(0.f, 0.f);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t preg[32];                                  // 64 keys as bf16 pairs
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        // two keys at a time on the packed fp32x2 pipe: x = s * c - m * c, then 2^x
                        float2 xy = __ffma2_rn(make_float2(__uint_as_float(sreg[2 * c + (i >> 4)][(2 * i) & 31]),
                                                           __uint_as_float(sreg[2 * c + (i >> 4)][(2 * i + 1) & 31])),
                                               sc2, nms2);
                        // one pair in eight goes to the FMA pipe instead of the special-function unit
                        if ((i & 7) == 7) {
                            xy = exp2_poly2(xy);
                        } else {
                            xy.x = exp2_approx(xy.x);
                            xy.y = exp2_approx(xy.y);
                        }
                        sum2 = __fadd2_rn(sum2, xy);
                        preg[i] = pack_bf16x2(xy.x, xy.y);
                    }
                    tmem_st_32x32b_x32(lane_addr + col_p + c * 32, preg);
                }
                const float sum = (sum2.x + sum2b.x) + (sum2.y + sum2b.y);
                l = l * alpha + sum;
                tmem_st_wait();
                if (x == 0 && j == n_steps - 1 && tile.ctx_len < n_steps * kTileN) {
                    // keys past the context hold no token: clear their V rows so 0 * garbage cannot
                    // poison O (tile A's group does it; tile B's issuer waits for tile A's hand-over too)
                    const int nv = kv_seq_v(j, n_steps), s = nv % kKvSlots;
                    if (!wait_or_abort(&kv_full[s], (uint32_t)(nv / kKvSlots) & 1u, abort_flag, wait_limit_ns)) { ok = false; break; }
                    uint8_t *v_tile = smem + Cfg::kOffK + s * Cfg::kKvTileBytes;
                    const int first = tile.ctx_len - tok0;           // first key of the step without a token
                    for (int idx = r; idx < (kTileN - first) * (D / 8); idx += 128) {
                        const int key = first + idx / (D / 8), ch = idx % (D / 8);
                        *(uint4 *)(v_tile + (key >> 3) * (1024 * Cfg::kHalves) + (ch >> 3) * 1024 + (key & 7) * 128 +
                                   ((ch & 7) << 4)) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_full[x]);
            }
            if (ok && wait_or_abort(&pv_done[x], (uint32_t)(n_steps - 1) & 1u, abort_flag, wait_limit_ns)) {
                tcgen05_fence_after();
                const float inv = 1.f / l;
                const bool valid = r < tile.rows;
                __nv_bfloat16 *orow = out + ((size_t)(tile.q_row0 + r) * Hq + q_head) * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t oreg[32];
                    tmem_ld_32x32b_x32(lane_addr + col_o + c * 32, oreg);
                    tmem_ld_wait();
                    if (valid) {
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            uint4 v;
                            v.x = pack_bf16x2(__uint_as_float(oreg[i]) * inv, __uint_as_float(oreg[i + 1]) * inv);
                            v.y = pack_bf16x2(__uint_as_float(oreg[i + 2]) * inv, __uint_as_float(oreg[i + 3]) * inv);
                            v.z = pack_bf16x2(__uint_as_float(oreg[i + 4]) * inv, __uint_as_float(oreg[i + 5]) * inv);
                            v.w = pack_bf16x2(__uint_as_float(oreg[i + 6]) * inv, __uint_as_float(oreg[i + 7]) * inv);
                            *(uint4 *)(orow + c * 32 + i) = v;
                        }
                    }
                }
                if (valid && lse_out)
                    lse_out[(size_t)(tile.q_row0 + r) * Hq + q_head] =
                        (m_used * scale_log2 + log2f(l)) * 0.6931471805599453f;
            } else {
                record_status(status, AP_ERR_TIMEOUT);
                *abort_flag = 1;
            }
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, Cfg::kTmemCols);
}


}  // namespace prefill
}  // namespace ap
