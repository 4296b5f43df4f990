// Prefill-chunk attention: causal tiled attention on tcgen05 tensor cores with
// accumulators in tensor memory (TMEM).
//
// One CTA handles one work unit: 128 consecutive query rows of one sequence for
// one q head, over keys 0 .. (position of its last row).  Keys and values come
// through the block table, one TMA per (page, kv head) tile, straight into the
// 128-byte-swizzled operand layout tcgen05.mma reads.
//
//   warps 0-3  softmax: thread r owns query row r (= TMEM lane r): reads S from
//              TMEM, masks, keeps the running max / sum in fp32, writes P (bf16)
//              to shared memory as the A operand of the second product,
//              rescales O in TMEM when the running max has moved enough, and
//              writes the normalised output at the end
//   warp 4     producer: Q tile once, then K and V tiles into a 2-stage ring
//   warp 5     MMA issuer: S = Q K^T (8 x M128 N128 K16), O += P V, completion
//              signalled to the other warps through tcgen05.commit -> mbarrier
//
// Every wait is bounded; a wait that runs out records AP_ERR_TIMEOUT, raises the
// CTA's abort flag, and all roles fall through to the common exit where TMEM is
// released.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace ap {

namespace {

using namespace ptx;

constexpr int kTileM = 128;                 // query rows per CTA
constexpr int kTileN = 128;                 // keys per step (8 pages)
constexpr int kPagesPerTile = kTileN / kPageSize;
constexpr int kKvStages = 2;
constexpr int kPrefillThreads = 192;
constexpr float kRescaleThreshold = 8.0f;   // in log2 units: P stays below 2^8

template <int D>
struct PrefillCfg {
    static constexpr int kHalves = D / 64;
    static constexpr int kPageTileBytes = kPageSize * D * 2;
    static constexpr int kQBytes = kTileM * D * 2;
    static constexpr int kKvTileBytes = kTileN * D * 2;
    static constexpr int kPBytes = kTileM * kTileN * 2;
    static constexpr int kOffQ = 0;
    static constexpr int kOffP = kOffQ + kQBytes;
    static constexpr int kOffK = kOffP + kPBytes;
    static constexpr int kOffV = kOffK + kKvStages * kKvTileBytes;
    static constexpr int kOffBar = kOffV + kKvStages * kKvTileBytes;
    static constexpr int kSmemBytes = 1024 + kOffBar + 256;
    static constexpr uint32_t kTmemCols = 256;   // S: 128 columns, O: D columns
    static constexpr uint32_t kColS = 0;
    static constexpr uint32_t kColO = 128;
};

__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = globaltimer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (globaltimer_ns() - t0 > 2000000000ull) return false;
    }
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

template <int D>
__global__ void __launch_bounds__(kPrefillThreads, 1)
prefill_tcgen05_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                       const __grid_constant__ CUtensorMap v_map, const PrefillTile *__restrict__ tiles,
                       const int32_t *__restrict__ bt_flat, __nv_bfloat16 *__restrict__ out,
                       float *__restrict__ lse_out, int Hq, int Hkv, int num_pages, float scale_log2, int *status) {
    using Cfg = PrefillCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + Cfg::kOffBar);
    uint64_t *q_full = bars + 0;
    uint64_t *k_full = bars + 1;                 // [kKvStages]
    uint64_t *v_full = bars + 1 + kKvStages;     // [kKvStages]
    uint64_t *kv_empty = bars + 1 + 2 * kKvStages;
    uint64_t *s_full = bars + 1 + 3 * kKvStages;
    uint64_t *p_full = s_full + 1;
    uint64_t *pv_done = s_full + 2;
    uint32_t *tmem_slot = (uint32_t *)(s_full + 3);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const PrefillTile tile = tiles[blockIdx.x];
    const int kv_len = tile.pos0 + tile.rows;                       // keys the last valid row attends
    const int n_steps = (kv_len + kTileN - 1) / kTileN;
    const int total_pages = (tile.ctx_len + kPageSize - 1) / kPageSize;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < kKvStages; ++s) {
            mbar_init(&k_full[s], 1);
            mbar_init(&v_full[s], 1);
            mbar_init(&kv_empty[s], 1);
        }
        mbar_init(s_full, 1);
        mbar_init(p_full, 128);
        mbar_init(pv_done, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 5) {
        tmem_alloc(tmem_slot, Cfg::kTmemCols);
        tmem_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        // ------------------------------------------------------ producer --
        if (lane == 0) {
            prefetch_tensormap(&q_map);
            prefetch_tensormap(&k_map);
            prefetch_tensormap(&v_map);
            mbar_arrive_expect_tx(q_full, Cfg::kQBytes);
            tma_load_3d(smem + Cfg::kOffQ, &q_map, q_full, 0, tile.q_row0, tile.q_head * Cfg::kHalves);
        }
        const int32_t *bt = bt_flat + tile.bt_offset;
        for (int j = 0; j < n_steps; ++j) {
            const int s = j % kKvStages;
            const uint32_t ph = (uint32_t)(j / kKvStages) & 1u;
            const int np = min(kPagesPerTile, total_pages - j * kPagesPerTile);
            int32_t page = lane < np ? __ldg(bt + j * kPagesPerTile + lane) : 0;
            if (!wait_or_abort(&kv_empty[s], ph ^ 1u, abort_flag)) {
                atomicCAS(status, 0, AP_ERR_TIMEOUT);
                *abort_flag = 1;
                break;
            }
            if (lane == 0) {
                mbar_arrive_expect_tx(&k_full[s], (uint32_t)(np * Cfg::kPageTileBytes));
                mbar_arrive_expect_tx(&v_full[s], (uint32_t)(np * Cfg::kPageTileBytes));
            }
            __syncwarp();
            if (lane < np) {
                if (page < 0 || page >= num_pages) {
                    atomicCAS(status, 0, AP_ERR_BAD_BLOCK_TABLE);
                    page = 0;
                }
                const int group = (page * Hkv + tile.kv_head) * 2;
                tma_load_4d(smem + Cfg::kOffK + s * Cfg::kKvTileBytes + lane * Cfg::kPageTileBytes, &k_map, &k_full[s],
                            0, 0, 0, group);
                tma_load_4d(smem + Cfg::kOffV + s * Cfg::kKvTileBytes + lane * Cfg::kPageTileBytes, &v_map, &v_full[s],
                            0, 0, 0, group);
            }
        }
    } else if (warp == 5) {
        // ---------------------------------------------------- MMA issuer --
        if (lane == 0) {
            constexpr uint32_t kIdescQK = instr_desc(kTileM, kTileN, false);
            constexpr uint32_t kIdescPV = instr_desc(kTileM, D, true);
            const uint32_t q_addr = smem_u32(smem + Cfg::kOffQ);
            const uint32_t p_addr = smem_u32(smem + Cfg::kOffP);
            const uint32_t tmem_s = tmem + Cfg::kColS, tmem_o = tmem + Cfg::kColO;
            bool ok = wait_or_abort(q_full, 0, abort_flag);
            auto issue_qk = [&](int j) {
                const int s = j % kKvStages;
                if (!wait_or_abort(&k_full[s], (uint32_t)(j / kKvStages) & 1u, abort_flag)) return false;
                tcgen05_fence_after();
                const uint32_t k_addr = smem_u32(smem + Cfg::kOffK + s * Cfg::kKvTileBytes);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    // Q: [half][128 rows][64], 8-row groups 1024 B apart.  K: [16 groups][half][8][64].
                    const uint64_t a = smem_desc(q_addr + (ks >> 2) * (kTileM * 128) + (ks & 3) * 32, 16, 1024);
                    const uint64_t b = smem_desc(k_addr + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 1024 * Cfg::kHalves);
                    umma_ss(tmem_s, a, b, kIdescQK, ks > 0 ? 1u : 0u);
                }
                umma_commit(s_full);
                return true;
            };
            if (ok) ok = issue_qk(0);
            for (int j = 0; ok && j < n_steps; ++j) {
                const int s = j % kKvStages;
                if (!wait_or_abort(p_full, (uint32_t)j & 1u, abort_flag) ||
                    !wait_or_abort(&v_full[s], (uint32_t)(j / kKvStages) & 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                tcgen05_fence_after();
                const uint32_t v_addr = smem_u32(smem + Cfg::kOffV + s * Cfg::kKvTileBytes);
#pragma unroll
                for (int ks = 0; ks < kTileN / 16; ++ks) {
                    // P: [half of 64 keys][128 rows][64].  V (MN-major): 16 keys = 2 groups of 8,
                    // 64-column halves 1024 B apart (LBO), 8-key groups 1024*halves apart (SBO).
                    const uint64_t a = smem_desc(p_addr + (ks >> 2) * (kTileM * 128) + (ks & 3) * 32, 16, 1024);
                    const uint64_t b = smem_desc(v_addr + ks * 2 * 1024 * Cfg::kHalves, 1024, 1024 * Cfg::kHalves);
                    umma_ss(tmem_o, a, b, kIdescPV, (j > 0 || ks > 0) ? 1u : 0u);
                }
                umma_commit(&kv_empty[s]);
                umma_commit(pv_done);
                if (j + 1 < n_steps) ok = issue_qk(j + 1);
            }
            if (!ok) {
                atomicCAS(status, 0, AP_ERR_TIMEOUT);
                *abort_flag = 1;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------- softmax --
        const int r = threadIdx.x;                                   // query row = TMEM lane
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        const int my_pos = min(tile.pos0 + r, tile.ctx_len - 1);     // last key this row attends
        float m_used = -INFINITY, l = 0.f;
        uint8_t *p_row = smem + Cfg::kOffP + (r >> 3) * 1024 + (r & 7) * 128;
        bool ok = true;
        for (int j = 0; j < n_steps; ++j) {
            if (!wait_or_abort(s_full, (uint32_t)j & 1u, abort_flag)) { ok = false; break; }
            tcgen05_fence_after();
            uint32_t sreg[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x32(lane_addr + Cfg::kColS + c * 32, sreg[c]);
            tmem_ld_wait();
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
                    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(sreg[c][i]));
            }
            // Keep the old reference max unless some row of the warp moved by more than the
            // threshold: P stays bounded by 2^threshold and O needs no rescale most steps.
            const float m_new = fmaxf(m_used, mx);
            const bool moved = (m_new - m_used) * scale_log2 > kRescaleThreshold;   // true when m_used = -inf
            const bool rescale = __any_sync(0xffffffffu, moved);
            float alpha = 1.f;
            if (rescale) {
                alpha = exp2_approx((m_used - m_new) * scale_log2);   // 0 on the first step
                m_used = m_new;
            }
            if (j > 0) {
                // the previous P V product must be done before P is overwritten or O is touched
                if (!wait_or_abort(pv_done, (uint32_t)(j - 1) & 1u, abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                if (rescale) {
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t oreg[32];
                        tmem_ld_32x32b_x32(lane_addr + Cfg::kColO + c * 32, oreg);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) oreg[i] = __float_as_uint(__uint_as_float(oreg[i]) * alpha);
                        tmem_st_32x32b_x32(lane_addr + Cfg::kColO + c * 32, oreg);
                    }
                    tmem_st_wait();
                }
            }
            const float ms = m_used * scale_log2;
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    float p[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        p[e] = exp2_approx(__uint_as_float(sreg[c][i + e]) * scale_log2 - ms);
                        sum += p[e];
                    }
                    const int chunk = c * 4 + (i >> 3);              // 16-byte chunk = 8 keys
                    uint4 v = make_uint4(pack_bf16x2(p[0], p[1]), pack_bf16x2(p[2], p[3]), pack_bf16x2(p[4], p[5]),
                                         pack_bf16x2(p[6], p[7]));
                    *(uint4 *)(p_row + (chunk >> 3) * (kTileM * 128) + (((chunk & 7) ^ (r & 7)) << 4)) = v;
                }
            }
            l = l * alpha + sum;
            if (j == n_steps - 1 && tile.ctx_len < n_steps * kTileN) {
                // keys past the context hold no token: clear their V rows so 0 * garbage cannot poison O
                const int s = j % kKvStages;
                if (!wait_or_abort(&v_full[s], (uint32_t)(j / kKvStages) & 1u, abort_flag)) { ok = false; break; }
                uint8_t *v_tile = smem + Cfg::kOffV + s * Cfg::kKvTileBytes;
                const int first = tile.ctx_len - tok0;               // first key of the step without a token
                for (int idx = r; idx < (kTileN - first) * (D / 8); idx += 128) {
                    const int key = first + idx / (D / 8), ch = idx % (D / 8);
                    *(uint4 *)(v_tile + (key >> 3) * (1024 * Cfg::kHalves) + (ch >> 3) * 1024 + (key & 7) * 128 +
                               ((ch & 7) << 4)) = make_uint4(0, 0, 0, 0);
                }
            }
            fence_proxy_async_smem();
            tcgen05_fence_before();
            mbar_arrive(p_full);
        }
        if (ok && wait_or_abort(pv_done, (uint32_t)(n_steps - 1) & 1u, abort_flag)) {
            tcgen05_fence_after();
            const float inv = 1.f / l;
            const bool valid = r < tile.rows;
            __nv_bfloat16 *orow = out + ((size_t)(tile.q_row0 + r) * Hq + tile.q_head) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t oreg[32];
                tmem_ld_32x32b_x32(lane_addr + Cfg::kColO + c * 32, oreg);
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
                lse_out[(size_t)(tile.q_row0 + r) * Hq + tile.q_head] =
                    (m_used * scale_log2 + log2f(l)) * 0.6931471805599453f;
        } else {
            atomicCAS(status, 0, AP_ERR_TIMEOUT);
            *abort_flag = 1;
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tmem, Cfg::kTmemCols);
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
    prefill_tcgen05_kernel<D><<<(unsigned)plan->info.prefill_tiles, kPrefillThreads, Cfg::kSmemBytes, stream>>>(
        q_map, pool->k_map, pool->v_map, plan->d_tiles, plan->d_bt_flat, (__nv_bfloat16 *)out, lse,
        plan->num_q_heads, pool->desc.num_kv_heads, pool->desc.num_pages, scale_log2, pool->d_status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefill(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                           cudaStream_t stream) {
    if (pool->desc.head_dim == 128) return launch_prefill_t<128>(pool, plan, q, out, lse, stream);
    return launch_prefill_t<64>(pool, plan, q, out, lse, stream);
}

}  // namespace ap
