// Host side of the serving-iteration library: pool, page allocator, planner,
// dispatch.  Every entry point validates on the host and returns a status;
// nothing here (or in the kernels) aborts or traps.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "internal.h"

using namespace ap;

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { prev = -1; (void)cudaGetLastError(); }
        ok = cudaSetDevice(dev) == cudaSuccess;
        if (!ok) (void)cudaGetLastError();
    }
    ~DeviceGuard() {
        if (prev >= 0 && ok) (void)cudaSetDevice(prev);
    }
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool desc_valid(const ap_pool_desc *d) {
    return d && d->num_pages > 0 && d->num_kv_heads > 0 && d->head_dim > 0 && d->page_size > 0;
}

// splitmix64: public-domain mixing function used as a counter-based stream.
inline uint64_t splitmix64(uint64_t &state) {
    uint64_t z = (state += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

void release_plan_buffer(PlanBuffer &b) {
    if (b.uploaded) (void)cudaEventDestroy(b.uploaded);
    if (b.host) (void)cudaFreeHost(b.host);
    if (b.dev) (void)cudaFree(b.dev);
    b = PlanBuffer{};
}

int acquire_plan_buffer(ap_kv_pool *pool, size_t n_ints, PlanBuffer *out) {
    for (size_t i = 0; i < pool->plan_buffers.size(); ++i) {
        if (pool->plan_buffers[i].capacity >= n_ints) {
            *out = pool->plan_buffers[i];
            pool->plan_buffers.erase(pool->plan_buffers.begin() + (long)i);
            // the previous upload from this staging area must have been consumed
            if (cudaEventSynchronize(out->uploaded) != cudaSuccess) {
                (void)cudaGetLastError();
                return AP_ERR_CUDA;
            }
            return AP_OK;
        }
    }
    PlanBuffer b;
    b.capacity = std::max<size_t>(n_ints + n_ints / 2, 4096);
    if (cudaMallocHost((void **)&b.host, b.capacity * sizeof(int32_t)) != cudaSuccess ||
        cudaMalloc((void **)&b.dev, b.capacity * sizeof(int32_t)) != cudaSuccess ||
        cudaEventCreateWithFlags(&b.uploaded, cudaEventDisableTiming) != cudaSuccess) {
        (void)cudaGetLastError();
        release_plan_buffer(b);
        return AP_ERR_CUDA;
    }
    *out = b;
    return AP_OK;
}

cudaEvent_t take_event(ap_kv_pool *pool) {
    if (!pool->spare_events.empty()) {
        cudaEvent_t e = pool->spare_events.back();
        pool->spare_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    return e;
}

// Side-by-side execution of a mixed iteration.  Decode is bound by HBM when it has the whole GPU
// (~41 GB/s per SM at 148 SMs) but one SM's decode pipeline sustains more (its ring keeps ~100 KB in
// flight over a ~1.2 us memory latency; with items that span a block of kv heads the TMA requests are
// large enough not to be the limit), while prefill is bound by the SMs it has.  So decode is confined
// to k SMs, where it is SM-bound, and prefill runs on the others at the same time; the iteration then
// takes about (W_d + W_p) / #SM, with W the SM-time of each part.  k is the smallest count that lets
// decode finish within 95 % of that time; beyond ~0.7 #SM decode would be HBM-bound again and nothing
// is gained, so the plan stays sequential.  The constants were measured on B200 (8B and 70B attention
// shapes, head_dim 128; both kernels running, i.e. at the clocks the power limit leaves: ~1.5 GHz).
// Returns 0 for "sequential".
constexpr double kDecodeSmGBs = 68.0;        // GB/s of KV one SM's decode pipeline sustains next to prefill
constexpr double kDecodeGpuGBs = 6000.0;     // GB/s decode reaches with all SMs
constexpr double kPrefillStepUs = 1.9;       // one 128-key step of a two-tile unit at d = 128
constexpr double kPrefillStepSingleUs = 1.35; // the same for a one-tile unit
constexpr double kPrefillUnitUs = 5.3;       // prologue + epilogue + relaunch gap of a unit
constexpr double kPrefillTailUs = 12.0;      // spread of the SMs' finishing times (about half a short unit) + ramp-up
constexpr double kDecodeFixedUs = 8.0;       // first-data latency and finishing spread of the decode kernel
constexpr double kAppendGBs = 4000.0;        // scatter of 256-byte rows
constexpr double kAppendFixedUs = 3.0;

// GB/s of KV one SM's decode pipeline sustains, by the size of its TMA requests (the tiles of one page
// that an item takes in one request): the TMA unit handles ~14 M requests per second.
inline double decode_sm_gbs(int request_bytes) {
    return request_bytes >= 16384 ? kDecodeSmGBs : request_bytes >= 8192 ? 50.0 : request_bytes >= 4096 ? 40.0 : 25.0;
}

// Time of a mixed iteration with decode on k SMs: decode streams at k times an SM's rate (or what HBM
// gives), and all SM-time of both parts has to fit on the GPU.
inline double side_by_side_us(double decode_bytes, double w_p, int k, double sm_rate, int sms) {
    const double t_dec = decode_bytes / std::min(k * sm_rate, kDecodeGpuGBs * 1e3);
    return std::max(t_dec, (t_dec * k + w_p) / sms);
}

int side_by_side_decode_ctas(const ap_kv_pool *pool, const ap_batch_desc *b, int d, int Hkv, int G, int max_ctas) {
    const int mode = pool->side_by_side_mode;
    if (mode == 0) return 0;
    double decode_bytes = 0.0, w_p = 0.0;
    int64_t decode_rows = 0, prefill_seqs = 0;
    const double d_scale = (double)d / 128.0;
    for (int s = 0; s < b->batch; ++s) {
        const int32_t ql = b->q_lens[s], cl = b->ctx_lens[s];
        if (ql == 1) {
            ++decode_rows;
            decode_bytes += (double)((cl + kPageSize - 1) / kPageSize) * kPageSize * Hkv * d * 4.0;
        } else if (ql > 1) {
            ++prefill_seqs;
            for (int32_t t0 = 0; t0 < ql; t0 += 128) {
                const int steps = (cl - ql + t0 + std::min(128, ql - t0) + 127) / 128;
                const int pairs = G / 2, singles = G % 2;
                w_p += (double)Hkv * (pairs * (steps * kPrefillStepUs * d_scale + kPrefillUnitUs) +
                                      singles * (steps * kPrefillStepSingleUs * d_scale + kPrefillUnitUs));
            }
        }
    }
    if (decode_rows == 0 || prefill_seqs == 0) return 0;
    if (mode >= 2) return std::min(mode, max_ctas);
    const int sms = pool->sm_count;
    const double sm_rate = decode_sm_gbs(pool->head_block * kPageSize * d * 2) * 1e3;      // bytes / us
    const double w_d = decode_bytes / sm_rate;                                             // SM-microseconds
    // k that lets decode end with the iteration, at most 0.7 #SM (more would leave prefill too little)
    int k = (int)std::ceil(w_d / (0.95 * (w_d + w_p) / sms));
    k = std::max(8, std::min(k, (7 * sms) / 10));
    if (k >= max_ctas) return 0;
    const double t_serial = decode_bytes / (kDecodeGpuGBs * 1e3) + w_p / sms;
    const double t_side = side_by_side_us(decode_bytes, w_p, k, sm_rate, sms);
    if (t_serial - t_side < 10.0 || t_serial - t_side < 0.05 * t_serial) return 0;
    return k;
}

// Brackets one kernel launch with events when profiling is on.
struct TimedScope {
    ap_kv_pool *pool;
    cudaStream_t stream;
    TimedLaunch rec{};
    bool on = false;
    TimedScope(ap_kv_pool *p, int kernel, cudaStream_t st) : pool(p), stream(st) {
        if (!p->profiling) return;
        rec.kernel = kernel;
        rec.start = take_event(p);
        rec.stop = take_event(p);
        on = rec.start && rec.stop && cudaEventRecord(rec.start, st) == cudaSuccess;
    }
    ~TimedScope() {
        if (!on) return;
        if (cudaEventRecord(rec.stop, stream) == cudaSuccess) pool->timed.push_back(rec);
    }
};

}  // namespace

namespace ap {

// The attention kernels of a plan, in the plan's dispatch mode.  Shared by every entry point that
// runs attention; allocates nothing (the second stream and the events belong to the pool).
cudaError_t launch_attention_kernels(ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                                     float *o_part, float *lse_part, cudaStream_t st) {
    cudaError_t e = cudaSuccess;
    if (plan->single_launch) {
        // One grid: the decode CTAs have the lowest block indices, so they are resident first and the
        // prefill units fill the remaining SMs and, as decode CTAs retire, those too.
        TimedScope timed(pool, AP_KERNEL_MIXED, st);
        e = launch_mixed_iteration(pool, plan, q, out, lse, o_part, lse_part, st);
    } else if (plan->side_by_side) {
        // Decode goes first, on the caller's stream, so that its few CTAs are resident when the
        // prefill kernel's units (second stream, lower priority) fill the remaining SMs; as decode
        // CTAs retire, prefill units take their SMs too.  The caller's stream continues after both.
        e = cudaEventRecord(pool->fork_event, st);
        if (e == cudaSuccess) {
            TimedScope timed(pool, AP_KERNEL_DECODE, st);
            e = launch_decode_splitk(pool, plan, q, out, lse, o_part, lse_part, st);
        }
        if (e == cudaSuccess) e = cudaStreamWaitEvent(pool->side_stream, pool->fork_event, 0);
        if (e == cudaSuccess) {
            TimedScope timed(pool, AP_KERNEL_PREFILL, pool->side_stream);
            e = launch_prefill(pool, plan, q, out, lse, pool->side_stream);
        }
        if (e == cudaSuccess) e = cudaEventRecord(pool->join_event, pool->side_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, pool->join_event, 0);
    } else {
        if (plan->info.decode_items > 0) {
            TimedScope timed(pool, AP_KERNEL_DECODE, st);
            e = launch_decode_splitk(pool, plan, q, out, lse, o_part, lse_part, st);
        }
        if (e == cudaSuccess && plan->info.prefill_tiles > 0) {
            TimedScope timed(pool, AP_KERNEL_PREFILL, st);
            e = launch_prefill(pool, plan, q, out, lse, st);
        }
    }
    return e;
}

}  // namespace ap

extern "C" {

const char *ap_status_string(int status) {
    switch (status) {
        case AP_OK: return "ok";
        case AP_ERR_INVALID_ARG: return "invalid argument";
        case AP_ERR_OUT_OF_PAGES: return "out of KV pages";
        case AP_ERR_BAD_BLOCK_TABLE: return "bad block table";
        case AP_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case AP_ERR_CUDA: return "CUDA error";
        case AP_ERR_TIMEOUT: return "device wait timed out";
        case AP_ERR_UNSUPPORTED: return "unsupported configuration";
        default: return "unknown status";
    }
}

size_t ap_kv_pool_bytes(const ap_pool_desc *d) {
    if (!desc_valid(d)) return 0;
    return (size_t)d->num_pages * (size_t)d->num_kv_heads * (size_t)d->page_size *
           (size_t)d->head_dim * 2u;
}

int ap_kv_pool_create(ap_kv_pool **out, const ap_pool_desc *desc) {
    if (!out) return AP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!desc_valid(desc)) return AP_ERR_INVALID_ARG;
    if (desc->page_size != kPageSize) return AP_ERR_UNSUPPORTED;
    if (desc->head_dim != 64 && desc->head_dim != 128) return AP_ERR_UNSUPPORTED;
    if ((desc->k_base == nullptr) != (desc->v_base == nullptr)) return AP_ERR_INVALID_ARG;
    // a tensor map's global address must be 16-byte aligned (the 1024-byte rule of the 128-byte
    // swizzle concerns the shared-memory side, which the kernels align themselves)
    if (((uintptr_t)desc->k_base | (uintptr_t)desc->v_base) & 15u) return AP_ERR_INVALID_ARG;
    // the tensor maps address 8-row groups with a 32-bit extent
    if ((int64_t)desc->num_pages * desc->num_kv_heads * 2 >= (int64_t)1 << 31) return AP_ERR_UNSUPPORTED;

    if (desc->device < 0) {
        // host-only pool: allocator and planner work, nothing can be launched
        if (desc->k_base) return AP_ERR_INVALID_ARG;
        ap_kv_pool *hp = new (std::nothrow) ap_kv_pool();
        if (!hp) return AP_ERR_CUDA;
        hp->desc = *desc;
        hp->head_block = decode_head_block(desc->num_kv_heads);
        hp->sm_count = 148;
        hp->free_list.resize((size_t)desc->num_pages);
        for (int32_t i = 0; i < desc->num_pages; ++i) hp->free_list[(size_t)i] = desc->num_pages - 1 - i;
        hp->allocated.assign((size_t)desc->num_pages, 0);
        *out = hp;
        return AP_OK;
    }

    DeviceGuard guard(desc->device);
    if (!guard.ok) return AP_ERR_CUDA;

    ap_kv_pool *p = new (std::nothrow) ap_kv_pool();
    if (!p) return AP_ERR_CUDA;
    p->desc = *desc;
    p->head_block = decode_head_block(desc->num_kv_heads);
    int rc = AP_OK;
    do {
        if (cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, desc->device) != cudaSuccess) {
            rc = AP_ERR_CUDA;
            break;
        }
        const size_t bytes = ap_kv_pool_bytes(desc);
        if (!desc->k_base) {
            p->owns_planes = true;
            if (cudaMalloc(&p->desc.k_base, bytes) != cudaSuccess ||
                cudaMalloc(&p->desc.v_base, bytes) != cudaSuccess ||
                cudaMemset(p->desc.k_base, 0, bytes) != cudaSuccess ||
                cudaMemset(p->desc.v_base, 0, bytes) != cudaSuccess) {
                rc = AP_ERR_CUDA;
                break;
            }
        }
        if (cudaMalloc((void **)&p->d_counters, sizeof(int) * kMaxMergeEntries) != cudaSuccess ||
            cudaMemset(p->d_counters, 0, sizeof(int) * kMaxMergeEntries) != cudaSuccess ||
            cudaHostAlloc((void **)&p->h_status, sizeof(int), cudaHostAllocMapped) != cudaSuccess ||
            cudaHostGetDevicePointer((void **)&p->status_dev, p->h_status, 0) != cudaSuccess) {
            rc = AP_ERR_CUDA;
            break;
        }
        *p->h_status = 0;
        {
            int least = 0, greatest = 0;
            if (cudaDeviceGetStreamPriorityRange(&least, &greatest) != cudaSuccess ||
                cudaStreamCreateWithPriority(&p->side_stream, cudaStreamNonBlocking, least) != cudaSuccess ||
                cudaEventCreateWithFlags(&p->fork_event, cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&p->join_event, cudaEventDisableTiming) != cudaSuccess) {
                rc = AP_ERR_CUDA;
                break;
            }
        }
        rc = prepare_static_workspace(desc->device);
        if (rc != AP_OK) break;
        rc = encode_pool_tensor_map(&p->k_map, p->desc.k_base, desc->num_pages, desc->num_kv_heads, desc->head_dim, 1);
        if (rc != AP_OK) break;
        rc = encode_pool_tensor_map(&p->v_map, p->desc.v_base, desc->num_pages, desc->num_kv_heads, desc->head_dim, 1);
        if (rc != AP_OK) break;
        rc = encode_pool_tensor_map(&p->k_map_blk, p->desc.k_base, desc->num_pages, desc->num_kv_heads, desc->head_dim,
                                    p->head_block);
        if (rc != AP_OK) break;
        rc = encode_pool_tensor_map(&p->v_map_blk, p->desc.v_base, desc->num_pages, desc->num_kv_heads, desc->head_dim,
                                    p->head_block);
        if (rc != AP_OK) break;
        p->free_list.resize((size_t)desc->num_pages);
        for (int32_t i = 0; i < desc->num_pages; ++i) p->free_list[(size_t)i] = desc->num_pages - 1 - i;
        p->allocated.assign((size_t)desc->num_pages, 0);
    } while (false);
    if (rc != AP_OK) {
        (void)cudaGetLastError();
        ap_kv_pool_destroy(p);
        return rc;
    }
    *out = p;
    return AP_OK;
}

int ap_kv_pool_destroy(ap_kv_pool *pool) {
    if (!pool) return AP_ERR_INVALID_ARG;
    if (pool->desc.device < 0) { delete pool; return AP_OK; }
    DeviceGuard guard(pool->desc.device);
    if (guard.ok) (void)cudaDeviceSynchronize();
    for (auto &b : pool->plan_buffers) release_plan_buffer(b);
    for (auto &t : pool->timed) { (void)cudaEventDestroy(t.start); (void)cudaEventDestroy(t.stop); }
    for (auto &e : pool->spare_events) (void)cudaEventDestroy(e);
    if (pool->side_stream) (void)cudaStreamDestroy(pool->side_stream);
    if (pool->fork_event) (void)cudaEventDestroy(pool->fork_event);
    if (pool->join_event) (void)cudaEventDestroy(pool->join_event);
    if (pool->stage_dev) (void)cudaFree(pool->stage_dev);
    if (pool->d_counters) (void)cudaFree(pool->d_counters);
    if (pool->h_status) (void)cudaFreeHost(pool->h_status);
    if (pool->owns_planes) {
        if (pool->desc.k_base) (void)cudaFree(pool->desc.k_base);
        if (pool->desc.v_base) (void)cudaFree(pool->desc.v_base);
    }
    (void)cudaGetLastError();
    delete pool;
    return AP_OK;
}

int ap_kv_pool_set_side_by_side(ap_kv_pool *pool, int32_t mode) {
    if (!pool || mode < 0) return AP_ERR_INVALID_ARG;
    pool->side_by_side_mode = mode;
    return AP_OK;
}

int ap_kv_pool_set_single_launch(ap_kv_pool *pool, int32_t on) {
    if (!pool) return AP_ERR_INVALID_ARG;
    pool->single_launch = on != 0;
    return AP_OK;
}

void *ap_kv_pool_k_base(const ap_kv_pool *pool) { return pool ? pool->desc.k_base : nullptr; }
void *ap_kv_pool_v_base(const ap_kv_pool *pool) { return pool ? pool->desc.v_base : nullptr; }

int ap_kv_pool_alloc_pages(ap_kv_pool *pool, int32_t n, int32_t *out_ids) {
    if (!pool || n < 0 || (n > 0 && !out_ids)) return AP_ERR_INVALID_ARG;
    if ((size_t)n > pool->free_list.size()) return AP_ERR_OUT_OF_PAGES;
    for (int32_t i = 0; i < n; ++i) {
        int32_t id = pool->free_list.back();
        pool->free_list.pop_back();
        pool->allocated[(size_t)id] = 1;
        out_ids[i] = id;
    }
    return AP_OK;
}

int ap_kv_pool_free_pages(ap_kv_pool *pool, int32_t n, const int32_t *ids) {
    if (!pool || n < 0 || (n > 0 && !ids)) return AP_ERR_INVALID_ARG;
    // first pass validates (and detects repeats inside the call), second frees
    for (int32_t i = 0; i < n; ++i) {
        int32_t id = ids[i];
        if (id < 0 || id >= pool->desc.num_pages || pool->allocated[(size_t)id] != 1) {
            for (int32_t j = 0; j < i; ++j) pool->allocated[(size_t)ids[j]] = 1;
            return AP_ERR_INVALID_ARG;
        }
        pool->allocated[(size_t)id] = 2;  // marked within this call
    }
    for (int32_t i = 0; i < n; ++i) {
        pool->allocated[(size_t)ids[i]] = 0;
        pool->free_list.push_back(ids[i]);
    }
    return AP_OK;
}

int ap_kv_pool_seed_free_list(ap_kv_pool *pool, uint64_t seed) {
    if (!pool) return AP_ERR_INVALID_ARG;
    auto &f = pool->free_list;
    uint64_t state = seed;
    for (size_t i = f.size(); i > 1; --i) {
        size_t j = (size_t)(splitmix64(state) % (uint64_t)i);
        std::swap(f[i - 1], f[j]);
    }
    return AP_OK;
}

int32_t ap_kv_pool_num_free(const ap_kv_pool *pool) {
    return pool ? (int32_t)pool->free_list.size() : 0;
}

// ---------------------------------------------------------------- planner --

int ap_plan_create(ap_plan **out, ap_kv_pool *pool, const ap_batch_desc *b, void *stream) {
    if (!out) return AP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!pool || !b || b->batch < 0 || b->num_q_heads <= 0) return AP_ERR_INVALID_ARG;
    if (b->batch > 0 && (!b->q_lens || !b->ctx_lens || !b->block_tables || b->table_stride <= 0))
        return AP_ERR_INVALID_ARG;
    const int Hkv = pool->desc.num_kv_heads, d = pool->desc.head_dim;
    if (b->num_q_heads % Hkv != 0) return AP_ERR_INVALID_ARG;
    const int G = b->num_q_heads / Hkv;
    if (G < 1 || G > 8) return AP_ERR_UNSUPPORTED;
    const int B = b->batch;
    const int32_t num_pages = pool->desc.num_pages;

    // ---- validation + row bookkeeping
    int64_t n_new = 0, kv_tokens = 0, bt_total = 0, pairs = 0;
    int64_t decode_rows = 0, prefill_seqs = 0;
    int64_t decode_kv = 0, decode_bt = 0, prefill_kv = 0, prefill_rows = 0;   // for the work figures of ap_plan_predict
    for (int s = 0; s < B; ++s) {
        const int32_t ql = b->q_lens[s], cl = b->ctx_lens[s];
        if (ql < 0 || cl < 0 || ql > cl) return AP_ERR_INVALID_ARG;
        if (ql == 0) continue;
        const int64_t need = ((int64_t)cl + kPageSize - 1) / kPageSize;
        if (need > b->table_stride) return AP_ERR_INVALID_ARG;
        const int32_t *row = b->block_tables + (size_t)s * (size_t)b->table_stride;
        for (int64_t i = 0; i < need; ++i)
            if (row[i] < 0 || row[i] >= num_pages) return AP_ERR_BAD_BLOCK_TABLE;
        n_new += ql;
        kv_tokens += cl;
        bt_total += need;
        if (ql == 1) ++decode_rows; else ++prefill_seqs;
        if (ql > 1) pairs += (int64_t)ql * (cl - ql) + (int64_t)ql * (ql + 1) / 2;
        if (ql == 1) { decode_kv += cl; decode_bt += need; } else { prefill_kv += cl; prefill_rows += ql; }
    }
    if (n_new > (int64_t)1 << 30) return AP_ERR_UNSUPPORTED;

    std::vector<int32_t> append_dst((size_t)n_new);
    std::vector<int32_t> bt_off((size_t)B, 0);
    std::vector<int32_t> row0((size_t)B + 1, 0);
    {
        int64_t r = 0, off = 0;
        for (int s = 0; s < B; ++s) {
            row0[(size_t)s] = (int32_t)r;
            const int32_t ql = b->q_lens[s], cl = b->ctx_lens[s];
            if (ql == 0) continue;
            bt_off[(size_t)s] = (int32_t)off;
            off += ((int64_t)cl + kPageSize - 1) / kPageSize;
            const int32_t *row = b->block_tables + (size_t)s * (size_t)b->table_stride;
            for (int32_t t = 0; t < ql; ++t) {
                const int32_t p = cl - ql + t;
                append_dst[(size_t)r++] = row[p / kPageSize] * kPageSize + p % kPageSize;
            }
        }
        row0[(size_t)B] = (int32_t)r;
        // No two appended slots may alias.  A sequence's new tokens fill a slot range in each page
        // they touch, so it is enough to sort those (page, first slot, last slot) ranges and look
        // for two that overlap in one page.
        struct Range { int32_t page, lo, hi; };
        std::vector<Range> touched;
        for (int s = 0; s < B; ++s) {
            const int32_t ql = b->q_lens[s], cl = b->ctx_lens[s];
            if (ql == 0) continue;
            const int32_t *row = b->block_tables + (size_t)s * (size_t)b->table_stride;
            for (int32_t p = cl - ql; p < cl;) {
                const int32_t lp = p / kPageSize, last = std::min(cl, (lp + 1) * kPageSize) - 1;
                touched.push_back({row[lp], p % kPageSize, last % kPageSize});
                p = last + 1;
            }
        }
        std::sort(touched.begin(), touched.end(), [](const Range &a, const Range &c) {
            return a.page != c.page ? a.page < c.page : a.lo < c.lo;
        });
        for (size_t i = 1; i < touched.size(); ++i) {
            if (touched[i].page != touched[i - 1].page) continue;
            if (touched[i].lo <= touched[i - 1].hi) return AP_ERR_BAD_BLOCK_TABLE;
            touched[i].hi = std::max(touched[i].hi, touched[i - 1].hi);
        }
    }

    // ---- decode: cut the (row, kv head block) page streams into per-CTA item lists
    int max_ctas = std::max(1, pool->sm_count * decode_ctas_per_sm(d));
    const int side_ctas = side_by_side_decode_ctas(pool, b, (int)d, (int)Hkv, G, max_ctas);
    if (side_ctas > 0) max_ctas = side_ctas;
    // Costs are counted in (page, kv head) tiles.  An item covers HB kv heads, so a page of it is HB
    // tiles; a ring stage of the kernel holds kStageTiles tiles = PS pages of an item, and streams are
    // cut on stage boundaries.
    // Items span a block of kv heads when decode is confined to part of the GPU (next to prefill):
    // there an SM's stream is bound by its TMA request rate, and requests of HB tiles lift it from
    // ~58 to ~90 GB/s.  With the whole GPU decode is HBM-bound at ~41 GB/s per SM either way, and
    // one kv head per item keeps the partials (and their merge in the kernel's tail) small -- except at
    // head_dim 64, where a tile is 2 KB and single-tile requests cannot even feed 148 SMs.
    const int HB = (side_ctas > 0 || d < 128) ? pool->head_block : 1, NB = Hkv / HB;
    constexpr int kStageTiles = kDecodeTilesPerStage;
    const int PS = kStageTiles / HB;      // pages of an item per stage
    constexpr int kItemCost = 3;          // fixed per-item cost (its query load, the hand-over of its result)
    std::vector<DecodeItem> items;
    std::vector<int32_t> cta_begin;
    std::vector<MergeEntry> merges;
    int n_slots = 0;
    if (decode_rows > 0) {
        // One pass with an adaptive share: each list gets (cost still to place) / (lists still to
        // fill), so rounding cuts to stage boundaries and the extra items that cuts create spread over
        // the lists that follow instead of piling up in a last one.  `left` counts tiles plus
        // kItemCost per item still to emit.
        int64_t left = 0;
        for (int s = 0; s < B; ++s)
            if (b->q_lens[s] == 1)
                left += (int64_t)NB * ((((int64_t)b->ctx_lens[s] + kPageSize - 1) / kPageSize) * HB + kItemCost);
        const int64_t min_share = 2 * kStageTiles + kItemCost;
        items.reserve((size_t)decode_rows * NB + 2 * (size_t)max_ctas);
        cta_begin.reserve((size_t)max_ctas + 1);
        cta_begin.push_back(0);
        // (+ kStageTiles: about what a list loses to rounding; without it the loss drifts to the last lists)
        int64_t cap = std::max<int64_t>((left + max_ctas - 1) / max_ctas + kStageTiles, min_share);
        auto next_cta = [&]() {
            if ((int32_t)items.size() > cta_begin.back()) cta_begin.push_back((int32_t)items.size());
            const int lists_left = max_ctas - ((int)cta_begin.size() - 1);
            cap = lists_left <= 1 ? INT64_MAX / 2
                                  : std::max<int64_t>((left + lists_left - 1) / lists_left + kStageTiles, min_share);
        };
        for (int s = 0; s < B; ++s) {
            if (b->q_lens[s] != 1) continue;
            const int32_t cl = b->ctx_lens[s];
            const int32_t pages = (cl + kPageSize - 1) / kPageSize;
            for (int hb = 0; hb < NB; ++hb) {
                int32_t rem = pages, pb = 0;
                const size_t first = items.size();
                while (rem > 0) {
                    const int64_t avail = (cap - kItemCost) / HB;          // pages this list can still take
                    if (avail < PS && avail < rem) { next_cta(); continue; }
                    int32_t take = (int32_t)std::min<int64_t>(rem, avail);
                    if (take < rem) take = take / PS * PS;
                    DecodeItem it{};
                    it.q_row = row0[(size_t)s];
                    it.kv_head = hb * HB;
                    it.bt_offset = bt_off[(size_t)s];
                    it.page_begin = pb;
                    it.page_count = take;
                    it.kv_len = cl;
                    it.part_slot = -1;
                    it.merge_index = -1;
                    items.push_back(it);
                    cap -= (int64_t)take * HB + kItemCost;
                    pb += take;
                    rem -= take;
                    left -= (int64_t)take * HB + (rem > 0 ? 0 : kItemCost);   // a cut leaves one more item to emit
                    if (cap < kItemCost + kStageTiles) next_cta();
                }
                if (items.size() - first > 1) {
                    MergeEntry m{row0[(size_t)s], hb * HB, n_slots, (int32_t)(items.size() - first)};
                    merges.push_back(m);
                    for (size_t i = first; i < items.size(); ++i) {
                        items[i].part_slot = n_slots++;
                        items[i].merge_index = (int32_t)merges.size() - 1;
                    }
                }
            }
        }
        if ((int32_t)items.size() > cta_begin.back()) cta_begin.push_back((int32_t)items.size());
    }
    const int n_ctas = cta_begin.empty() ? 0 : (int)cta_begin.size() - 1;
    // Inside a CTA, items of cut streams go first: their partials are then merged
    // in mid-kernel, behind the running pipeline, and not in the kernel's tail.
    for (int c = 0; c < n_ctas; ++c)
        std::stable_partition(items.begin() + cta_begin[(size_t)c], items.begin() + cta_begin[(size_t)c + 1],
                              [](const DecodeItem &it) { return it.part_slot >= 0; });
    // (streams are cut at CTA boundaries only, so a CTA has at most two partial items and the
    // workspace at most two slots per CTA)
    if ((int)merges.size() > kMaxMergeEntries) return AP_ERR_UNSUPPORTED;

    // ---- prefill tiles, longest first
    std::vector<PrefillTile> tiles;
    for (int s = 0; s < B; ++s) {
        const int32_t ql = b->q_lens[s], cl = b->ctx_lens[s];
        if (ql <= 1) continue;
        for (int32_t t0 = 0; t0 < ql; t0 += 128) {
            // two q heads of one kv head share a work unit (and its K/V stream); an odd head is alone
            for (int h = 0; h < b->num_q_heads; h += ((h % G) + 1 < G ? 2 : 1)) {
                PrefillTile t{};
                t.q_row0 = row0[(size_t)s] + t0;
                t.rows = std::min(128, ql - t0);
                t.q_head = h;
                t.q_head_b = (h % G) + 1 < G ? h + 1 : -1;
                t.kv_head = h / G;
                t.bt_offset = bt_off[(size_t)s];
                t.pos0 = cl - ql + t0;
                t.ctx_len = cl;
                tiles.push_back(t);
            }
        }
    }
    std::stable_sort(tiles.begin(), tiles.end(), [](const PrefillTile &a, const PrefillTile &c) {
        return a.pos0 + a.rows > c.pos0 + c.rows;
    });

    // ---- blob layout (int32 units, every section 32-byte aligned)
    auto sec = [](size_t &cursor, size_t n_ints) {
        size_t at = cursor;
        cursor = (cursor + n_ints + 7) / 8 * 8;
        return at;
    };
    size_t cursor = 0;
    const size_t o_append = sec(cursor, (size_t)n_new);
    const size_t o_bt = sec(cursor, (size_t)bt_total);
    const size_t o_items = sec(cursor, items.size() * 8);
    const size_t o_cta = sec(cursor, cta_begin.size());
    const size_t o_merge = sec(cursor, merges.size() * 4);
    const size_t o_tiles = sec(cursor, tiles.size() * 8);
    const size_t total_ints = std::max<size_t>(cursor, 8);

    ap_plan *plan = new (std::nothrow) ap_plan();
    if (!plan) return AP_ERR_CUDA;
    plan->blob.assign(total_ints, 0);
    int32_t *h = plan->blob.data();
    if (n_new) std::memcpy(h + o_append, append_dst.data(), (size_t)n_new * 4);
    for (int s = 0; s < B; ++s) {
        if (b->q_lens[s] == 0) continue;
        const size_t need = ((size_t)b->ctx_lens[s] + kPageSize - 1) / kPageSize;
        std::memcpy(h + o_bt + bt_off[(size_t)s], b->block_tables + (size_t)s * (size_t)b->table_stride, need * 4);
    }
    if (!items.empty()) std::memcpy(h + o_items, items.data(), items.size() * sizeof(DecodeItem));
    if (!cta_begin.empty()) std::memcpy(h + o_cta, cta_begin.data(), cta_begin.size() * 4);
    if (!merges.empty()) std::memcpy(h + o_merge, merges.data(), merges.size() * sizeof(MergeEntry));
    if (!tiles.empty()) std::memcpy(h + o_tiles, tiles.data(), tiles.size() * sizeof(PrefillTile));
    plan->layout.total_ints = (int64_t)total_ints;
    plan->layout.append_dst = (int64_t)o_append;
    plan->layout.bt_flat = (int64_t)o_bt;
    plan->layout.decode_items = (int64_t)o_items;
    plan->layout.cta_begin = (int64_t)o_cta;
    plan->layout.merge_entries = (int64_t)o_merge;
    plan->layout.prefill_tiles = (int64_t)o_tiles;
    plan->layout.n_bt = bt_total;
    plan->layout.n_cta_begin = (int64_t)cta_begin.size();

    if (pool->desc.device >= 0) {
        DeviceGuard guard(pool->desc.device);
        if (!guard.ok) { delete plan; return AP_ERR_CUDA; }
        int rc = acquire_plan_buffer(pool, total_ints, &plan->buf);
        if (rc != AP_OK) { delete plan; return rc; }
        std::memcpy(plan->buf.host, h, total_ints * 4);
        cudaStream_t st = (cudaStream_t)stream;
        if (cudaMemcpyAsync(plan->buf.dev, plan->buf.host, total_ints * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaEventRecord(plan->buf.uploaded, st) != cudaSuccess) {
            (void)cudaGetLastError();
            pool->plan_buffers.push_back(plan->buf);
            delete plan;
            return AP_ERR_CUDA;
        }
    }

    plan->pool = pool;
    plan->num_q_heads = b->num_q_heads;
    plan->group = G;
    plan->scale = b->softmax_scale > 0.f ? b->softmax_scale : 1.0f / std::sqrt((float)d);
    plan->n_part_slots = n_slots;
    plan->head_block = HB;
    plan->d_append_dst = plan->buf.dev + o_append;
    plan->d_bt_flat = plan->buf.dev + o_bt;
    plan->d_items = (const DecodeItem *)(plan->buf.dev + o_items);
    plan->d_cta_begin = plan->buf.dev + o_cta;
    plan->d_merge = (const MergeEntry *)(plan->buf.dev + o_merge);
    plan->d_tiles = (const PrefillTile *)(plan->buf.dev + o_tiles);
    plan->ws.o_part_off = 0;
    plan->ws.lse_part_off = align_up((size_t)n_slots * HB * G * d * sizeof(float), 256);
    plan->ws.bytes = n_slots ? plan->ws.lse_part_off + align_up((size_t)n_slots * HB * G * sizeof(float), 256) : 0;

    ap_plan_info &info = plan->info;
    info.n_new = n_new;
    info.kv_tokens = kv_tokens;
    info.decode_rows = decode_rows;
    info.prefill_seqs = prefill_seqs;
    info.prefill_pairs = pairs;
    info.decode_items = (int64_t)items.size();
    info.decode_ctas = n_ctas;
    info.merge_entries = (int64_t)merges.size();
    info.prefill_tiles = (int64_t)tiles.size();
    info.launches_append = n_new > 0 ? 1 : 0;
    {
        // algorithmic work of one layer: every attended KV token's K and V once per kv head, q read,
        // out + lse written, used block-table entries once; 4 d flop per (q head, query row, unmasked key)
        const double per_kv_token = 2.0 * (double)Hkv * (double)d * 2.0;
        const double per_row = 2.0 * (double)b->num_q_heads * (double)d * 2.0 + (double)b->num_q_heads * 4.0;
        plan->work.decode_bytes = (double)decode_kv * per_kv_token + (double)decode_rows * per_row + (double)decode_bt * 4.0;
        plan->work.prefill_bytes = (double)prefill_kv * per_kv_token + (double)prefill_rows * per_row;
        plan->work.append_bytes = 2.0 * (double)n_new * per_kv_token;
        plan->work.decode_flops = 4.0 * (double)b->num_q_heads * (double)d * (double)decode_kv;
        plan->work.prefill_flops = 4.0 * (double)b->num_q_heads * (double)d * (double)pairs;
        double w_p = 0.0;
        for (const PrefillTile &t : tiles) {
            const int steps = (t.pos0 + t.rows + 127) / 128;
            w_p += steps * (t.q_head_b >= 0 ? kPrefillStepUs : kPrefillStepSingleUs) * ((double)d / 128.0) + kPrefillUnitUs;
        }
        plan->work.prefill_sm_us = w_p;
    }
    plan->side_by_side = side_ctas > 0 && !items.empty() && !tiles.empty();
    plan->single_launch = plan->side_by_side && pool->single_launch;
    info.launches_attention = plan->single_launch ? 1 : (items.empty() ? 0 : 1) + (tiles.empty() ? 0 : 1);
    info.side_by_side = plan->side_by_side ? 1 : 0;
    info.decode_head_block = HB;
    *out = plan;
    return AP_OK;
}

int ap_plan_predict(const ap_plan *plan, double hbm_gbs, double tensor_tflops, ap_plan_prediction *out) {
    if (!plan || !out || !plan->pool) return AP_ERR_INVALID_ARG;
    const double B = (hbm_gbs > 0.0 ? hbm_gbs : 6448.0) * 1e9;             // bytes / s
    const double F = (tensor_tflops > 0.0 ? tensor_tflops : 1642.0) * 1e12; // flop / s
    const PlanWork &w = plan->work;
    ap_plan_prediction e{};
    e.decode_bytes = w.decode_bytes;
    e.decode_flops = w.decode_flops;
    e.prefill_bytes = w.prefill_bytes;
    e.prefill_flops = w.prefill_flops;
    e.append_bytes = w.append_bytes;
    // Eq. "roofline": pi = min(F/A * B_g, F_g), T_op = F / pi; an operator without flops moves its bytes
    auto t_op_us = [&](double flops, double bytes) {
        if (bytes <= 0.0) return 0.0;
        if (flops <= 0.0) return bytes / B * 1e6;
        return flops / std::min(flops / bytes * B, F) * 1e6;
    };
    e.roofline_decode_us = t_op_us(w.decode_flops, w.decode_bytes);
    e.roofline_prefill_us = t_op_us(w.prefill_flops, w.prefill_bytes);
    e.roofline_append_us = t_op_us(0.0, w.append_bytes);
    // calibrated model (the one the planner's side-by-side decision uses)
    const int sms = plan->pool->sm_count;
    const double ctas = (double)std::max<int64_t>(plan->info.decode_ctas, 1);
    const double decode_rate = std::min(ctas * decode_sm_gbs(plan->head_block * kPageSize * plan->pool->desc.head_dim * 2),
                                        kDecodeGpuGBs) * 1e3;                             // bytes / us
    e.model_decode_us = w.decode_bytes > 0.0 ? w.decode_bytes / decode_rate + kDecodeFixedUs : 0.0;
    e.model_prefill_us = w.prefill_sm_us > 0.0 ? w.prefill_sm_us / sms + kPrefillTailUs : 0.0;
    const double append_us = w.append_bytes > 0.0 ? w.append_bytes / (kAppendGBs * 1e3) + kAppendFixedUs : 0.0;
    if (plan->side_by_side)
        e.model_step_us = append_us + kPrefillTailUs +
                          side_by_side_us(w.decode_bytes, w.prefill_sm_us, (int)plan->info.decode_ctas,
                                          decode_sm_gbs(plan->head_block * kPageSize * plan->pool->desc.head_dim * 2) * 1e3, sms);
    else
        e.model_step_us = append_us + e.model_decode_us + e.model_prefill_us;
    *out = e;
    return AP_OK;
}

int ap_plan_destroy(ap_plan *plan) {
    if (!plan) return AP_ERR_INVALID_ARG;
    if (plan->pool && plan->buf.dev) plan->pool->plan_buffers.push_back(plan->buf);
    delete plan;
    return AP_OK;
}

size_t ap_plan_workspace_bytes(const ap_plan *plan) { return plan ? plan->ws.bytes : 0; }

int ap_plan_get_info(const ap_plan *plan, ap_plan_info *info) {
    if (!plan || !info) return AP_ERR_INVALID_ARG;
    *info = plan->info;
    return AP_OK;
}

int ap_plan_export(const ap_plan *plan, int32_t *blob, size_t capacity_ints, ap_plan_layout *layout) {
    if (!plan || !layout) return AP_ERR_INVALID_ARG;
    *layout = plan->layout;
    if (blob) {
        if (capacity_ints < plan->blob.size()) return AP_ERR_INVALID_ARG;
        std::memcpy(blob, plan->blob.data(), plan->blob.size() * 4);
    }
    return AP_OK;
}

// --------------------------------------------------------------- dispatch --

int ap_kv_append(ap_kv_pool *pool, const ap_plan *plan, const void *k_new, const void *v_new, void *stream) {
    if (!pool || !plan || plan->pool != pool) return AP_ERR_INVALID_ARG;
    if (pool->desc.device < 0) return AP_ERR_CUDA;
    if (plan->info.n_new == 0) return AP_OK;
    if (!k_new || !v_new || (((uintptr_t)k_new | (uintptr_t)v_new) & 15u)) return AP_ERR_INVALID_ARG;
    DeviceGuard guard(pool->desc.device);
    if (!guard.ok) return AP_ERR_CUDA;
    TimedScope timed(pool, AP_KERNEL_APPEND, (cudaStream_t)stream);
    if (launch_kv_append(pool, plan, k_new, v_new, (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return AP_ERR_CUDA;
    }
    return AP_OK;
}

int ap_kv_copy_pages(ap_kv_pool *dst_pool, const ap_kv_pool *src_pool, int32_t n, const int32_t *dst_ids,
                     const int32_t *src_ids, void *stream) {
    if (!dst_pool || !src_pool || n < 0 || (n > 0 && (!dst_ids || !src_ids))) return AP_ERR_INVALID_ARG;
    const ap_pool_desc &dd = dst_pool->desc, &sd = src_pool->desc;
    if (dd.num_kv_heads != sd.num_kv_heads || dd.head_dim != sd.head_dim || dd.page_size != sd.page_size)
        return AP_ERR_INVALID_ARG;
    if ((dd.device < 0) != (sd.device < 0) || (dd.device >= 0 && dd.device != sd.device)) return AP_ERR_UNSUPPORTED;
    // Validation on the host, before anything is queued.  The copies run in parallel, so a
    // destination may appear once only and, inside one pool, may not be another pair's source.
    const bool same = dst_pool == src_pool || (dd.device >= 0 && dd.k_base == sd.k_base);
    std::vector<uint8_t> is_dst((size_t)dd.num_pages, 0);
    std::vector<int32_t> pairs;
    pairs.reserve(2 * (size_t)n);
    for (int32_t i = 0; i < n; ++i) {
        if (dst_ids[i] < 0 || dst_ids[i] >= dd.num_pages || src_ids[i] < 0 || src_ids[i] >= sd.num_pages)
            return AP_ERR_BAD_BLOCK_TABLE;
        if (is_dst[(size_t)dst_ids[i]]) return AP_ERR_INVALID_ARG;
        is_dst[(size_t)dst_ids[i]] = 1;
        if (same && dst_ids[i] == src_ids[i]) continue;           // a page copied onto itself: nothing to do
        pairs.push_back(dst_ids[i]);
        pairs.push_back(src_ids[i]);
    }
    if (same)
        for (int32_t i = 0; i < n; ++i)
            if (dst_ids[i] != src_ids[i] && is_dst[(size_t)src_ids[i]]) return AP_ERR_INVALID_ARG;
    if (pairs.empty() || dd.device < 0) return AP_OK;             // a host-only pool has no planes to copy
    DeviceGuard guard(dd.device);
    if (!guard.ok) return AP_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    PlanBuffer buf;
    int rc = acquire_plan_buffer(dst_pool, pairs.size(), &buf);
    if (rc != AP_OK) return rc;
    std::memcpy(buf.host, pairs.data(), pairs.size() * sizeof(int32_t));
    cudaError_t e = cudaMemcpyAsync(buf.dev, buf.host, pairs.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = launch_kv_copy_pages(dst_pool, src_pool, buf.dev, (int)(pairs.size() / 2), st);
    // the staging area is free again once the kernel has read the pair list
    if (e == cudaSuccess) e = cudaEventRecord(buf.uploaded, st);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        (void)cudaStreamSynchronize(st);
        release_plan_buffer(buf);
        return AP_ERR_CUDA;
    }
    dst_pool->plan_buffers.push_back(buf);
    return AP_OK;
}

int ap_attention_iteration(ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                           void *workspace, size_t workspace_bytes, void *stream) {
    if (!pool || !plan || plan->pool != pool) return AP_ERR_INVALID_ARG;
    if (pool->desc.device < 0) return AP_ERR_CUDA;
    if (plan->info.n_new == 0) return AP_OK;
    if (!q || !out || (((uintptr_t)q | (uintptr_t)out) & 15u)) return AP_ERR_INVALID_ARG;
    if (plan->ws.bytes > 0) {
        if (!workspace || workspace_bytes < plan->ws.bytes) return AP_ERR_WORKSPACE_TOO_SMALL;
        if ((uintptr_t)workspace & 255u) return AP_ERR_INVALID_ARG;
    }
    DeviceGuard guard(pool->desc.device);
    if (!guard.ok) return AP_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    float *o_part = plan->ws.bytes ? (float *)((char *)workspace + plan->ws.o_part_off) : nullptr;
    float *lse_part = plan->ws.bytes ? (float *)((char *)workspace + plan->ws.lse_part_off) : nullptr;
    const cudaError_t e = ap::launch_attention_kernels(pool, plan, q, out, lse, o_part, lse_part, st);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return e == cudaErrorNotSupported ? AP_ERR_UNSUPPORTED : AP_ERR_CUDA;
    }
    return AP_OK;
}

int ap_last_device_status(ap_kv_pool *pool, void *stream) {
    if (!pool) return AP_ERR_INVALID_ARG;
    if (pool->desc.device < 0) return AP_ERR_CUDA;
    DeviceGuard guard(pool->desc.device);
    if (!guard.ok) return AP_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    // the kernels write the word straight into host memory: after the synchronisation it can be read here
    if (cudaStreamSynchronize(st) != cudaSuccess) {
        (void)cudaGetLastError();
        return AP_ERR_CUDA;
    }
    const int status = *reinterpret_cast<volatile int *>(pool->h_status);
    if (status != 0) {
        *reinterpret_cast<volatile int *>(pool->h_status) = 0;
        // a kernel that gave up may have left merge arrival counters behind: clear them too
        if (cudaMemsetAsync(pool->d_counters, 0, sizeof(int) * kMaxMergeEntries, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess) {
            (void)cudaGetLastError();
            return AP_ERR_CUDA;
        }
    }
    return status;
}

int ap_kv_pool_set_wait_limit(ap_kv_pool *pool, uint64_t limit_ns) {
    if (!pool) return AP_ERR_INVALID_ARG;
    pool->wait_limit_ns = limit_ns ? limit_ns : kDefaultWaitLimitNs;
    return AP_OK;
}

int ap_selftest_wait_timeout(ap_kv_pool *pool, uint64_t limit_ns, int leave_counter, void *stream) {
    if (!pool || limit_ns == 0 || limit_ns > kDefaultWaitLimitNs) return AP_ERR_INVALID_ARG;
    if (pool->desc.device < 0) return AP_ERR_CUDA;
    DeviceGuard guard(pool->desc.device);
    if (!guard.ok) return AP_ERR_CUDA;
    if (launch_selftest_wait(pool, limit_ns, leave_counter != 0, (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return AP_ERR_CUDA;
    }
    return AP_OK;
}

int ap_profile_enable(ap_kv_pool *pool, int on) {
    if (!pool) return AP_ERR_INVALID_ARG;
    if (pool->desc.device < 0) return AP_ERR_CUDA;
    for (auto &t : pool->timed) {
        pool->spare_events.push_back(t.start);
        pool->spare_events.push_back(t.stop);
    }
    pool->timed.clear();
    pool->profiling = on != 0;
    return AP_OK;
}

int ap_profile_collect(ap_kv_pool *pool, void *stream, ap_kernel_times *out) {
    if (!pool || !out) return AP_ERR_INVALID_ARG;
    if (pool->desc.device < 0) return AP_ERR_CUDA;
    DeviceGuard guard(pool->desc.device);
    if (!guard.ok) return AP_ERR_CUDA;
    std::memset(out, 0, sizeof(*out));
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) { (void)cudaGetLastError(); return AP_ERR_CUDA; }
    int rc = AP_OK;
    for (auto &t : pool->timed) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, t.start, t.stop) == cudaSuccess && t.kernel >= 0 && t.kernel < AP_KERNEL_COUNT) {
            out->ms[t.kernel] += ms;
            out->launches[t.kernel] += 1;
        } else {
            (void)cudaGetLastError();
            rc = AP_ERR_CUDA;
        }
        pool->spare_events.push_back(t.start);
        pool->spare_events.push_back(t.stop);
    }
    pool->timed.clear();
    return rc;
}

int ap_serving_iteration_host(ap_kv_pool *pool, const ap_batch_desc *batch, const void *q_host,
                              const void *k_new_host, const void *v_new_host, void *out_host,
                              float *lse_host, void *stream) {
    if (!pool || !batch) return AP_ERR_INVALID_ARG;
    if (pool->desc.device < 0) return AP_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    if (batch->batch < 0 || batch->num_q_heads <= 0 || (batch->batch > 0 && !batch->q_lens)) return AP_ERR_INVALID_ARG;
    // The input copies do not depend on the plan, so they are issued first and run while the host
    // plans; only their sizes (the number of new tokens) are needed up front.
    size_t n = 0;
    for (int s = 0; s < batch->batch; ++s) {
        if (batch->q_lens[s] < 0) return AP_ERR_INVALID_ARG;
        n += (size_t)batch->q_lens[s];
    }
    if (n > (size_t)1 << 30) return AP_ERR_UNSUPPORTED;
    if (n > 0 && (!q_host || !k_new_host || !v_new_host || !out_host)) return AP_ERR_INVALID_ARG;
    DeviceGuard guard(pool->desc.device);
    if (!guard.ok) return AP_ERR_CUDA;
    const size_t d = (size_t)pool->desc.head_dim, Hq = (size_t)batch->num_q_heads, Hkv = (size_t)pool->desc.num_kv_heads;
    if (Hq % Hkv != 0 || Hq / Hkv > 8) return Hq % Hkv != 0 ? AP_ERR_INVALID_ARG : AP_ERR_UNSUPPORTED;
    const size_t q_bytes = align_up(n * Hq * d * 2, 256), kv_bytes = align_up(n * Hkv * d * 2, 256);
    const size_t lse_bytes = align_up(n * Hq * 4, 256);
    // every decode CTA leaves at most two partials, which bounds the workspace before planning
    const size_t max_slots = 2 * (size_t)std::max(1, pool->sm_count * decode_ctas_per_sm((int)d));
    const size_t part_heads = (size_t)pool->head_block * (Hq / Hkv);      // query heads of one decode item
    const size_t ws_bytes = align_up(max_slots * part_heads * d * sizeof(float), 256) +
                            align_up(max_slots * part_heads * sizeof(float), 256);
    const size_t total = 2 * q_bytes + 2 * kv_bytes + lse_bytes + ws_bytes;
    if (total > pool->stage_bytes) {
        if (pool->stage_dev) {
            (void)cudaDeviceSynchronize();
            (void)cudaFree(pool->stage_dev);
            pool->stage_dev = nullptr;
            pool->stage_bytes = 0;
        }
        const size_t want = total + total / 4;
        if (cudaMalloc(&pool->stage_dev, want) != cudaSuccess) {
            (void)cudaGetLastError();
            return AP_ERR_CUDA;
        }
        pool->stage_bytes = want;
    }
    char *base = (char *)pool->stage_dev;
    void *dq = base, *dout = base + q_bytes, *dk = base + 2 * q_bytes, *dv = base + 2 * q_bytes + kv_bytes;
    float *dlse = (float *)(base + 2 * q_bytes + 2 * kv_bytes);
    void *dws = base + 2 * q_bytes + 2 * kv_bytes + lse_bytes;
    bool ok = n == 0 ||
              (cudaMemcpyAsync(dq, q_host, n * Hq * d * 2, cudaMemcpyHostToDevice, st) == cudaSuccess &&
               cudaMemcpyAsync(dk, k_new_host, n * Hkv * d * 2, cudaMemcpyHostToDevice, st) == cudaSuccess &&
               cudaMemcpyAsync(dv, v_new_host, n * Hkv * d * 2, cudaMemcpyHostToDevice, st) == cudaSuccess);
    if (!ok) {
        (void)cudaGetLastError();
        return AP_ERR_CUDA;
    }
    ap_plan *plan = nullptr;
    int rc = ap_plan_create(&plan, pool, batch, stream);
    if (rc != AP_OK) {               // the copies already queued only touch the staging buffer,
        (void)cudaStreamSynchronize(st);   // but they read the caller's memory: let them finish
        return rc;
    }
    if (n == 0) { ap_plan_destroy(plan); return AP_OK; }
    if (plan->ws.bytes > ws_bytes) { ap_plan_destroy(plan); return AP_ERR_WORKSPACE_TOO_SMALL; }
    rc = ap_kv_append(pool, plan, dk, dv, stream);
    if (rc == AP_OK) rc = ap_attention_iteration(pool, plan, dq, dout, dlse, dws, ws_bytes, stream);
    if (rc == AP_OK) {
        ok = cudaMemcpyAsync(out_host, dout, n * Hq * d * 2, cudaMemcpyDeviceToHost, st) == cudaSuccess;
        if (ok && lse_host)
            ok = cudaMemcpyAsync(lse_host, dlse, n * Hq * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    }
    if (!ok) { (void)cudaGetLastError(); rc = AP_ERR_CUDA; }
    const int dev_status = ap_last_device_status(pool, stream);  // synchronises the stream
    ap_plan_destroy(plan);
    return rc != AP_OK ? rc : dev_status;
}

}  // extern "C"
