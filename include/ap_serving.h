/*
 * ap_serving.h -- C ABI of the paged-KV serving-iteration library (sm_100a).
 *
 * One continuous-batching serving iteration over a ragged batch: the new
 * tokens' K/V are appended into a paged KV pool through per-sequence block
 * tables, then every new token attends its sequence's context with
 * grouped-query attention.  Sequences with one new token are decode steps,
 * sequences with more are prefill chunks (causal inside the chunk).
 *
 * Where the operations come from.  The paper treats this iteration as the unit
 * of work whose batch composition the scheduling policy decides and models it
 * only by cost: continuous batching and per-operator time (Sec. 5.3 "Serving
 * simulator"); a decode step k attends a context of k tokens including the new
 * one, prefill is the separate longer-query operation (App. B, Eq.
 * "serve-latency"); attention heads A_z, KV heads K_z <= A_z, head dimension
 * d_z (App. B, model description); the KV cache is a finite pool counted in
 * tokens (App. B Eq. "oom", theta = 0.8; App. C.2 "token-capacity limits");
 * KV caches are relocatable (Sec. 5.1, Phase 2), hence block-table
 * indirection; paged KV memory and chunked prefill are the data-plane
 * techniques of the served systems (App. H).  The arithmetic itself is the
 * textbook definition:
 *     x_j = scale * <q, k_j>, j = 0..p;  out = softmax(x) V;  lse = ln sum_j e^{x_j}.
 *
 * Conventions
 *   - All functions return int: AP_OK (0) or a negative ap_status.  Nothing
 *     aborts, throws or traps the GPU.  Host-side validation happens before
 *     any launch.
 *   - "host" / "device" on a pointer says which memory it must point to.
 *   - bf16 tensors are passed as void* (16-bit storage); page size is 16.
 *   - Layouts (row-major, innermost last):
 *         pool planes  K, V : [num_pages][num_kv_heads][16][head_dim]  bf16
 *         q, out            : [N_new][num_q_heads][head_dim]           bf16
 *         k_new, v_new      : [N_new][num_kv_heads][head_dim]          bf16
 *         lse               : [N_new][num_q_heads]                     fp32, natural log
 *     N_new = sum of q_lens; rows of all sequences are concatenated in batch
 *     order.  q head h uses kv head h / (num_q_heads / num_kv_heads).
 *   - Calls taking a stream are asynchronous and stream-ordered: ap_kv_append
 *     followed by ap_attention_iteration on the same stream needs no sync.
 *   - A plan must outlive the launches that use it (destroy it after the stream
 *     has passed them, or after ap_last_device_status).
 *   - A pool and its plans are not thread-safe: calls that name the same pool must
 *     come from one host thread at a time (the pool owns staging buffers, a second
 *     stream with its fork / join events, and the allocator state).  Different pools
 *     are independent.  Launches of one pool on different streams that may overlap
 *     on the GPU are not supported either: they share the split-K arrival counters.
 */
#ifndef AP_SERVING_H
#define AP_SERVING_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum ap_status {
    AP_OK = 0,
    AP_ERR_INVALID_ARG = -1,
    AP_ERR_OUT_OF_PAGES = -2,
    AP_ERR_BAD_BLOCK_TABLE = -3,
    AP_ERR_WORKSPACE_TOO_SMALL = -4,
    AP_ERR_CUDA = -5,
    AP_ERR_TIMEOUT = -6,
    AP_ERR_UNSUPPORTED = -7
};

typedef struct ap_kv_pool ap_kv_pool; /* opaque */
typedef struct ap_plan ap_plan;       /* opaque */

/* ------------------------------------------------------------------ pool -- */

/*
 * KV page pool (finite token capacity: App. B Eq. "oom", App. C.2).
 * k_base/v_base: device, each ap_kv_pool_bytes() long and 16-byte aligned
 * (what a tensor map's base address needs), owned by the caller; or both NULL,
 * then the library allocates (and zero fills) and frees them.  head_dim is 64 or 128; page_size must be 16;
 * num_q_heads / num_kv_heads may be 1..8 (given per batch).
 */
typedef struct ap_pool_desc {
    int32_t num_pages;
    int32_t page_size;
    int32_t num_kv_heads;
    int32_t head_dim;
    void *k_base; /* device or NULL */
    void *v_base; /* device or NULL */
    int32_t device;
} ap_pool_desc;

/* Bytes of ONE plane (K or V) for this description; 0 if the description is invalid. */
size_t ap_kv_pool_bytes(const ap_pool_desc *desc);

/*
 * Creates the pool handle on desc->device: free list with all pages free in
 * ascending order, tensor maps over both planes, a device status word.
 * desc->device < 0 (with both bases NULL) creates a HOST-ONLY pool: the page
 * allocator, ap_plan_create and ap_plan_export work (planning for 148 SMs);
 * every call that would launch returns AP_ERR_CUDA.
 * Errors: INVALID_ARG (bad sizes, one base NULL, misaligned), UNSUPPORTED
 * (head_dim/page_size), CUDA (no device, allocation failure). */
int ap_kv_pool_create(ap_kv_pool **out, const ap_pool_desc *desc);

/* Frees the handle and only what the library allocated.  Synchronises the device. */
int ap_kv_pool_destroy(ap_kv_pool *pool);

/* Device addresses of the planes (caller's or the library's). */
void *ap_kv_pool_k_base(const ap_kv_pool *pool);
void *ap_kv_pool_v_base(const ap_kv_pool *pool);

/*
 * Side-by-side execution of mixed iterations (Sec. 5.3: the batch an iteration
 * runs, prefill chunks next to decode tokens, is what the scheduling policy
 * composes).  When a plan holds both decode rows and prefill chunks, decode can
 * be confined to k persistent CTAs (where it is bound by what an SM can stream,
 * not by HBM) while the prefill units run on the other SMs at the same time and
 * take over the decode CTAs' SMs as those retire.  Both parts then go out in ONE
 * launch on the caller's stream: the decode CTAs are the first k blocks of the
 * grid, every later block is one prefill unit.
 * mode 0: never (decode kernel, then prefill kernel); mode 1 (default):
 * ap_plan_create decides per plan from a cost model and picks k; mode >= 2:
 * always, with k = mode decode CTAs (clamped).  Applies to plans created
 * afterwards; results are identical in every mode up to the summation order of
 * split-K partials.  ap_plan_info.side_by_side reports what a plan does.
 * mode < 0 -> INVALID_ARG.
 */
int ap_kv_pool_set_side_by_side(ap_kv_pool *pool, int32_t mode);
/* on = 0: side-by-side plans use two launches instead, the decode kernel on the caller's stream and the
 * prefill kernel on a low-priority stream the pool owns, forked and joined with events (kept for
 * comparison); on != 0 (default): the single launch.  Applies to plans created afterwards. */
int ap_kv_pool_set_single_launch(ap_kv_pool *pool, int32_t on);

/* Host page allocator (per-request page ownership; pages are relocatable units,
 * Sec. 5.1 Phase 2).  alloc is all-or-nothing: OUT_OF_PAGES leaves the free
 * list unchanged.  out_ids / ids: host.  free of a page that is not allocated,
 * out of range or repeated in the call -> INVALID_ARG, nothing freed. */
int ap_kv_pool_alloc_pages(ap_kv_pool *pool, int32_t n, int32_t *out_ids);
int ap_kv_pool_free_pages(ap_kv_pool *pool, int32_t n, const int32_t *ids);
/* Shuffles the order in which FREE pages will be handed out (Fisher-Yates on a
 * splitmix64 stream).  Allocated pages are unaffected. */
int ap_kv_pool_seed_free_list(ap_kv_pool *pool, uint64_t seed);
int32_t ap_kv_pool_num_free(const ap_kv_pool *pool);

/* ------------------------------------------------------------------ plan -- */

/*
 * One iteration's batch (Sec. 5.3: the batch the policy composed).
 * All arrays are HOST memory and are only read during ap_plan_create.
 */
typedef struct ap_batch_desc {
    int32_t batch;               /* number of sequences B (>= 0) */
    int32_t num_q_heads;         /* multiple of the pool's num_kv_heads, ratio 1..8 */
    const int32_t *q_lens;       /* [B] new tokens this iteration: 0 skipped, 1 decode, >1 prefill chunk */
    const int32_t *ctx_lens;     /* [B] context length INCLUDING this iteration's new tokens */
    const int32_t *block_tables; /* [B][table_stride] logical -> physical page; entries past ceil(ctx/16) are never read */
    int32_t table_stride;
    float softmax_scale;         /* <= 0 selects 1/sqrt(head_dim) */
} ap_batch_desc;

/*
 * Validates the batch and builds the device work lists (append destinations,
 * split-K decode items balanced over the SMs, LSE-merge entries, prefill
 * tiles), uploaded with one asynchronous copy on `stream`.
 * Validation: 0 <= q_len <= ctx_len; table_stride >= ceil(ctx_len/16) for every
 * sequence with q_len > 0; every used entry in [0, num_pages)
 * (BAD_BLOCK_TABLE); no two appended token slots alias (BAD_BLOCK_TABLE);
 * head ratio 1..8 (UNSUPPORTED).  Pages shared between sequences for reading
 * are legal.  On error *out is NULL and nothing was launched.
 */
int ap_plan_create(ap_plan **out, ap_kv_pool *pool, const ap_batch_desc *batch, void *stream);
int ap_plan_destroy(ap_plan *plan);

/* Bytes of caller-provided device workspace (split-K partials) that
 * ap_attention_iteration needs for this plan; may be 0. */
size_t ap_plan_workspace_bytes(const ap_plan *plan);

typedef struct ap_plan_info {
    int64_t n_new;           /* rows of q / k_new / v_new / out */
    int64_t kv_tokens;       /* sum of ctx_len over sequences with q_len > 0 */
    int64_t decode_rows;     /* sequences with q_len == 1 */
    int64_t prefill_seqs;    /* sequences with q_len > 1 */
    int64_t prefill_pairs;   /* unmasked (query row, key) pairs of the prefill chunks, one head */
    int64_t decode_items;    /* split-K work items */
    int64_t decode_ctas;     /* persistent CTAs of the decode kernel */
    int64_t merge_entries;   /* (row, kv head) results assembled from > 1 partial */
    int64_t prefill_tiles;   /* work units of the prefill kernel */
    int64_t launches_append; /* kernels ap_kv_append launches for this plan */
    int64_t launches_attention; /* kernels ap_attention_iteration launches for this plan */
    int64_t side_by_side;    /* 1 if the decode and prefill kernels of this plan run concurrently */
    int64_t decode_head_block; /* kv heads one decode item covers: 1, or 4 / 2 (the largest that divides the
                                  pool's kv heads) when decode is confined to part of the GPU */
} ap_plan_info;
int ap_plan_get_info(const ap_plan *plan, ap_plan_info *info);

/*
 * Predicted time of a plan's kernels (App. B, "Roofline-Based Serve Cost").
 * *_bytes / *_flops: the algorithmic work of one attention layer -- every
 * attended KV token's K and V once per kv head, q read, out and lse written,
 * used block-table entries once, new K/V read and written once; 4 * head_dim
 * flop per (q head, query row, unmasked key).
 * roofline_*_us: the paper's operator model, Eq. "roofline":
 *   pi = min(F / A * B_g, F_g),  T_op = F / pi   (an operator without flops: A / B_g)
 * with B_g = hbm_gbs (GB/s) and F_g = tensor_tflops (TFLOP/s); a value <= 0
 * selects the figures measured on B200 (6448 GB/s copy bandwidth, 1642 TFLOP/s
 * dense bf16).
 * model_*_us: the cost model the planner itself uses, calibrated on B200 (per-SM
 * decode bandwidth, per-step and per-unit prefill cost, fixed costs);
 * model_step_us accounts for decode running beside prefill when the plan does.
 * Pure host arithmetic on the plan; works on host-only pools.
 */
typedef struct ap_plan_prediction {
    double decode_bytes, decode_flops, prefill_bytes, prefill_flops, append_bytes;
    double roofline_decode_us, roofline_prefill_us, roofline_append_us;
    double model_decode_us, model_prefill_us, model_step_us;
} ap_plan_prediction;
int ap_plan_predict(const ap_plan *plan, double hbm_gbs, double tensor_tflops, ap_plan_prediction *out);

/*
 * Host copy of the work lists a plan uploads, for inspection and tests.  The
 * blob is an int32 array; the layout gives the offset (in int32 units) of each
 * section:
 *   append_dst    [n_new]             page*16 + slot of every new token row
 *   bt_flat       [n_bt]              used block-table entries, sequences with q_len > 0 concatenated
 *   decode_items  [decode_items][8]   q_row, first kv_head of the item's block, bt_offset, page_begin, page_count, kv_len, part_slot, merge_index
 *   cta_begin     [n_cta_begin]       item range of decode CTA c is [cta_begin[c], cta_begin[c+1])
 *   merge_entries [merge_entries][4]  q_row, first kv_head of the block, part_begin, part_count
 *   prefill_tiles [prefill_tiles][8]  q_row0, rows, q_head, kv_head, bt_offset, pos0, ctx_len, q_head_b (-1: none)
 * blob: host, capacity_ints >= layout.total_ints, or NULL to query the layout only.
 */
typedef struct ap_plan_layout {
    int64_t total_ints, append_dst, bt_flat, decode_items, cta_begin, merge_entries, prefill_tiles;
    int64_t n_bt, n_cta_begin;
} ap_plan_layout;
int ap_plan_export(const ap_plan *plan, int32_t *blob, size_t capacity_ints, ap_plan_layout *layout);

/* --------------------------------------------------------------- kernels -- */

/*
 * KV page copy (Sec. 5.1, execution model, Phase 2 "Reconfiguration": moving
 * from one serving plan to the next migrates KV caches; the page is the unit
 * that moves).  For i in [0, n): page src_ids[i] of src_pool -- every kv head,
 * every slot, K and V -- is copied bit for bit to page dst_ids[i] of dst_pool.
 * The pools must have the same kv heads, head_dim and page size (else
 * INVALID_ARG) and live on the same device (else UNSUPPORTED: a move between
 * GPUs is the caller's peer copy); they may be the same pool (copy-on-write of
 * a shared prefix page).  dst_ids, src_ids: host, n entries each; they are read
 * before the call returns.  An id out of range -> BAD_BLOCK_TABLE; a
 * destination listed twice, or, inside one pool, a destination that is also
 * another pair's source -> INVALID_ARG (the copies run in parallel); a page
 * copied onto itself is skipped.  Nothing is queued when an error is
 * returned.  Neither pool's allocator state changes: allocate the destination
 * pages and free the source pages with the calls above.  Stream-ordered, no
 * host synchronisation: a following ap_kv_append / ap_attention_iteration on
 * the same stream sees the copied pages.  Host-only pools: validation only.
 */
int ap_kv_copy_pages(ap_kv_pool *dst_pool, const ap_kv_pool *src_pool, int32_t n, const int32_t *dst_ids,
                     const int32_t *src_ids, void *stream);

/*
 * KV append (App. B Eq. "serve-latency": every step extends the context).
 * Token t of sequence s sits at position p = ctx_len - q_len + t and is copied,
 * bit for bit, to K/V[block_table[s][p/16]][kv_head][p%16][:].
 * k_new, v_new: device, [N_new][num_kv_heads][head_dim] bf16, 16-byte aligned.
 */
int ap_kv_append(ap_kv_pool *pool, const ap_plan *plan, const void *k_new, const void *v_new,
                 void *stream);

/*
 * Attention for every new token of the batch (decode rows: split-K
 * flash-decoding, the LSE merge done by the last-arriving split; prefill
 * chunks: causal tiled attention on tcgen05 tensor cores).  The pool must
 * already hold the iteration's tokens.  Attention calls on the same pool must
 * not overlap on the GPU (they share the pool's merge arrival counters).
 * q, out: device, 16-byte aligned; lse: device or NULL; workspace: device,
 * 256-byte aligned, at least ap_plan_workspace_bytes() (else
 * WORKSPACE_TOO_SMALL), contents undefined before and after.
 */
int ap_attention_iteration(ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out,
                           float *lse, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Attention without any device-memory allocation.  (The paper has no
 * counterpart to this call; it exists for integration reasons only.)
 *
 * Who needs it: code that is not allowed to call cudaMalloc at the point where
 * attention runs -- a serving loop whose memory is entirely owned by a
 * framework's caching allocator (a raw cudaMalloc can then fail even though
 * memory is "free"), a latency-critical path that cannot take cudaMalloc's
 * device-wide synchronisation, or a plug-in that is handed tensors but no
 * allocator.  Such callers have nowhere to get the split-K workspace that
 * ap_attention_iteration asks for.
 *
 * This variant does the same work as ap_attention_iteration but keeps the
 * split-K partials in a fixed array of AP_STATIC_WORKSPACE_BYTES (8 MiB) that
 * is part of the library image: every GPU context that loads the library
 * holds those 8 MiB until the process exits, used or not.  The call itself
 * performs no cudaMalloc / cudaFree and calls no allocating routine; q, out
 * and lse are still the caller's.  (Building the plan is a separate, earlier
 * call; ap_plan_create recycles its upload buffers and only allocates when it
 * needs a larger one than it has seen before.)
 *
 *  - A plan whose ap_plan_workspace_bytes() exceeds AP_STATIC_WORKSPACE_BYTES
 *    is rejected with AP_ERR_WORKSPACE_TOO_SMALL before anything is launched
 *    (A plan needs at most 2 partials per decode CTA, each head_dim + 1 floats for
 *    every query head of a block of up to 4 kv heads: 4.9 MB on 148 SMs at
 *    head_dim 128 with 8 query heads per kv head, whatever the context lengths.)
 *  - The array's device address is looked up once per device when a pool is
 *    created on it (ap_kv_pool_create, which allocates anyway and must not run
 *    inside a stream capture); that is also when the runtime brings the array
 *    into being on the device.  The call here only reads the cached address.
 *  - All calls on a device share the one array, and it keeps whatever the last
 *    call left in it.  Nothing has to start at zero: every partial is written
 *    in full before it is read within the same call.  Two calls that overlap
 *    on the GPU (different streams, no ordering between them) race on the
 *    array and produce garbage; order them, or use ap_attention_iteration with
 *    separate workspaces.
 */
#define AP_STATIC_WORKSPACE_BYTES (8u << 20)
size_t ap_static_workspace_bytes(void);
int ap_attention_iteration_static(ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out,
                                  float *lse, void *stream);

/*
 * The whole iteration from HOST buffers: plan, host->device copies of q,
 * k_new, v_new, append, attention, device->host copy of out (and lse if not
 * NULL), and a stream synchronisation.  Staging buffers belong to the pool and
 * grow on demand.  q_host ... lse_host: host (pinned memory makes the copies
 * asynchronous).  Returns the device status after the sync.
 */
int ap_serving_iteration_host(ap_kv_pool *pool, const ap_batch_desc *batch, const void *q_host,
                              const void *k_new_host, const void *v_new_host, void *out_host,
                              float *lse_host, void *stream);

/* Synchronises `stream` and returns (and clears) the device status word:
 * AP_OK, AP_ERR_BAD_BLOCK_TABLE (a kernel met an out-of-range page id) or
 * AP_ERR_TIMEOUT (a bounded wait inside a kernel ran out).  After an error it
 * also clears the split-K arrival counters, which a kernel that gave up may
 * have left raised, so the pool can be used again. */
int ap_last_device_status(ap_kv_pool *pool, void *stream);

const char *ap_status_string(int status);

/*
 * Bound of every wait inside the kernels (failure detection: Sec. 5.1 counts a
 * stalled or failed serving plan as stale time, so a kernel must end and report
 * rather than hang).  Every mbarrier wait in the attention kernels gives up
 * after limit_ns nanoseconds on the GPU's global timer, records AP_ERR_TIMEOUT
 * in the pool's status word and lets the kernel return; outputs of that launch
 * are then undefined.  Default 2 s; limit_ns = 0 restores it.  Applies to
 * launches made afterwards.
 */
int ap_kv_pool_set_wait_limit(ap_kv_pool *pool, uint64_t limit_ns);

/*
 * Self-test of that error path: queues a one-warp kernel on `stream` that
 * waits, through the same bounded-wait routine the attention kernels use, on a
 * barrier nothing ever arrives on.  It ends by itself after limit_ns
 * (0 < limit_ns <= 2 s, else INVALID_ARG) and leaves AP_ERR_TIMEOUT in the
 * pool's status word, which the next ap_last_device_status returns and clears.
 * With leave_counter != 0 it also leaves one split-K arrival counter raised, as
 * an attention kernel that gave up mid-stream would; ap_last_device_status
 * clears those too.  The GPU context stays usable.
 */
int ap_selftest_wait_timeout(ap_kv_pool *pool, uint64_t limit_ns, int leave_counter, void *stream);

/* ----------------------------------------------------------- diagnostics -- */

/*
 * Per-kernel device timing for benchmarks.  While enabled, every kernel the
 * library launches for this pool is bracketed by CUDA events recorded on the
 * launching stream.  ap_profile_collect synchronises `stream`, adds up the
 * elapsed times per kernel since the last enable/collect, and clears the
 * records.  Index: 0 kv_append, 1 decode split-K (which also performs the LSE
 * merge), 2 prefill, 3 the single launch that holds both parts of a mixed plan.
 */
enum { AP_KERNEL_APPEND = 0, AP_KERNEL_DECODE = 1, AP_KERNEL_PREFILL = 2, AP_KERNEL_MIXED = 3, AP_KERNEL_COUNT = 4 };
typedef struct ap_kernel_times {
    double ms[AP_KERNEL_COUNT];
    int64_t launches[AP_KERNEL_COUNT];
} ap_kernel_times;
int ap_profile_enable(ap_kv_pool *pool, int on);
int ap_profile_collect(ap_kv_pool *pool, void *stream, ap_kernel_times *out);

#ifdef __cplusplus
}
#endif
#endif /* AP_SERVING_H */
