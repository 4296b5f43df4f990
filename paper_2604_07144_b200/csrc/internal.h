// Internal declarations shared by the host code and the kernels of the
// serving-iteration library.  Not part of the public ABI.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

#include "ap_serving.h"

namespace ap {

constexpr int kPageSize = 16;
constexpr uint64_t kDefaultWaitLimitNs = 2000000000ull;   // 2 s
constexpr int kMaxMergeEntries = 4096;   // arrival counters kept per pool (the planner makes < 2 per CTA)

// ---- device work lists (all int32, uploaded as one blob per plan) ---------

// One split-K decode work item: the query heads of one block of kv heads (HB consecutive kv heads,
// HB = decode_head_block(Hkv), i.e. HB * G query heads) of one decode row over a contiguous range of
// that sequence's logical pages.  The HB (page, kv head) tiles of a page lie next to one another in a
// pool plane, so a page costs the decode kernel one TMA request of HB tiles per plane.
struct DecodeItem {
    int32_t q_row;       // row in q / out
    int32_t kv_head;     // first kv head of the block
    int32_t bt_offset;   // offset of the sequence's first block-table entry in bt_flat
    int32_t page_begin;  // first logical page of the range
    int32_t page_count;  // pages in the range (>= 1)
    int32_t kv_len;      // attended length of the row (position + 1)
    int32_t part_slot;   // slot in the partial buffers, or -1: write out/lse directly
    int32_t merge_index; // entry in the merge list this partial belongs to, or -1
};
static_assert(sizeof(DecodeItem) == 32, "DecodeItem layout");

// One (row, kv head block) result assembled from several partials.
struct MergeEntry {
    int32_t q_row;
    int32_t kv_head;     // first kv head of the block
    int32_t part_begin;
    int32_t part_count;
};

// One prefill work unit: 128 consecutive query rows of one sequence for two
// q heads of the same kv head (or one, when the group has an odd head left),
// over all keys up to the last row's position.
struct PrefillTile {
    int32_t q_row0;      // global row of the tile's first query
    int32_t rows;        // valid rows in the tile (1..128)
    int32_t q_head;
    int32_t kv_head;
    int32_t bt_offset;
    int32_t pos0;        // position of the first query row in its sequence
    int32_t ctx_len;     // sequence context length (positions >= ctx_len hold no token)
    int32_t q_head_b;    // second q head of the same kv head sharing the K/V stream, or -1
};
static_assert(sizeof(PrefillTile) == 32, "PrefillTile layout");

// Partial buffers inside the caller's workspace: o_part [slots][HB * G][d] fp32
// followed by lse_part [slots][HB * G] fp32.
struct WorkspaceLayout {
    size_t o_part_off = 0;
    size_t lse_part_off = 0;
    size_t bytes = 0;
};

// ---- host objects ----------------------------------------------------------

struct PlanBuffer {            // reusable staging for one plan upload
    int32_t *host = nullptr;   // pinned
    int32_t *dev = nullptr;
    size_t capacity = 0;       // int32 elements
    cudaEvent_t uploaded = nullptr;
};

struct PlanWork {              // algorithmic work of a plan (one attention layer), for ap_plan_predict
    double decode_bytes = 0, decode_flops = 0, prefill_bytes = 0, prefill_flops = 0, append_bytes = 0;
    double prefill_sm_us = 0;  // SM-time of the prefill units by the planner's cost model
};

struct TimedLaunch {
    int kernel;
    cudaEvent_t start, stop;
};

}  // namespace ap

struct ap_kv_pool {
    ap_pool_desc desc{};
    bool owns_planes = false;
    int sm_count = 0;
    int *h_status = nullptr;          // the status word: pinned host memory mapped into the device's address space
    int *status_dev = nullptr;        // ... and the address the kernels write it at
    int *d_counters = nullptr;        // device: arrival counters of the merge entries
    uint64_t wait_limit_ns = ap::kDefaultWaitLimitNs;   // bound of every wait inside a kernel
    CUtensorMap k_map{}, v_map{};          // box = one (page, kv head) tile (prefill)
    CUtensorMap k_map_blk{}, v_map_blk{};  // box = the head_block tiles of a page that lie together (decode)
    int head_block = 1;                    // HB: kv heads per decode item
    // allocator
    std::vector<int32_t> free_list;     // pages handed out from the back
    std::vector<uint8_t> allocated;     // per page
    // recycled plan staging
    std::vector<ap::PlanBuffer> plan_buffers;
    // staging for ap_serving_iteration_host
    void *stage_dev = nullptr;
    size_t stage_bytes = 0;
    // Side-by-side execution of mixed iterations: a low-priority second stream for the prefill
    // kernel and the fork / join events that tie it to the caller's stream.
    cudaStream_t side_stream = nullptr;
    cudaEvent_t fork_event = nullptr, join_event = nullptr;
    int side_by_side_mode = 1;        // 0 never, 1 decided per plan, >= 2 that many decode CTAs
    bool single_launch = true;        // side-by-side plans: one launch for both parts (else two streams)
    // per-kernel event timing (diagnostics)
    bool profiling = false;
    std::vector<ap::TimedLaunch> timed;
    std::vector<cudaEvent_t> spare_events;
};

struct ap_plan {
    ap_kv_pool *pool = nullptr;
    ap::PlanBuffer buf{};
    int num_q_heads = 0;
    int group = 0;               // G = Hq / Hkv
    int head_block = 1;          // HB: kv heads per decode item of this plan (1, or the pool's head_block)
    float scale = 0.f;
    ap_plan_info info{};
    ap_plan_layout layout{};
    std::vector<int32_t> blob;   // host copy of the uploaded work lists
    int n_part_slots = 0;
    ap::PlanWork work{};
    bool side_by_side = false;   // decode confined to part of the GPU, prefill on the rest at the same time
    bool single_launch = false;  // ... and both in one launch (else: two kernels on two streams)
    ap::WorkspaceLayout ws{};
    // device pointers into buf.dev
    const int32_t *d_append_dst = nullptr;
    const int32_t *d_bt_flat = nullptr;
    const ap::DecodeItem *d_items = nullptr;
    const int32_t *d_cta_begin = nullptr;
    const ap::MergeEntry *d_merge = nullptr;
    const ap::PrefillTile *d_tiles = nullptr;
};

namespace ap {

// Kernel launchers (each returns a cudaError_t from the launch).
cudaError_t launch_kv_append(const ap_kv_pool *pool, const ap_plan *plan, const void *k_new,
                             const void *v_new, cudaStream_t stream);
cudaError_t launch_decode_splitk(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out,
                                 float *lse, float *o_part, float *lse_part, cudaStream_t stream);
cudaError_t launch_prefill(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out,
                           float *lse, cudaStream_t stream);
// Both parts of a mixed plan in one launch: the plan's decode CTAs first, then one block per prefill unit.
cudaError_t launch_mixed_iteration(const ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                                   float *o_part, float *lse_part, cudaStream_t stream);
// Decode and prefill kernels of a plan: one after the other on `stream`, or, for a side-by-side plan,
// both in one launch (or, if the pool asks for it, decode on `stream` and prefill on the pool's second
// stream, joined back into `stream`).
cudaError_t launch_attention_kernels(ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                                     float *o_part, float *lse_part, cudaStream_t stream);
// One warp waits on an mbarrier that nothing arrives on, with the given limit (see ap_selftest_wait_timeout).
cudaError_t launch_selftest_wait(const ap_kv_pool *pool, uint64_t limit_ns, int leave_counter, cudaStream_t stream);
// d_pairs: device [n_pairs][2] = (destination page, source page)
cudaError_t launch_kv_copy_pages(const ap_kv_pool *dst_pool, const ap_kv_pool *src_pool, const int32_t *d_pairs,
                                 int n_pairs, cudaStream_t stream);

// Launch with programmatic stream serialization: the kernel may begin (up to its griddep_wait)
// before the previous kernel in the stream has drained, which hides launch latency and preamble.
// Every kernel launched this way touches data written by earlier work only after griddep_wait.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                                     cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Per-device set-up of the library's fixed split-K scratch array (static_workspace.cu).
int prepare_static_workspace(int device);

// Decode kernel launch geometry (used by the planner to size the item lists).
int decode_ctas_per_sm(int head_dim);
constexpr int kDecodeTilesPerStage = 4;    // (page, kv head) tiles of one plane in a ring stage: one per warp of a consumer group
// kv heads per decode item: the largest of 4, 2, 1 that divides the number of kv heads.  A stage then holds
// kDecodeTilesPerStage / HB pages of HB heads each.
inline int decode_head_block(int num_kv_heads) {
    return num_kv_heads % 4 == 0 ? 4 : num_kv_heads % 2 == 0 ? 2 : 1;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no libcuda link).
int encode_pool_tensor_map(CUtensorMap *map, void *base, int num_pages, int num_kv_heads, int head_dim,
                           int tiles_per_box);
int encode_q_tensor_map(CUtensorMap *map, const void *q, int64_t n_rows, int num_q_heads, int head_dim);

}  // namespace ap
