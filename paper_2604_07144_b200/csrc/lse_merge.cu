// LSE merge of split-K partials: for every (decode row, kv head) whose key
// range was cut into several work items,
//     lse = m* + ln sum_k exp(lse_k - m*),   o = sum_k exp(lse_k - lse) o_k,
// with m* = max_k lse_k; o is rounded to bf16 once, here.  Small and HBM-bound.
#include <cuda_bf16.h>

#include "internal.h"

namespace ap {

namespace {

// One CTA per merge entry; thread i handles columns of the G x D result.
__global__ void __launch_bounds__(128) lse_merge_kernel(const MergeEntry *__restrict__ entries,
                                                        const float *__restrict__ o_part,
                                                        const float *__restrict__ lse_part,
                                                        __nv_bfloat16 *__restrict__ out, float *__restrict__ lse_out,
                                                        int Hq, int G, int D) {
    const MergeEntry e = entries[blockIdx.x];
    for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
        const int head = idx / D, col = idx % D;
        float mstar = -INFINITY;
        for (int k = 0; k < e.part_count; ++k)
            mstar = fmaxf(mstar, __ldg(lse_part + (size_t)(e.part_begin + k) * G + head));
        float sum = 0.f, acc = 0.f;
        for (int k = 0; k < e.part_count; ++k) {
            const size_t row = (size_t)(e.part_begin + k) * G + head;
            const float w = __expf(__ldg(lse_part + row) - mstar);
            sum += w;
            acc += w * __ldg(o_part + row * D + col);
        }
        const size_t orow = (size_t)e.q_row * Hq + (size_t)e.kv_head * G + head;
        out[orow * D + col] = __float2bfloat16_rn(acc / sum);
        if (col == 0 && lse_out) lse_out[orow] = mstar + __logf(sum);
    }
}

}  // namespace

cudaError_t launch_lse_merge(const ap_kv_pool *pool, const ap_plan *plan, const float *o_part,
                             const float *lse_part, void *out, float *lse, cudaStream_t stream) {
    lse_merge_kernel<<<(unsigned)plan->info.merge_entries, 128, 0, stream>>>(
        plan->d_merge, o_part, lse_part, (__nv_bfloat16 *)out, lse, plan->num_q_heads, plan->group,
        pool->desc.head_dim);
    return cudaGetLastError();
}

}  // namespace ap
