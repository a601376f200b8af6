// Helpers shared by the kernels that write a read plan.
#pragma once

#include "common.cuh"

namespace santapp {

// Writes the plan's suffix segment (if any) and the pair totals. One thread.
__device__ inline void finish_plan(const SelectParams &p, int pair, int b, int nseg, int prompt_rows)
{
    const int cap = p.plan.seg_cap;
    int32_t *seg_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
    int t = 0;
    if (p.suffix_len != nullptr && p.suffix_cap > 0) t = max(0, min(p.suffix_len[b], p.suffix_cap));
    int total = prompt_rows;
    if (t > 0) {
        p.plan.seg_row[(size_t)pair * cap + nseg] = pair * p.suffix_cap;     // pair = b * n_kv + j
        p.plan.seg_mask[(size_t)pair * cap + nseg] = ((1u << p.bv.group) - 1u) | kSrcSuffix;
        for (int h = 0; h < kMaxGroup; ++h)
            p.plan.seg_logc[((size_t)pair * cap + nseg) * kMaxGroup + h] = 0.f;
        seg_prefix[nseg] = total;
        total += t;
        ++nseg;
    }
    seg_prefix[nseg] = total;
    p.plan.pair_nseg[pair] = nseg;
    p.plan.pair_rows[pair] = total;
    p.plan.pair_union_rows[pair] = prompt_rows;
    if (p.dbg_union_rows) p.dbg_union_rows[pair] = prompt_rows;
}

// The last pair to finish turns pair_rows into the global exclusive prefix. All threads call.
__device__ inline void publish_pair_prefix(const SelectParams &p, int *flag_smem, int *scan_smem /* [33] */)
{
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *flag_smem = (atomicAdd(p.ctl.plan_ticket, 1) == p.n_pairs - 1);
    __syncthreads();
    if (!*flag_smem) return;
    __threadfence();
    if (threadIdx.x == 0) *p.ctl.plan_ticket = 0;                  // every pair has arrived
    int64_t carry = 0;
    for (int base = 0; base < p.n_pairs; base += (int)blockDim.x) {
        const int i = base + (int)threadIdx.x;
        const int v = i < p.n_pairs ? __ldcg(p.plan.pair_rows + i) : 0;
        int total;
        const int excl = block_exclusive_scan(v, scan_smem, total);
        if (i < p.n_pairs) p.plan.pair_row_prefix[i] = carry + excl;
        carry += total;
    }
    if (threadIdx.x == 0) p.plan.pair_row_prefix[p.n_pairs] = carry;
}

}  // namespace santapp
