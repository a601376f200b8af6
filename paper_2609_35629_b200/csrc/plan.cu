// Read plans in global memory, for the attention kernel's equal-range split:
//   plan_kernel         one block per (sequence, KV head) pair: union of the heads' samples
//                       (pairplan.cuh), copied out to the workspace with the pair's row count.
//   dense_plan_kernel   the trivial plan that reads every prompt row and the suffix.
//   pair_prefix_kernel  the pairs' row counts as one exclusive prefix, for batches of more pairs
//                       than the attention kernel stages (and sums) by itself.
#include "common.cuh"
#include "pairplan.cuh"

namespace santapp {

namespace {

constexpr int kPlanThreads = 256;

struct PlanKernelSmem {
    PlanScratch scratch;
    int seg_prefix[kSegMax + 3];
    int seg_row[kSegMax + 3];
    uint32_t seg_mask[kSegMax + 3];
};

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(PlanParams p, int max_words)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    PlanKernelSmem &sm = *reinterpret_cast<PlanKernelSmem *>(smem_raw);
    const int pair = blockIdx.x, tid = threadIdx.x;
    const int cap = p.plan.seg_cap;
    trace_mark(p.in.trace, 2, 0);
    int nseg, rows;
    build_pair_plan<kPlanThreads>(p.in, pair, max_words, sm.scratch, sm.seg_prefix, sm.seg_row, sm.seg_mask,
                                  p.plan.seg_logc + (size_t)pair * cap * kMaxGroup, nseg, rows, true);
    int32_t *g_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
    int32_t *g_row = p.plan.seg_row + (size_t)pair * cap;
    uint32_t *g_mask = p.plan.seg_mask + (size_t)pair * cap;
    for (int i = tid; i <= nseg; i += kPlanThreads) g_prefix[i] = sm.seg_prefix[i];
    for (int i = tid; i < nseg; i += kPlanThreads) { g_row[i] = sm.seg_row[i]; g_mask[i] = sm.seg_mask[i]; }
    if (tid == 0) { p.plan.pair_nseg[pair] = nseg; p.plan.pair_rows[pair] = rows; }
    if (pair == 0 && tid < 2) p.plan.tail_counter[tid] = 0;
    trace_mark(p.in.trace, 2, 1);
}

// A thread per pair.
__global__ void __launch_bounds__(256)
dense_plan_kernel(PlanParams p)
{
    const uint32_t all_heads = (1u << p.in.bv.group) - 1u;
    const int pair = blockIdx.x * blockDim.x + threadIdx.x;
    if (pair < 2) p.plan.tail_counter[pair] = 0;
    if (pair >= p.n_pairs) return;
    const int b = pair / p.in.bv.n_kv;
    const int cap = p.plan.seg_cap;
    const int64_t row0 = p.in.bv.seq_row_off[b];
    const int N = (int)(p.in.bv.seq_row_off[b + 1] - row0);
    int t = 0;
    if (p.in.suffix_len != nullptr && p.in.suffix_cap > 0) t = max(0, min(p.in.suffix_len[b], p.in.suffix_cap));
    int32_t *g_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
    p.plan.seg_row[(size_t)pair * cap] = (int32_t)row0;
    p.plan.seg_mask[(size_t)pair * cap] = all_heads;
    g_prefix[0] = 0;
    int nseg = 1, rows = N;
    if (t > 0) {
        g_prefix[1] = rows;
        p.plan.seg_row[(size_t)pair * cap + 1] = pair * p.in.suffix_cap;
        p.plan.seg_mask[(size_t)pair * cap + 1] = all_heads | kSrcSuffix;
        rows += t;
        nseg = 2;
    }
    g_prefix[nseg] = rows;
    for (int h = 0; h < 2 * kMaxGroup; ++h) p.plan.seg_logc[(size_t)pair * cap * kMaxGroup + h] = 0.f;
    p.plan.pair_nseg[pair] = nseg;
    p.plan.pair_rows[pair] = rows;
}

// One block: pair_row_prefix[i] = rows of the pairs before pair i, i = 0 .. n_pairs.
__global__ void __launch_bounds__(1024)
pair_prefix_kernel(PlanView plan, int n_pairs)
{
    __shared__ int scan[33];
    int64_t carry = 0;
    for (int base = 0; base < n_pairs; base += (int)blockDim.x) {
        const int i = base + (int)threadIdx.x;
        const int v = i < n_pairs ? plan.pair_rows[i] : 0;
        int total;
        const int excl = block_exclusive_scan(v, scan, total);
        if (i < n_pairs) plan.pair_row_prefix[i] = carry + excl;
        carry += total;
    }
    if (threadIdx.x == 0) plan.pair_row_prefix[n_pairs] = carry;
}

}  // namespace

cudaError_t launch_plan(const PlanParams &p, int max_teams_per_seq, cudaStream_t s)
{
    const size_t smem = sizeof(PlanKernelSmem);
    static std::atomic<unsigned long long> done;
    cudaError_t err = ensure_dynamic_smem((const void *)plan_kernel, (int)smem, done);
    if (err != cudaSuccess) return err;
    return launch_kernel(plan_kernel, dim3(p.n_pairs), dim3(kPlanThreads), smem, s, p, (max_teams_per_seq + 31) / 32);
}

cudaError_t launch_dense_plan(const PlanParams &p, cudaStream_t s)
{
    return launch_kernel(dense_plan_kernel, dim3((p.n_pairs + 255) / 256), dim3(256), 0, s, p);
}

cudaError_t launch_pair_prefix(const PlanParams &p, cudaStream_t s)
{
    return launch_kernel(pair_prefix_kernel, dim3(1), dim3(1024), 0, s, p.plan, p.n_pairs);
}

}  // namespace santapp
