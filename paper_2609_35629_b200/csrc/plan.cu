// Read plans in global memory, for the attention kernel's equal-range split:
//   plan_kernel        one block per (sequence, KV head) pair: union of the heads' samples
//                      (pairplan.cuh), copied out to the workspace; the last block to finish turns
//                      the pairs' row counts into the global row prefix.
//   dense_plan_kernel  the trivial plan that reads every prompt row and the suffix.
#include "common.cuh"
#include "pairplan.cuh"

namespace santapp {

namespace {

// The last block to finish turns pair_rows into the global exclusive prefix. All threads call.
__device__ void publish_pair_prefix(const PlanParams &p, int *flag_smem, int *scan_smem /* [33] */)
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

template <int G>
struct PlanKernelSmem {
    PlanScratch scratch;
    int seg_prefix[kSegMax + 3];
    int seg_row[kSegMax + 3];
    uint32_t seg_mask[kSegMax + 3];
    int flag;
};

template <int G>
__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(PlanParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    PlanKernelSmem<G> &sm = *reinterpret_cast<PlanKernelSmem<G> *>(smem_raw);
    const int pair = blockIdx.x, tid = threadIdx.x;
    const int cap = p.plan.seg_cap;
    int nseg, rows;
    build_pair_plan<G>(p.in, pair, sm.scratch, sm.seg_prefix, sm.seg_row, sm.seg_mask,
                       p.plan.seg_logc + (size_t)pair * cap * kMaxGroup, nseg, rows, true);
    int32_t *g_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
    int32_t *g_row = p.plan.seg_row + (size_t)pair * cap;
    uint32_t *g_mask = p.plan.seg_mask + (size_t)pair * cap;
    for (int i = tid; i <= nseg; i += kPlanThreads) g_prefix[i] = sm.seg_prefix[i];
    for (int i = tid; i < nseg; i += kPlanThreads) { g_row[i] = sm.seg_row[i]; g_mask[i] = sm.seg_mask[i]; }
    if (tid == 0) { p.plan.pair_nseg[pair] = nseg; p.plan.pair_rows[pair] = rows; }
    publish_pair_prefix(p, &sm.flag, sm.scratch.scan);
}

// One block; a thread per pair.
__global__ void dense_plan_kernel(PlanParams p)
{
    __shared__ int flag;
    __shared__ int scan[33];
    const uint32_t all_heads = (1u << p.in.bv.group) - 1u;
    for (int pair = threadIdx.x; pair < p.n_pairs; pair += blockDim.x) {
        const int b = pair / p.in.bv.n_kv;
        p.ctl.attend_ticket[pair] = 0;
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
    if (threadIdx.x == 0) *p.ctl.plan_ticket = p.n_pairs - 1;    // this block is the last arrival
    __syncthreads();
    publish_pair_prefix(p, &flag, scan);
}

template <int G>
cudaError_t launch_plan_g(const PlanParams &p, cudaStream_t s)
{
    const size_t smem = sizeof(PlanKernelSmem<G>);
    static std::atomic<unsigned long long> done;
    cudaError_t err = ensure_dynamic_smem((const void *)plan_kernel<G>, (int)smem, done);
    if (err != cudaSuccess) return err;
    plan_kernel<G><<<p.n_pairs, kPlanThreads, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_plan(const PlanParams &p, cudaStream_t s)
{
    switch (p.in.bv.group) {
        case 1: return launch_plan_g<1>(p, s);
        case 2: return launch_plan_g<2>(p, s);
        case 3: return launch_plan_g<3>(p, s);
        case 4: return launch_plan_g<4>(p, s);
        case 5: return launch_plan_g<5>(p, s);
        case 6: return launch_plan_g<6>(p, s);
        case 7: return launch_plan_g<7>(p, s);
        case 8: return launch_plan_g<8>(p, s);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_dense_plan(const PlanParams &p, cudaStream_t s)
{
    dense_plan_kernel<<<1, 256, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace santapp
