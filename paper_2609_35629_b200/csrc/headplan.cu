// Sampling kernel: one block per (sequence, query head) runs select_head (headplan.cuh).
#include "common.cuh"
#include "headplan.cuh"

namespace santapp {

namespace {

// Few heads: 512 threads each, so that every per-thread loop is short (the kernel is a chain of
// dependent steps, not a throughput problem); many heads: 128 threads and more resident blocks.
template <int kHeadThreads, bool kHalf>
__global__ void __launch_bounds__(kHeadThreads, 512 / kHeadThreads)
headplan_kernel(PlanInputs in)
{
    __shared__ HeadSmem sm;
    trace_mark(in.trace, 1, 0);
    select_head<kHeadThreads, kHeadThreads >= 512 ? 4 : 8, kHalf>(in, blockIdx.x, sm);
    trace_mark(in.trace, 1, 1);
}

}  // namespace

cudaError_t launch_headplan(const PlanInputs &in, cudaStream_t s)
{
    const int n_heads = in.bv.n_seqs * in.bv.n_q;
    const bool wide = n_heads <= attend_grid_size();
    if (in.bv.elem) {
        if (wide) return launch_kernel(headplan_kernel<512, true>, dim3(n_heads), dim3(512), 0, s, in);
        return launch_kernel(headplan_kernel<128, true>, dim3(n_heads), dim3(128), 0, s, in);
    }
    if (wide) return launch_kernel(headplan_kernel<512, false>, dim3(n_heads), dim3(512), 0, s, in);
    return launch_kernel(headplan_kernel<128, false>, dim3(n_heads), dim3(128), 0, s, in);
}

}  // namespace santapp
