// Sampling kernel: one block per (sequence, query head) runs select_head (headplan.cuh).
#include "common.cuh"
#include "headplan.cuh"

namespace santapp {

namespace {

// Few heads: 512 threads each, so that every per-thread loop is short (the kernel is a chain of
// dependent steps, not a throughput problem); more heads: 256 threads and four resident blocks per
// SM, then 128 threads and eight.
template <int kHeadThreads, bool kHalf>
__global__ void __launch_bounds__(kHeadThreads, kHeadThreads >= 512 ? 1 : 1024 / kHeadThreads)
headplan_kernel(PlanInputs in)
{
    __shared__ HeadSmem sm;
    trace_mark(in.trace, 1, 0);
    select_head<kHeadThreads, kHeadThreads >= 512 ? 4 : 2, kHalf>(in, blockIdx.x, sm);
    trace_mark(in.trace, 1, 1);
}

}  // namespace

cudaError_t launch_headplan(const PlanInputs &in, cudaStream_t s)
{
    const int n_heads = in.bv.n_seqs * in.bv.n_q;
    const int sms = attend_grid_size();
    if (in.bv.elem) {
        if (n_heads <= sms) return launch_kernel(headplan_kernel<512, true>, dim3(n_heads), dim3(512), 0, s, in);
        if (n_heads <= 4 * sms) return launch_kernel(headplan_kernel<256, true>, dim3(n_heads), dim3(256), 0, s, in);
        return launch_kernel(headplan_kernel<128, true>, dim3(n_heads), dim3(128), 0, s, in);
    }
    if (n_heads <= sms) return launch_kernel(headplan_kernel<512, false>, dim3(n_heads), dim3(512), 0, s, in);
    if (n_heads <= 4 * sms) return launch_kernel(headplan_kernel<256, false>, dim3(n_heads), dim3(256), 0, s, in);
    return launch_kernel(headplan_kernel<128, false>, dim3(n_heads), dim3(128), 0, s, in);
}

}  // namespace santapp
