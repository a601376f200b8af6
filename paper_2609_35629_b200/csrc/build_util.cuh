// Helpers shared by the team builders: block-wide arg-min / arg-max with the paper's index
// tie-break ("Shared team construction": ties go to the smaller token index).
#pragma once
#include <cuda_runtime.h>

namespace santapp {

struct ValIdx {
    double v;
    int i;
};

template <bool kMin>
__device__ __forceinline__ ValIdx pick(const ValIdx &a, const ValIdx &b)
{
    bool take_b;
    if (kMin) take_b = (b.v < a.v) || (b.v == a.v && b.i < a.i);
    else      take_b = (b.v > a.v) || (b.v == a.v && b.i < a.i);
    return take_b ? b : a;
}

// Block-wide arg-min / arg-max; ties go to the smaller index. Result valid in every thread.
template <bool kMin>
__device__ ValIdx block_arg(ValIdx x, ValIdx *scratch /* [33] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ValIdx y;
        y.v = __shfl_xor_sync(0xFFFFFFFFu, x.v, o);
        y.i = __shfl_xor_sync(0xFFFFFFFFu, x.i, o);
        x = pick<kMin>(x, y);
    }
    __syncthreads();
    if (lane == 0) scratch[warp] = x;
    __syncthreads();
    if (warp == 0) {
        ValIdx y = scratch[lane < n_warps ? lane : 0];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ValIdx z;
            z.v = __shfl_xor_sync(0xFFFFFFFFu, y.v, o);
            z.i = __shfl_xor_sync(0xFFFFFFFFu, y.i, o);
            y = pick<kMin>(y, z);
        }
        if (lane == 0) scratch[32] = y;
    }
    __syncthreads();
    return scratch[32];
}

}  // namespace santapp
