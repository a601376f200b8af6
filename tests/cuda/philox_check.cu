// Test-only kernel: for a list of (counter, key) pairs, evaluate the library's Philox4x32-10
// device function and cuRAND's header-only curand_Philox4x32_10, side by side. The Python test
// compares both with the CPU oracle's words. Not part of the product library.
#include <cuda_runtime.h>
#include <curand_kernel.h>
#include <curand_philox4x32_x.h>
#include <stdint.h>

#include "common.cuh"

__global__ void philox_both(const uint32_t *ctr_key /* [n][6] */, int n, uint32_t *mine /* [n][4] */,
                            uint32_t *theirs /* [n][4] */, double *gumbel /* [n][4] */)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint32_t *c = ctr_key + 6 * i;
    const uint4 a = santapp::philox4x32_10(make_uint4(c[0], c[1], c[2], c[3]), c[4], c[5]);
    const uint4 b = curand_Philox4x32_10(make_uint4(c[0], c[1], c[2], c[3]), make_uint2(c[4], c[5]));
    mine[4 * i + 0] = a.x; mine[4 * i + 1] = a.y; mine[4 * i + 2] = a.z; mine[4 * i + 3] = a.w;
    theirs[4 * i + 0] = b.x; theirs[4 * i + 1] = b.y; theirs[4 * i + 2] = b.z; theirs[4 * i + 3] = b.w;
    gumbel[4 * i + 0] = santapp::gumbel_from_word(a.x);
    gumbel[4 * i + 1] = santapp::gumbel_from_word(a.y);
    gumbel[4 * i + 2] = santapp::gumbel_from_word(a.z);
    gumbel[4 * i + 3] = santapp::gumbel_from_word(a.w);
}

extern "C" int philox_check_run(const uint32_t *ctr_key_dev, int n, uint32_t *mine_dev, uint32_t *theirs_dev,
                                double *gumbel_dev)
{
    philox_both<<<(n + 127) / 128, 128>>>(ctr_key_dev, n, mine_dev, theirs_dev, gumbel_dev);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return (int)err;
    return (int)cudaDeviceSynchronize();
}
