// Representative scoring of one tile of 16 teams for the GQA group of a KV head (Algorithm 1,
// routing logits and their Gumbel perturbation), in fp32 on tensor cores:
//   Y32_{h,g} = log n_g + q_h . l_g * scale + G_{h,g}          (Eq. method-routing plus noise)
// Device functions shared by the stand-alone scoring kernels (score.cu) and the single-launch
// decode kernel (attend.cu). These scores only choose which teams are re-evaluated exactly; the
// sample itself is decided in fp64 (headplan.cuh).
//
// The GQA group is the M tile of S^T = q K^T (mma.sync m16n8k16, 16-bit inputs, fp32
// accumulation). A lane feeds the tensor core 16-byte pieces of the representative keys exactly
// as they lie in memory: the contraction index is permuted consistently on both operands, so
// no transpose is needed.
#pragma once

#include "common.cuh"

namespace santapp {

constexpr int kScoreTeamsPerWarp = 16;

// Where the scores go and which random stream perturbs them.
struct ScoreCtx {
    float *y32;                     // [n_q][n_seqs][y_stride]
    int64_t y_stride;
    int n_q, n_seqs;
    const uint16_t *q;              // [n_seqs][n_q][128]
    uint32_t seed_lo, seed_hi, stream_base;
};

template <bool kHalf>
__device__ __forceinline__ void mma_score(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    // A rows 8..15 are zero (a1 = a3 = 0): only heads 0..7 exist
    if constexpr (kHalf)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// Gumbel(0,1) in fp32 from a 32-bit word: u = (x + 0.5) / 2^32, G = -log(-log u), to an absolute
// error well inside the additive term of the guard (score_guard in headplan.cuh).
// Lower half of the range (u <= 1/2): -log u >= 0.69 from the fast logarithm (3 ulp there).
// Upper half: u = 1 - z with z = (2^32 - x - 0.5) / 2^32 in (0, 1/2]; -log(1 - z) from four series
// terms when z < 2^-6 (relative truncation z^4 / 5 < 1.2e-8), else from the fast logarithm, whose
// absolute error 2^-21.4 is then below 2.3e-5 of the result. The outer logarithm sees values in
// (1e-10, 23) where the fast logarithm is accurate to 3 ulp or 2^-21.4 absolute.
__device__ __forceinline__ float gumbel32_from_word(uint32_t x)
{
    // straight-line: both halves are evaluated and one is selected, so lanes never diverge
    const bool upper = x >= 0x80000000u;
    const float u = ((float)x + 0.5f) * 2.3283064365386963e-10f;
    const float z = ((float)(~x) + 0.5f) * 2.3283064365386963e-10f;      // 1 - u
    const float by_log = -__logf(upper ? 1.f - z : u);
    const float by_series = z * (1.f + z * (0.5f + z * (0.33333334f + z * 0.25f)));
    const float nl = (upper && z < 0.015625f) ? by_series : by_log;
    return -__logf(nl);
}

// A fragments of q for the GQA group of (b, j): k-step s of thread column c covers dims
// (c + 4 (s / 2)) * 8 + 4 (s % 2) + {0,1} (a0) and + {2,3} (a2); the B fragments use the same
// permutation of the 128 dims, so a lane feeds the tensor core the 16-byte pieces c, c+4, c+8,
// c+12 of a key row exactly as they lie in memory.
template <int G>
__device__ __forceinline__ void load_q_fragments(const ScoreCtx &p, int b, int j, int g, int c, uint32_t (&qa)[8][2])
{
    const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
        p.q + ((size_t)b * p.n_q + (size_t)j * G + (g < G ? g : 0)) * kHeadDim);
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        const int w = (c + 4 * (s >> 1)) * 4 + 2 * (s & 1);
        qa[s][0] = g < G ? __ldg(qrow + w) : 0u;
        qa[s][1] = g < G ? __ldg(qrow + w + 1) : 0u;
    }
}

// This lane's pieces of the 16 keys of a tile that starts at team `base` of a pair with M team
// slots (rows past the last team repeat it; their scores are not stored).
__device__ __forceinline__ void load_key_pieces(const uint16_t *rep, int base, int M, int g, int c, uint4 (&kb)[2][4])
{
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const uint4 *row = reinterpret_cast<const uint4 *>(rep + (size_t)min(base + 8 * t + g, M - 1) * kHeadDim);
#pragma unroll
        for (int i = 0; i < 4; ++i) kb[t][i] = __ldg(row + c + 4 * i);
    }
}

// Scores of one tile of 16 teams (two n-tiles of 8; B row n = team base + 8 t + g) from the key
// pieces kb of this lane: writes Y32 for the G heads.
// csr_tile points at the 17 row offsets of the tile's teams (global or shared memory).
template <int G, bool kHalf>
__device__ __forceinline__ void score_tile(const ScoreCtx &p, int b, int j, int64_t team0, int M, int base,
                                           const int32_t *csr_tile, const uint4 (&kb)[2][4], const uint32_t (&qa)[8][2],
                                           uint32_t step, float scale, int g, int c)
{
    const uint32_t head = (uint32_t)(j * G + (g < G ? g : 0));
    float *y = p.y32 + ((size_t)head * p.n_seqs + b) * p.y_stride;
    // team sizes of this lane's four teams (teams base + 8 t + 2 c, + 1)
    int n_team[2][2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int t0 = base + 8 * t + 2 * c, o = 8 * t + 2 * c;
        const int r0 = t0 < M ? csr_tile[o] : 0, r1 = t0 < M ? csr_tile[o + 1] : 1, r2 = t0 + 1 < M ? csr_tile[o + 2] : 2;
        n_team[t][0] = r1 - r0;
        n_team[t][1] = r2 - r1;
    }
    float acc[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            mma_score<kHalf>(acc[t], qa[2 * i][0], qa[2 * i][1], kb[t][i].x, kb[t][i].y);
            mma_score<kHalf>(acc[t], qa[2 * i + 1][0], qa[2 * i + 1][1], kb[t][i].z, kb[t][i].w);
        }
    }
    // One Philox block covers four consecutive teams of a head: teams base + 8 t + {0..3} belong
    // to thread columns 0 and 1, + {4..7} to columns 2 and 3. The even column computes the block
    // of n-tile 0, the odd one that of n-tile 1, and the two exchange halves.
    const int my_t = c & 1;
    const uint4 words = philox4x32_10(
        make_uint4((uint32_t)(base + 8 * my_t + 4 * (c >> 1)) >> 2, step, head, p.stream_base + (uint32_t)b),
        p.seed_lo, p.seed_hi);
    // this lane needs words {2 (c & 1), 2 (c & 1) + 1} of both n-tiles' blocks
    uint32_t w[2][2];
    {
        const uint32_t give0 = (c & 1) ? words.x : words.z, give1 = (c & 1) ? words.y : words.w;
        const uint32_t got0 = __shfl_xor_sync(0xFFFFFFFFu, give0, 1), got1 = __shfl_xor_sync(0xFFFFFFFFu, give1, 1);
        const uint32_t keep0 = (c & 1) ? words.z : words.x, keep1 = (c & 1) ? words.w : words.y;
        w[0][0] = my_t ? got0 : keep0;
        w[0][1] = my_t ? got1 : keep1;
        w[1][0] = my_t ? keep0 : got0;
        w[1][1] = my_t ? keep1 : got1;
    }
    // acc[t][0], acc[t][1]: head g, teams base + 8 t + 2 c, + 1
    if (g < G) {
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int t0 = base + 8 * t + 2 * c;
            const float y0 = __logf((float)n_team[t][0]) + acc[t][0] * scale + gumbel32_from_word(w[t][0]);
            const float y1 = __logf((float)n_team[t][1]) + acc[t][1] * scale + gumbel32_from_word(w[t][1]);
            if (t0 + 1 < M) *reinterpret_cast<float2 *>(y + t0) = make_float2(y0, y1);      // t0 is even, the row 16-byte aligned
            else if (t0 < M) y[t0] = y0;
        }
    }
}

}  // namespace santapp
