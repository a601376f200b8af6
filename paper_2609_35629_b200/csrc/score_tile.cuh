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
    int tune_flags;                 // diagnostic builds only: bits switch parts of the tile off
};

// D (16 teams x 8 heads) += A (16 teams x 16 dims, row) * B (16 dims x 8 heads, col), fp32 accumulation.
template <bool kHalf>
__device__ __forceinline__ void mma_score(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    if constexpr (kHalf)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
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

// What the first half of a tile's work leaves for the second half (all in registers).
struct TileScores {
    float dot[4];                   // q . l for (team g, head 2c), (g, 2c+1), (g+8, 2c), (g+8, 2c+1)
    float log_lo, log_hi;           // log n of teams g and g + 8
    float *y_row[2];                // score rows of heads 2c and 2c + 1 for the tile's sequence
    int t_lo;                       // team base + g; -1 when the tile is empty
    int M;
};

// Scores of one tile of 16 teams from the key pieces kb of this lane (kb[t][i]: 16-byte piece
// c + 4 i of the key of team base + 8 t + g), in two halves so that a kernel walking many tiles can
// run the tensor-core instructions of one tile beside the arithmetic of the previous one.
// The 16 teams are the M rows of the tensor-core tile and the query heads its 8 columns, so one
// instruction per 16 dimensions covers the whole tile (the legacy tensor-core instruction is slow
// on this GPU, and a tile's time is mostly spent waiting for them). A lane ends up with the
// scores of teams g and g + 8 for heads 2 c and 2 c + 1.
// csr_tile points at the 17 row offsets of the tile's teams (global or shared memory);
// words_smem: 128 words of this warp's own shared memory (the tile's Philox words, [head][team]);
// the caller orders writes and reads of that buffer (__syncwarp) between the two halves.
template <int G, bool kHalf>
__device__ __forceinline__ void score_tile_front(const ScoreCtx &p, int b, int j, int M, int base, const int32_t *csr_tile,
                                                 const uint4 (&kb)[2][4], const uint32_t (&qa)[8][2], uint32_t step, int g,
                                                 int c, uint32_t *words_smem, TileScores &out)
{
    const int lane = 4 * g + c;
    // One Philox block covers four consecutive teams of a head: 4 blocks per head and tile, lane
    // 4 h + tb computes the block of head h, teams base + 4 tb .. + 3, and leaves its words in
    // shared memory at [h][4 tb .. 4 tb + 3].
    {
        const int h = lane >> 2, tb = lane & 3;
        uint4 words = make_uint4((uint32_t)(base >> 2) + (uint32_t)tb, step, (uint32_t)(j * G + (h < G ? h : 0)),
                                 p.stream_base + (uint32_t)b);
#ifdef SANTAPP_TUNE
        if (!(p.tune_flags & 2))
#endif
        words = philox4x32_10(words, p.seed_lo, p.seed_hi);
        reinterpret_cast<uint4 *>(words_smem)[lane] = words;
    }
    // sizes of this lane's two teams
    const int t_lo = base + g, t_hi = base + g + 8;
    const int n_lo = t_lo < M ? csr_tile[g + 1] - csr_tile[g] : 1;
    const int n_hi = t_hi < M ? csr_tile[g + 9] - csr_tile[g + 8] : 1;
    out.log_lo = __logf((float)n_lo);
    out.log_hi = __logf((float)n_hi);
    out.t_lo = t_lo;
    out.M = M;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int h = min(2 * c + e, G - 1);
        out.y_row[e] = p.y32 + ((size_t)(j * G + h) * p.n_seqs + b) * p.y_stride;
    }
    // two accumulators (even and odd steps of 16 dimensions)
    float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
#ifdef SANTAPP_TUNE
    if (p.tune_flags & 1) { acc0[0] = __uint_as_float(kb[0][0].x ^ kb[1][1].y); acc0[2] = __uint_as_float(kb[0][2].z ^ kb[1][3].w); } else
#endif
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        mma_score<kHalf>(acc0, kb[0][i].x, kb[1][i].x, kb[0][i].y, kb[1][i].y, qa[2 * i][0], qa[2 * i][1]);
        mma_score<kHalf>(acc1, kb[0][i].z, kb[1][i].z, kb[0][i].w, kb[1][i].w, qa[2 * i + 1][0], qa[2 * i + 1][1]);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) out.dot[e] = acc0[e] + acc1[e];
}

template <int G>
__device__ __forceinline__ void score_tile_back(const TileScores &t, float scale, int g, int c, const uint32_t *words_smem)
{
    if (t.t_lo < 0) return;
#pragma unroll
    for (int e = 0; e < 2; ++e) {                          // head 2 c + e
        const int h = 2 * c + e;
        if (h < G) {
            const float y_lo = t.log_lo + t.dot[e] * scale + gumbel32_from_word(words_smem[h * 16 + g]);
            const float y_hi = t.log_hi + t.dot[2 + e] * scale + gumbel32_from_word(words_smem[h * 16 + g + 8]);
            if (t.t_lo < t.M) t.y_row[e][t.t_lo] = y_lo;
            if (t.t_lo + 8 < t.M) t.y_row[e][t.t_lo + 8] = y_hi;
        }
    }
}

}  // namespace santapp
