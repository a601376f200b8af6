// Representative scoring for SANTA++ decode attention (Algorithm 1, routing logits and their
// Gumbel perturbation), in fp32 on tensor cores:
//   Y32_{h,g} = log n_g + q_h . l_g * scale + G_{h,g}          (Eq. method-routing plus noise)
// for every query head h of a KV head and every team g, one representative key l_g per team.
// These scores only choose which teams are re-evaluated exactly (see pairplan.cuh); the sample
// itself is decided in fp64 there.
//
// The GQA group is the M tile of S^T = q K^T (mma.sync m16n8k16, bf16 inputs, fp32
// accumulation). Lanes load 16-byte pieces of the representative keys straight from global
// memory; the contraction index is permuted consistently on both operands, so no shared memory
// staging is needed.
#include "common.cuh"

namespace santapp {

namespace {

constexpr int kScoreThreads = 256;
constexpr int kScoreTeamsPerWarp = 16;
constexpr int kScoreTeamsPerCta = kScoreTeamsPerWarp * (kScoreThreads / 32);

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    // A rows 8..15 are zero (a1 = a3 = 0): only heads 0..7 exist
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                 "{%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// Gumbel(0,1) in fp32 from a 32-bit word: u = (x + 0.5) / 2^32, G = -log(-log u). The upper half
// of the range goes through log1p so that -log u keeps its relative accuracy as u -> 1.
__device__ __forceinline__ float gumbel32_from_word(uint32_t x)
{
    float nl;
    if (x >= 0x80000000u) {
        const float w = (float)(0xFFFFFFFFu - x) + 0.5f;              // 2^32 - x - 0.5
        nl = -log1pf(-w * 2.3283064365386963e-10f);
    } else {
        nl = -logf(((float)x + 0.5f) * 2.3283064365386963e-10f);
    }
    return -logf(nl);
}

template <int G>
__global__ void __launch_bounds__(kScoreThreads)
score32_kernel(ScoreParams p)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    const int pair = blockIdx.y;
    const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;

    // The first block clears the tickets the later kernels of this call count on.
    if (blockIdx.x == 0 && blockIdx.y == 0) {
        for (int i = tid; i < p.n_pairs; i += kScoreThreads) p.ctl.attend_ticket[i] = 0;
        if (tid == 0) {
            *p.ctl.plan_ticket = 0;
            if (p.status) *p.status = 0;
        }
    }

    const int64_t team0 = p.bv.seq_team_off[b];
    const int M = (int)(p.bv.seq_team_off[b + 1] - team0);
    if (p.n_sample >= M) return;                       // every team is read; nothing is drawn
    const int base = blockIdx.x * kScoreTeamsPerCta + warp * kScoreTeamsPerWarp;
    if (base >= M) return;

    // A fragments of q: k-step s of thread column c covers dims (c + 4 (s / 2)) * 8 + 4 (s % 2) + {0,1}
    // (a0) and + {2,3} (a2); the B fragments below use the same permutation of the 128 dims.
    uint32_t qa[8][2];
    {
        const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
            p.q + ((size_t)b * p.bv.n_q + (size_t)j * G + (g < G ? g : 0)) * kHeadDim);
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const int w = (c + 4 * (s >> 1)) * 4 + 2 * (s & 1);
            qa[s][0] = g < G ? __ldg(qrow + w) : 0u;
            qa[s][1] = g < G ? __ldg(qrow + w + 1) : 0u;
        }
    }
    const uint16_t *rep = p.rep_keys + ((size_t)j * p.bv.teams_total + team0) * kHeadDim;
    const int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    const uint32_t step = p.step + (p.step_dev ? *p.step_dev : 0u);
    const float scale = (float)p.scale;

    // two n-tiles of 8 teams; B row n = team base + 8 tile + g, this lane holds chunks c, c+4, c+8, c+12
    uint4 kb[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int team = min(base + 8 * t + g, M - 1);
        const uint4 *row = reinterpret_cast<const uint4 *>(rep + (size_t)team * kHeadDim);
#pragma unroll
        for (int i = 0; i < 4; ++i) kb[t][i] = __ldg(row + c + 4 * i);
    }
    float acc[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            mma_bf16_16816(acc[t], qa[2 * i][0], qa[2 * i][1], kb[t][i].x, kb[t][i].y);
            mma_bf16_16816(acc[t], qa[2 * i + 1][0], qa[2 * i + 1][1], kb[t][i].z, kb[t][i].w);
        }
    }
    // acc[t][0], acc[t][1]: head g, teams base + 8 t + 2c, + 1
    float blk_max = -INFINITY;
    const uint32_t head = (uint32_t)(j * G + (g < G ? g : 0));
    if (g < G) {
        float *y = p.y32 + (size_t)head * p.bv.teams_total + team0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int t0 = base + 8 * t + 2 * c;                      // even team id: both share a Philox block
            if (t0 < M) {
                const uint4 words = philox4x32_10(
                    make_uint4((uint32_t)t0 >> 2, step, head, p.stream_base + (uint32_t)b), p.seed_lo, p.seed_hi);
                const int r0 = csr[t0], r1 = csr[t0 + 1];
                const float y0 = logf((float)(r1 - r0)) + acc[t][0] * scale
                                 + gumbel32_from_word(pick_word(words, t0 & 3));
                y[t0] = y0;
                blk_max = fmaxf(blk_max, y0);
                if (t0 + 1 < M) {
                    const int r2 = csr[t0 + 2];
                    const float y1 = logf((float)(r2 - r1)) + acc[t][1] * scale
                                     + gumbel32_from_word(pick_word(words, (t0 & 3) + 1));
                    y[t0 + 1] = y1;
                    blk_max = fmaxf(blk_max, y1);
                }
            }
        }
    }
    // largest score of the warp's 16-team block, per head (the quad of a head holds its 16 scores)
    blk_max = fmaxf(blk_max, __shfl_xor_sync(0xFFFFFFFFu, blk_max, 1));
    blk_max = fmaxf(blk_max, __shfl_xor_sync(0xFFFFFFFFu, blk_max, 2));
    if (g < G && c == 0)
        p.ymax[(size_t)head * p.ymax_stride + (size_t)(team0 >> 4) + b + (base >> 4)] = blk_max;
}

// One block per (sequence, KV head): largest |element| among the pair's representative keys.
__global__ void __launch_bounds__(256)
rep_abs_max_kernel(BatchView bv, const uint16_t *rep_keys, float *rep_abs_max)
{
    __shared__ uint32_t red[8];
    const int b = blockIdx.x, j = blockIdx.y;
    const int64_t team0 = bv.seq_team_off[b];
    const int64_t n = (bv.seq_team_off[b + 1] - team0) * kHeadDim / 2;     // 32-bit words
    const uint32_t *w = reinterpret_cast<const uint32_t *>(rep_keys + ((size_t)j * bv.teams_total + team0) * kHeadDim);
    uint32_t m = 0u;                                                        // bf16 magnitudes order like integers
    for (int64_t i = threadIdx.x; i < n; i += blockDim.x) {
        const uint32_t v = w[i];
        m = max(m, max(v & 0x7FFFu, (v >> 16) & 0x7FFFu));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) m = max(m, red[i]);
        rep_abs_max[(size_t)j * bv.n_seqs + b] = __uint_as_float(m << 16);
    }
}

template <int G>
cudaError_t launch_score32_g(const ScoreParams &p, int max_teams, cudaStream_t s)
{
    dim3 grid((max_teams + kScoreTeamsPerCta - 1) / kScoreTeamsPerCta, p.n_pairs);
    score32_kernel<G><<<grid, kScoreThreads, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score32(const ScoreParams &p, int max_teams_per_seq, cudaStream_t s)
{
    switch (p.bv.group) {
        case 1: return launch_score32_g<1>(p, max_teams_per_seq, s);
        case 2: return launch_score32_g<2>(p, max_teams_per_seq, s);
        case 3: return launch_score32_g<3>(p, max_teams_per_seq, s);
        case 4: return launch_score32_g<4>(p, max_teams_per_seq, s);
        case 5: return launch_score32_g<5>(p, max_teams_per_seq, s);
        case 6: return launch_score32_g<6>(p, max_teams_per_seq, s);
        case 7: return launch_score32_g<7>(p, max_teams_per_seq, s);
        case 8: return launch_score32_g<8>(p, max_teams_per_seq, s);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_rep_abs_max(const BatchView &bv, const uint16_t *rep_keys, float *rep_abs_max, cudaStream_t s)
{
    rep_abs_max_kernel<<<dim3(bv.n_seqs, bv.n_kv), 256, 0, s>>>(bv, rep_keys, rep_abs_max);
    return cudaGetLastError();
}

}  // namespace santapp
