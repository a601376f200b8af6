// Shared-latent rows (appendix "Token sparsity after latent compression"): one stored row per
// token, a 512-value content latent followed by a 64-value rotary key, shared by up to 16 query
// heads. Teams come from the latents alone (Algorithm 4 + Algorithm 2), every head runs
// Algorithm 1 on the shared teams with its own query against the whole row, a row is read once
// when any head selected its team, and its latent part is the value.
//
// Kernels of one decode step:
//   latent_score_kernel    fp32 routing scores of all 16 heads for 16 teams per warp (mma.sync,
//                          teams as the M tile, heads as two N tiles, 36 k-steps), Gumbel added
//   latent_select_kernel   Algorithm 1's sample per (sequence, head): select_head over 576 values
//   latent_plan_kernel     union of the heads' samples per sequence, written row by row: source
//                          row and segment of every row to read, per-segment log c (or -inf) per head
//   latent_attend_kernel   one block per SM, 32-row tiles: four warps compute S = Q K^T (contraction
//                          split between them), softmax and P, four copy the rows and accumulate
//                          O += P V (value columns split between them); one partial per (block, sequence)
//                          (latent_tc.cuh: the same operator on tcgen05, chosen by the environment)
//   latent_merge_kernel    log-sum-exp merge of the partials
#include <cuda_bf16.h>
#include <limits.h>
#include <math_constants.h>

#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <vector>

#include "build_util.cuh"
#include "common.cuh"
#include "headplan.cuh"
#include "santapp_latent.h"
#include "score_tile.cuh"

using namespace santapp;

namespace {

constexpr int kRowDim = SANTAPP_LATENT_ROW;          // 576 values per row
constexpr int kLatDim = SANTAPP_LATENT_DIM;          // 512: distances, means and values use these
constexpr int kRowBytes = kRowDim * 2;               // 1152
constexpr int kRowChunks = kRowBytes / 16;           // 72 16-byte pieces
constexpr int kHeads = SANTAPP_LATENT_MAX_HEADS;     // 16: the M tile of the attention MMAs
constexpr int kMaxP = SANTAPP_LATENT_MAX_PARENT;
constexpr int kLatPartialStride = 4 + kLatDim;       // floats per (slot, head): m, l, 2 pad, acc[512]
constexpr int kMaxLatentSeqs = 4096;

struct LatentView {
    int n_seqs, n_heads;
    const int64_t *seq_row_off, *seq_team_off;
    int64_t rows_total, teams_total;
};

// ---------------------------------------------------------------------------------------------
// Records: contiguous parents, Algorithm 2 on the latent columns
// ---------------------------------------------------------------------------------------------
struct LatentBuildParams {
    LatentView lv;
    int parent_size, reps, teams_per_full_parent;
    const uint16_t *rows_prompt;
    uint16_t *rows_packed, *rep_rows;
    int32_t *team_row_start, *row_token;
    float *rep_abs_max;
    uint8_t *owner;                 // workspace [rows_total]
    int max_parents_per_seq;
};

constexpr int kLbThreads = 128;

// Squared distance between two rows' latent parts in fp64: dims in increasing order, multiply
// and add rounded separately (the order the records are defined with).
__device__ __forceinline__ double latent_sqdist(const uint32_t *a, const uint32_t *b)
{
    double s = 0.0;
#pragma unroll 8
    for (int w = 0; w < kLatDim / 2; ++w) {
        const uint32_t x = a[w], y = b[w];
        const double e0 = __dsub_rn((double)bf16_lo(x), (double)bf16_lo(y));
        const double e1 = __dsub_rn((double)bf16_hi(x), (double)bf16_hi(y));
        s = __dadd_rn(s, __dmul_rn(e0, e0));
        s = __dadd_rn(s, __dmul_rn(e1, e1));
    }
    return s;
}

// One block per (parent, sequence).
__global__ void __launch_bounds__(kLbThreads)
latent_build_parent_kernel(LatentBuildParams p)
{
    constexpr int kPitch = kRowDim / 2 + 1;                 // words per staged row (+1: conflict-free column walks)
    __shared__ uint32_t rows[kMaxP * kPitch];
    __shared__ double mu[kLatDim];
    __shared__ double mind[kMaxP];
    __shared__ ValIdx scratch[33];
    __shared__ int owner[kMaxP], count[kMaxP], rep_of[kMaxP];
    __shared__ unsigned char is_rep[kMaxP];

    const int parent = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const int64_t row0 = p.lv.seq_row_off[b];
    const int N = (int)(p.lv.seq_row_off[b + 1] - row0);
    const int P = p.parent_size;
    const int first = parent * P;
    if (first >= N) return;
    const int nC = min(P, N - first);
    const int r = min(p.reps, nC);

    const uint32_t *src = reinterpret_cast<const uint32_t *>(p.rows_prompt) + (size_t)(row0 + first) * (kRowDim / 2);
    for (int e = tid; e < nC * (kRowDim / 2); e += kLbThreads) rows[(e / (kRowDim / 2)) * kPitch + e % (kRowDim / 2)] = src[e];
    for (int i = tid; i < nC; i += kLbThreads) { is_rep[i] = 0; count[i] = 0; }
    __syncthreads();

    // parent mean of the latent columns: rows added in token order, then one division
    for (int d = tid; d < kLatDim; d += kLbThreads) {
        double s = 0.0;
        for (int i = 0; i < nC; ++i) {
            const uint32_t word = rows[i * kPitch + (d >> 1)];
            s = __dadd_rn(s, (double)((d & 1) ? bf16_hi(word) : bf16_lo(word)));
        }
        mu[d] = __ddiv_rn(s, (double)nC);
    }
    __syncthreads();

    // first representative: the row whose latent is nearest the mean
    {
        ValIdx best = {INFINITY, INT_MAX};
        for (int i = tid; i < nC; i += kLbThreads) {
            double s = 0.0;
            const uint32_t *row = rows + i * kPitch;
            for (int w = 0; w < kLatDim / 2; ++w) {
                const uint32_t word = row[w];
                const double e0 = __dsub_rn((double)bf16_lo(word), mu[2 * w]);
                const double e1 = __dsub_rn((double)bf16_hi(word), mu[2 * w + 1]);
                s = __dadd_rn(s, __dmul_rn(e0, e0));
                s = __dadd_rn(s, __dmul_rn(e1, e1));
            }
            ValIdx c = {s, i};
            best = pick<true>(best, c);
        }
        best = block_arg<true>(best, scratch);
        if (tid == 0) { rep_of[0] = best.i; is_rep[best.i] = 1; }
    }
    __syncthreads();

    // farthest-first representatives with the running nearest-representative assignment
    for (int i = tid; i < nC; i += kLbThreads) { mind[i] = INFINITY; owner[i] = 0; }
    for (int u = 0; u < r; ++u) {
        const uint32_t *ref = rows + rep_of[u] * kPitch;
        ValIdx far = {-2.0, INT_MAX};
        for (int i = tid; i < nC; i += kLbThreads) {
            const double dist = latent_sqdist(rows + i * kPitch, ref);
            if (dist < mind[i]) { mind[i] = dist; owner[i] = u; }
            ValIdx c = {is_rep[i] ? -1.0 : mind[i], i};
            far = pick<false>(far, c);
        }
        if (u + 1 < r) {
            far = block_arg<false>(far, scratch);
            if (tid == 0) { rep_of[u + 1] = far.i; is_rep[far.i] = 1; }
            __syncthreads();
        }
    }
    __syncthreads();
    for (int u = tid; u < r; u += kLbThreads) owner[rep_of[u]] = u;      // a representative owns its own row
    __syncthreads();
    for (int i = tid; i < nC; i += kLbThreads) atomicAdd(&count[owner[i]], 1);
    __syncthreads();

    uint8_t *owner_out = p.owner + row0 + first;
    for (int i = tid; i < nC; i += kLbThreads) owner_out[i] = (uint8_t)owner[i];
    const int64_t team0 = p.lv.seq_team_off[b];
    const int team_local0 = parent * p.teams_per_full_parent;
    int32_t *csr = p.team_row_start + team0 + b;
    if (parent == 0 && tid == 0) csr[0] = 0;
    for (int u = tid; u < r; u += kLbThreads) csr[1 + team_local0 + u] = count[u];    // sizes; scanned next
    uint32_t *rep_dst = reinterpret_cast<uint32_t *>(p.rep_rows) + (size_t)(team0 + team_local0) * (kRowDim / 2);
    for (int e = tid; e < r * (kRowDim / 2); e += kLbThreads)
        rep_dst[e] = rows[rep_of[e / (kRowDim / 2)] * kPitch + e % (kRowDim / 2)];
}

// One block per sequence: team sizes -> CSR offsets, and the largest |value| of the representatives.
__global__ void __launch_bounds__(256)
latent_scan_kernel(LatentBuildParams p)
{
    __shared__ int scratch[33];
    __shared__ uint32_t red[8];
    const int b = blockIdx.x;
    const int64_t team0 = p.lv.seq_team_off[b];
    const int M = (int)(p.lv.seq_team_off[b + 1] - team0);
    int32_t *csr = p.team_row_start + team0 + b + 1;
    int carry = 0;
    for (int base = 0; base < M; base += 256) {
        const int g = base + threadIdx.x;
        const int v = g < M ? csr[g] : 0;
        int total;
        const int excl = block_exclusive_scan(v, scratch, total);
        if (g < M) csr[g] = carry + excl + v;
        carry += total;
    }
    const uint32_t *w = reinterpret_cast<const uint32_t *>(p.rep_rows) + (size_t)team0 * (kRowDim / 2);
    const int64_t n = (int64_t)M * (kRowDim / 2);
    uint32_t m = 0u;                                        // bf16 magnitudes order like integers
    for (int64_t i = threadIdx.x; i < n; i += 256) {
        const uint32_t v = w[i];
        m = max(m, max(v & 0x7FFFu, (v >> 16) & 0x7FFFu));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) m = max(m, red[i]);
        p.rep_abs_max[b] = __uint_as_float(m << 16);
    }
}

// One block per (parent, sequence): stable partition of the parent's rows by team, row copies.
__global__ void __launch_bounds__(kLbThreads)
latent_pack_kernel(LatentBuildParams p)
{
    __shared__ uint8_t owner[kMaxP];
    __shared__ int dest[kMaxP];
    const int parent = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const int64_t row0 = p.lv.seq_row_off[b];
    const int N = (int)(p.lv.seq_row_off[b + 1] - row0);
    const int first = parent * p.parent_size;
    if (first >= N) return;
    const int nC = min(p.parent_size, N - first);
    for (int i = tid; i < nC; i += kLbThreads) owner[i] = p.owner[row0 + first + i];
    __syncthreads();
    const int32_t *csr = p.team_row_start + p.lv.seq_team_off[b] + b;
    const int team_local0 = parent * p.teams_per_full_parent;
    for (int i = tid; i < nC; i += kLbThreads) {
        const int u = owner[i];
        int rank = 0;
        for (int a = 0; a < i; ++a) rank += (owner[a] == u);
        dest[i] = csr[team_local0 + u] + rank;              // members in increasing token index
    }
    __syncthreads();
    const uint4 *src = reinterpret_cast<const uint4 *>(p.rows_prompt) + (size_t)(row0 + first) * kRowChunks;
    uint4 *dst = reinterpret_cast<uint4 *>(p.rows_packed) + (size_t)row0 * kRowChunks;
    for (int e = tid; e < nC * kRowChunks; e += kLbThreads) {
        const int i = e / kRowChunks, c = e - i * kRowChunks;
        dst[(size_t)dest[i] * kRowChunks + c] = src[e];
    }
    for (int i = tid; i < nC; i += kLbThreads) p.row_token[row0 + dest[i]] = first + i;
}

// ---------------------------------------------------------------------------------------------
// Routing scores (Eq. method-routing plus the Gumbel term), fp32 on tensor cores
// ---------------------------------------------------------------------------------------------
struct LatentScoreParams {
    LatentView lv;
    const uint16_t *rep_rows;       // [teams_total][576]
    const int32_t *team_row_start;  // [teams_total + n_seqs]
    const uint16_t *q;              // [n_seqs][n_heads][576]
    float *y32;                     // [n_heads][n_seqs][y_stride]
    int64_t y_stride;
    int n_sample, tiles_per_warp;
    uint32_t seed_lo, seed_hi, step, stream_base;
    const uint32_t *step_dev;
    float scale;
};

constexpr int kLsThreads = 256;
constexpr int kLsTeamsPerBlock = (kLsThreads / 32) * 16;

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 32 bytes from global memory in one instruction (read-only path; the address is 32-byte aligned).
struct Words8 { uint32_t v[8]; };
__device__ __forceinline__ Words8 ldg256(const void *p)
{
    Words8 w;
    asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w.v[0]), "=r"(w.v[1]), "=r"(w.v[2]), "=r"(w.v[3]), "=r"(w.v[4]), "=r"(w.v[5]), "=r"(w.v[6]), "=r"(w.v[7])
                 : "l"(p));
    return w;
}

// Grid (ceil(max teams / (128 tiles_per_warp)), sequences); a warp scores tiles_per_warp consecutive
// tiles of 16 teams for all heads: the teams are the MMA's 16 rows, the heads its columns (two tiles
// of 8), the 576 values 36 k-steps. Both operands use the same permutation of the contraction index
// inside every segment of 64 values (128 bytes), so a lane feeds the tensor core 32-byte pieces of a
// representative row (and of a query) as they lie in memory: lane t of a row's four lanes takes bytes
// [32 t, 32 t + 32) of the segment with one 256-bit load, and the s-th eight bytes of its piece are
// its k-slots {2t, 2t+1, 2t+8, 2t+9} of the segment's s-th MMA. One load instruction of a warp then
// touches eight whole 128-byte lines (with 16-byte pieces it touched eight half lines, and the kernel
// was bound by the number of line accesses in L1: 70 % of its peak at 48 % of the DRAM bandwidth).
// The host picks tiles_per_warp so that all blocks
// are resident at once (two per SM): a second, partly filled wave of blocks costs as much as a full one.
__global__ void __launch_bounds__(kLsThreads)
latent_score_kernel(LatentScoreParams p)
{
    constexpr int kQPitchW = (kRowBytes + 16) / 4;                  // words per staged query (+16 bytes: conflict-free LDS.128)
    __shared__ __align__(16) uint32_t q_s[kHeads * kQPitchW];
    __shared__ __align__(16) uint32_t words_s[kLsThreads / 32][kHeads][16];
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t team0 = p.lv.seq_team_off[b];
    const int M = (int)(p.lv.seq_team_off[b + 1] - team0);
    const int tpw = p.tiles_per_warp;
    if (p.n_sample >= M || (int)blockIdx.x * kLsTeamsPerBlock * tpw >= M) return;    // nothing is drawn / no team here
    const int H = p.lv.n_heads;
    // the warp's first pieces of its representatives' rows are requested before anything else: they
    // do not depend on the queries, and the block's set-up (queries into shared memory) runs while
    // they are on their way
    constexpr int kBatch = 3;                                       // segments of 64 values requested together
    constexpr int kSegs = kRowDim / 64;                             // 9 segments of 128 bytes per row
    const int t_first = ((int)blockIdx.x * (kLsThreads / 32) + warp) * tpw * 16;
    const bool live = t_first < M;
    const int r = lane >> 2, t = lane & 3;
    const uint16_t *rep = p.rep_rows + (size_t)team0 * kRowDim;
    auto row_ptr = [&](int team) { return reinterpret_cast<const unsigned char *>(rep + (size_t)min(team, M - 1) * kRowDim) + 32 * t; };
    Words8 wa[kBatch], wb[kBatch];
    if (live) {
        const unsigned char *ka = row_ptr(t_first + r), *kb = row_ptr(t_first + r + 8);
#pragma unroll
        for (int i = 0; i < kBatch; ++i) { wa[i] = ldg256(ka + i * 128); wb[i] = ldg256(kb + i * 128); }
    }
    const int32_t *csr = p.team_row_start + team0 + b;
    const uint32_t step = p.step + (p.step_dev ? *p.step_dev : 0u);
    {
        const uint4 *qg = reinterpret_cast<const uint4 *>(p.q + (size_t)b * H * kRowDim);
        constexpr int kMine = (kHeads * kRowChunks + kLsThreads - 1) / kLsThreads;
        uint4 v[kMine];
#pragma unroll
        for (int u = 0; u < kMine; ++u) {                           // all of a thread's pieces in flight at once
            const int e = tid + u * kLsThreads, h = e / kRowChunks, c = e - h * kRowChunks;
            v[u] = (e < kHeads * kRowChunks && h < H) ? __ldg(qg + (size_t)h * kRowChunks + c) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kMine; ++u) {
            const int e = tid + u * kLsThreads, h = e / kRowChunks, c = e - h * kRowChunks;
            if (e < kHeads * kRowChunks) *reinterpret_cast<uint4 *>(q_s + h * kQPitchW + c * 4) = v[u];
        }
    }
    __syncthreads();
    if (!live) return;

#pragma unroll 1
    for (int it = 0; it < tpw; ++it) {
        const int t0 = t_first + it * 16;
        if (t0 >= M) break;
        const int ga = t0 + r, gb = t0 + r + 8;                     // the lane's two teams (rows r and r + 8 of the tile)
        const unsigned char *ka = row_ptr(ga), *kb = row_ptr(gb);
        const bool more = it + 1 < tpw && t0 + 16 < M;              // the next tile's first pieces follow this tile's last
        const unsigned char *ka_next = row_ptr(ga + 16), *kb_next = row_ptr(gb + 16);
        int na = 1, nb = 1;
        if (ga < M) na = csr[ga + 1] - csr[ga];
        if (gb < M) nb = csr[gb + 1] - csr[gb];
        // Philox words of the tile: lane computes the blocks of head (lane & 15) for two groups of four teams
        {
            const int h = lane & 15, tg = (lane >> 4) * 2;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint4 w = philox4x32_10(make_uint4((uint32_t)(t0 >> 2) + tg + u, step, (uint32_t)h, p.stream_base + (uint32_t)b),
                                              p.seed_lo, p.seed_hi);
                *reinterpret_cast<uint4 *>(&words_s[warp][h][(tg + u) * 4]) = w;
            }
        }
        float acc[2][4] = {};
#pragma unroll 1
        for (int sg0 = 0; sg0 < kSegs; sg0 += kBatch) {
            const bool last = sg0 + kBatch >= kSegs;
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                // the lane's 32 bytes of the two queries (heads r and r + 8) for this segment
                const uint32_t *qa = q_s + r * kQPitchW + (sg0 + i) * 32 + 8 * t;
                const uint32_t *qb = qa + 8 * kQPitchW;
                const uint4 qa0 = *reinterpret_cast<const uint4 *>(qa), qa1 = *reinterpret_cast<const uint4 *>(qa + 4);
                const uint4 qb0 = *reinterpret_cast<const uint4 *>(qb), qb1 = *reinterpret_cast<const uint4 *>(qb + 4);
                const uint32_t q0[8] = {qa0.x, qa0.y, qa0.z, qa0.w, qa1.x, qa1.y, qa1.z, qa1.w};
                const uint32_t q1[8] = {qb0.x, qb0.y, qb0.z, qb0.w, qb1.x, qb1.y, qb1.z, qb1.w};
#pragma unroll
                for (int s4 = 0; s4 < 4; ++s4) {
                    mma_bf16(acc[0], wa[i].v[2 * s4], wb[i].v[2 * s4], wa[i].v[2 * s4 + 1], wb[i].v[2 * s4 + 1], q0[2 * s4], q0[2 * s4 + 1]);
                    mma_bf16(acc[1], wa[i].v[2 * s4], wb[i].v[2 * s4], wa[i].v[2 * s4 + 1], wb[i].v[2 * s4 + 1], q1[2 * s4], q1[2 * s4 + 1]);
                }
                if (!last) {                                        // the same piece of the next batch
                    wa[i] = ldg256(ka + (sg0 + kBatch + i) * 128);
                    wb[i] = ldg256(kb + (sg0 + kBatch + i) * 128);
                } else if (more) {
                    wa[i] = ldg256(ka_next + i * 128);
                    wb[i] = ldg256(kb_next + i * 128);
                }
            }
        }
        __syncwarp();
        const float log_a = __logf((float)na), log_b = __logf((float)nb);
#pragma unroll
        for (int n = 0; n < 2; ++n) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int h = 8 * n + 2 * t + e;
                if (h < H) {
                    float *row = p.y32 + ((size_t)h * p.lv.n_seqs + b) * p.y_stride;
                    if (ga < M) row[ga] = log_a + acc[n][e] * p.scale + gumbel32_from_word(words_s[warp][h][r]);
                    if (gb < M) row[gb] = log_b + acc[n][2 + e] * p.scale + gumbel32_from_word(words_s[warp][h][r + 8]);
                }
            }
        }
        __syncwarp();                                               // the words are rewritten for the next tile
    }
}

// ---------------------------------------------------------------------------------------------
// Sampling per (sequence, head): Algorithm 1 on 576-value routing keys
// ---------------------------------------------------------------------------------------------
template <int kT>
__global__ void __launch_bounds__(kT, kT >= 512 ? 1 : 1024 / kT)
latent_select_kernel(PlanInputs in)
{
    __shared__ HeadSmemT<kRowDim> sm;
    trace_mark(in.trace, 1, 0);
    select_head<kT, kT >= 512 ? 4 : 2, false, kRowDim>(in, blockIdx.x, sm);
    trace_mark(in.trace, 1, 1);
}

// ---------------------------------------------------------------------------------------------
// Union of the heads' samples per sequence, written row by row
// ---------------------------------------------------------------------------------------------
struct LatentPlanParams {
    LatentView lv;
    const int32_t *sel_team;        // [n_seqs][n_heads][K]
    const float *sel_logc;
    const int2 *sel_rows;
    const int32_t *suffix_len;      // nullable
    int suffix_cap, n_sample, seg_cap;
    int2 *row_meta;                 // [rows_total + n_seqs * suffix_cap] {source row, segment}: sequence b's rows to
                                    //   read, in team order then suffix, start at seq_row_off[b] + b * suffix_cap
    float *seg_bias;                // [n_seqs][seg_cap][16] -log2(e) log c_g of each head (a row's weight is e^s / c_g),
                                    //   -inf where the head did not select the team
    int32_t *pair_rows;             // [n_seqs] rows to read
    int32_t *dbg_sel_idx;
    float *dbg_sel_logc;
    double *dbg_tau;
    int32_t *dbg_union_rows;
};

constexpr int kLpThreads = 512;
constexpr int kLatMaxSample = 256;                          // K: the paper's largest budget, S = 1024 rows at R / P = 1 / 4
constexpr int kLatSegMax = kHeads * kLatMaxSample + 1;      // 16 heads x K teams, + the suffix
constexpr int kLpPerThread = kHeads * kLatMaxSample / kLpThreads;     // sampled teams of a sequence per thread
static_assert(kLpPerThread * kLpThreads == kHeads * kLatMaxSample, "a block holds a sequence's samples in registers");

struct LatentPlanSmem {
    uint32_t bitmap[kMaxTeamsPerSeq / 32];
    int wprefix[kMaxTeamsPerSeq / 32];
    int seg_start[kLatSegMax], seg_n[kLatSegMax], seg_prefix[kLatSegMax + 1];
    int scan[40];
};

__global__ void __launch_bounds__(kLpThreads)
latent_plan_kernel(LatentPlanParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    LatentPlanSmem &sm = *reinterpret_cast<LatentPlanSmem *>(smem_raw);
    const int b = blockIdx.x, tid = threadIdx.x;
    const int H = p.lv.n_heads, K = p.n_sample;
    const int64_t row0 = p.lv.seq_row_off[b];
    const int N = (int)(p.lv.seq_row_off[b + 1] - row0);
    const int M = (int)(p.lv.seq_team_off[b + 1] - p.lv.seq_team_off[b]);
    int t_suffix = 0;
    if (p.suffix_len != nullptr && p.suffix_cap > 0) t_suffix = max(0, min(p.suffix_len[b], p.suffix_cap));
    int2 *line = p.row_meta + row0 + (int64_t)b * p.suffix_cap;
    float *bias = p.seg_bias + (size_t)b * p.seg_cap * kHeads;
    const size_t head0 = (size_t)b * H;
    const float kLog2e = 1.4426950408889634f;

    if (K >= M) {
        // every team is read with correction one; nothing was drawn
        for (int i = tid; i < N; i += kLpThreads) line[i] = make_int2((int)(row0 + i), 0);
        for (int i = tid; i < t_suffix; i += kLpThreads) line[N + i] = make_int2((int)(kSrcSuffix | (uint32_t)(b * p.suffix_cap + i)), 0);
        if (tid < kHeads) bias[tid] = 0.f;
        if (tid == 0) {
            p.pair_rows[b] = N + t_suffix;
            if (p.dbg_union_rows) p.dbg_union_rows[b] = N;
        }
        for (int e = tid; e < H * K; e += kLpThreads) {
            const int a = e % K;
            if (p.dbg_sel_idx) p.dbg_sel_idx[head0 * K + e] = a < M ? a : -1;
            if (p.dbg_sel_logc) p.dbg_sel_logc[head0 * K + e] = 0.f;
        }
        if (tid < H && p.dbg_tau) p.dbg_tau[head0 + tid] = __longlong_as_double(0x7FF8000000000000ll);
        return;
    }

    const int n_words = (M + 31) / 32, E = H * K;
    // a thread's share of the samples (at most kLpPerThread entries), all requested at once
    int my_team[kLpPerThread];
    int2 my_rows[kLpPerThread];
    float my_logc[kLpPerThread];
#pragma unroll
    for (int u = 0; u < kLpPerThread; ++u) {
        const int e = tid + u * kLpThreads;
        my_team[u] = -1;
        if (e < E) {
            my_team[u] = __ldcg(p.sel_team + head0 * K + e);
            my_rows[u] = __ldcg(p.sel_rows + head0 * K + e);
            my_logc[u] = __ldcg(p.sel_logc + head0 * K + e);
            if (my_team[u] >= M) my_team[u] = -1;                              // cannot come from the sampler
        }
    }
    for (int i = tid; i < n_words; i += kLpThreads) sm.bitmap[i] = 0u;
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kLpPerThread; ++u)
        if (my_team[u] >= 0) atomicOr(&sm.bitmap[my_team[u] >> 5], 1u << (my_team[u] & 31));
    __syncthreads();
    int nseg;
    {
        const int wpt = (n_words + kLpThreads - 1) / kLpThreads;
        const int lo = min(tid * wpt, n_words), hi = min(lo + wpt, n_words);
        int sum = 0;
        for (int w = lo; w < hi; ++w) sum += __popc(sm.bitmap[w]);
        int run = block_exclusive_scan(sum, sm.scan, nseg);
        for (int w = lo; w < hi; ++w) { sm.wprefix[w] = run; run += __popc(sm.bitmap[w]); }
    }
    for (int i = tid; i < nseg * kHeads; i += kLpThreads) bias[i] = -CUDART_INF_F;
    if (tid < kHeads) bias[(size_t)nseg * kHeads + tid] = 0.f;              // the suffix segment
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kLpPerThread; ++u) {
        const int team = my_team[u], e = tid + u * kLpThreads;
        if (team < 0) continue;
        const int seg = sm.wprefix[team >> 5] + __popc(sm.bitmap[team >> 5] & ((1u << (team & 31)) - 1u));
        bias[(size_t)seg * kHeads + e / K] = -kLog2e * my_logc[u];             // weight e^s / c_g
        sm.seg_start[seg] = my_rows[u].x;                                      // the same from every selecting head
        sm.seg_n[seg] = my_rows[u].y;
    }
    __syncthreads();
    int total;
    {
        const int spt = (nseg + kLpThreads - 1) / kLpThreads;
        const int lo = min(tid * spt, nseg), hi = min(lo + spt, nseg);
        int sum = 0;
        for (int sg = lo; sg < hi; ++sg) sum += sm.seg_n[sg];
        int run = block_exclusive_scan(sum, sm.scan, total);
        for (int sg = lo; sg < hi; ++sg) { sm.seg_prefix[sg] = run; run += sm.seg_n[sg]; }
    }
    __syncthreads();
    total = min(total, N);                                                     // distinct teams cannot hold more rows
    for (int sg = tid; sg < nseg; sg += kLpThreads) {
        const int at = sm.seg_prefix[sg], n = sm.seg_n[sg], start = sm.seg_start[sg];
        for (int i = 0; i < n && at + i < N; ++i) line[at + i] = make_int2((int)(row0 + min(start + i, N - 1)), sg);
    }
    for (int i = tid; i < t_suffix; i += kLpThreads)
        line[total + i] = make_int2((int)(kSrcSuffix | (uint32_t)(b * p.suffix_cap + i)), nseg);
    if (tid == 0) {
        p.pair_rows[b] = total + t_suffix;
        if (p.dbg_union_rows) p.dbg_union_rows[b] = total;
    }
}

// ---------------------------------------------------------------------------------------------
// Attention over the rows to read, and the merge of the blocks' partial results
// ---------------------------------------------------------------------------------------------
struct LatentAttendParams {
    LatentView lv;
    const uint16_t *rows_packed;    // [rows_total][576]
    const uint16_t *suffix_rows;    // [n_seqs][suffix_cap][576]
    const uint16_t *q;              // [n_seqs][n_heads][576]
    const int2 *row_meta;           // see LatentPlanParams (not read by the dense variant)
    const float *seg_bias;
    const int32_t *pair_rows;
    const int32_t *suffix_len;      // nullable
    int suffix_cap, seg_cap;
    float qk_scale_log2;            // scale * log2(e)
    float *partials;                // [grid + n_seqs][16][kLatPartialStride]: block c leaves sequence b's share in slot c + b
    uint32_t *pair_prefix;          // [n_seqs + 1] rows to read before each sequence; written by block 0 for the merge
    unsigned long long *trace;      // nullable: device-timer marks of the third tile of a block's first share (diagnostic)
};

constexpr int kTileRows = 32;
constexpr int kTileBytes = kTileRows * kRowBytes;                   // 36864
constexpr int kBiasPitch = 20;                                      // floats per tile row (16 heads + pad: conflict-free reads)

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}

// One block per SM. The rows to read of all sequences form one line, cut into equal ranges, one per
// block; a block walks the sequences its range touches, 32 rows (a tile) at a time, and leaves one
// partial result per sequence. Eight warps in two roles. Four compute S = Q Rows^T of a tile with
// the contraction split between them (each keeps its 144 of the 576 query values as A fragments in
// registers), add the four partial S tiles up through shared memory, take a quarter of the tile's
// rows each through the softmax step (tile maxima exchanged through shared memory) and hand P (two
// bf16 terms, already laid out as the A fragments of the next product) and the factors by which the
// running maxima moved over through shared memory. The other four copy the rows from global memory
// into a ring of four tiles (eight lanes copy 128 contiguous bytes of a row into one XOR-swizzled
// line, so ldmatrix is conflict-free and a global sector lands in one piece) and accumulate
// O += P V for their 128 of the 512 value columns. S of a tile runs beside P V of the tile before it
// while two more tiles are on their way from memory; named barriers order the hand-overs.
constexpr int kLfThreads = 256;
constexpr int kLfStages = 4;
constexpr int kLfOffBias = kLfStages * kTileBytes;                              // [stage][32 rows][kBiasPitch] floats
constexpr int kLfOffXch = kLfOffBias + kLfStages * kTileRows * kBiasPitch * 4;  // [tile parity][4 warps][4][32 lanes] float4
constexpr int kLfOffP = kLfOffXch + 2 * 4 * 4 * 32 * 16 + 2 * 64 * 4;            // (+ the warps' tile maxima [parity][4][16]); P: [tile parity][16 registers][32 lanes]
constexpr int kLfOffAlpha = kLfOffP + 2 * 16 * 32 * 4;                          // [tile parity][16 heads]
constexpr int kLfOffMl = kLfOffAlpha + 2 * 16 * 4;                              // [m 16 | l of each S warp 4 x 16]
constexpr int kLfOffPrefix = kLfOffMl + 80 * 4;
constexpr int kLfOffScan = kLfOffPrefix + (kMaxLatentSeqs + 4) * 4;
constexpr int kLfSmemBytes = kLfOffScan + 48 * 4;

__device__ __forceinline__ void named_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void named_arrive(int id, int count) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory"); }
// named barriers: rows of a tile are in shared memory (by tile parity), P of a tile is in shared
// memory (by parity), the S warps among themselves, the P V warps among themselves
enum { kLfBarData = 1, kLfBarP = 3, kLfBarS = 5, kLfBarV = 6, kLfBarS2 = 7 };

// Diagnostic: the calling thread notes its SM's cycle counter in mark `slot` of its block (kernel 3 of the trace).
__device__ __forceinline__ void lf_mark(unsigned long long *trace, bool on, int slot)
{
    if (trace != nullptr && on && blockIdx.x < (unsigned)kTraceBlocks) {
        trace[((size_t)3 * kTraceBlocks + blockIdx.x) * kTraceSlots + slot] = (unsigned long long)clock64();   // SM cycles
    }
}

template <bool kAll>
__global__ void __launch_bounds__(kLfThreads, 1)
latent_attend_kernel(LatentAttendParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pv_role = warp >> 2, gw = warp & 3, gt = gw * 32 + lane;
    const int r = lane >> 2, t = lane & 3;
    uint32_t *prefix = reinterpret_cast<uint32_t *>(smem + kLfOffPrefix);
    int *scan = reinterpret_cast<int *>(smem + kLfOffScan);
    const int n = p.lv.n_seqs, H = p.lv.n_heads;
    {
        uint32_t carry = 0;
        for (int base = 0; base < n; base += kLfThreads) {
            const int i = base + tid;
            int v = 0;
            if (i < n) {
                if (kAll) {
                    v = (int)(p.lv.seq_row_off[i + 1] - p.lv.seq_row_off[i]);
                    if (p.suffix_len != nullptr && p.suffix_cap > 0) v += max(0, min(p.suffix_len[i], p.suffix_cap));
                } else {
                    v = __ldcg(p.pair_rows + i);
                }
            }
            int total;
            const int excl = block_exclusive_scan(v, scan, total);
            if (i < n) prefix[i] = carry + (uint32_t)excl;
            carry += (uint32_t)total;
        }
        if (tid == 0) prefix[n] = carry;
        __syncthreads();
    }
    if (blockIdx.x == 0)
        for (int i = tid; i <= n; i += kLfThreads) p.pair_prefix[i] = prefix[i];
    const uint32_t total = prefix[n];
    const uint32_t per = (total + gridDim.x - 1) / gridDim.x;
    const uint32_t lo = min(total, blockIdx.x * per), hi = min(total, lo + per);
    if (lo >= hi) return;
    int pr = 0;
    {
        int a = 0, c = n;                                   // largest pr with prefix[pr] <= lo
        while (c - a > 1) {
            const int mid = (a + c) >> 1;
            if (prefix[mid] <= lo) a = mid; else c = mid;
        }
        pr = a;
    }
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
    const float *bias_all = reinterpret_cast<const float *>(smem + kLfOffBias);
    float4 *xch_all = reinterpret_cast<float4 *>(smem + kLfOffXch);
    uint32_t *p_all = reinterpret_cast<uint32_t *>(smem + kLfOffP);
    float *alpha_all = reinterpret_cast<float *>(smem + kLfOffAlpha);
    float *ml = reinterpret_cast<float *>(smem + kLfOffMl);
    const uint4 *rows_g = reinterpret_cast<const uint4 *>(p.rows_packed);
    const uint4 *suffix_g = reinterpret_cast<const uint4 *>(p.suffix_rows);

    for (; pr < n && prefix[pr] < hi; ++pr) {
        if (prefix[pr + 1] <= lo) continue;
        const int b = pr;
        const int s_lo = (int)(max(lo, prefix[pr]) - prefix[pr]), s_hi = (int)(min(hi, prefix[pr + 1]) - prefix[pr]);
        const int64_t row0 = p.lv.seq_row_off[b];
        const int N = (int)(p.lv.seq_row_off[b + 1] - row0);
        const int n_tiles = (s_hi - s_lo + kTileRows - 1) / kTileRows;

        if (!pv_role) {
            // ================= S, softmax, P =================
            float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F, l0 = 0.f, l1 = 0.f;       // heads r and r + 8
            uint32_t qa[9][4];                              // the warp's share of the queries: values [144 gw, 144 gw + 144)
            {
                const uint32_t *q32 = reinterpret_cast<const uint32_t *>(p.q + (size_t)b * H * kRowDim);
#pragma unroll
                for (int ks = 0; ks < 9; ++ks) {
                    const int d0 = 16 * (9 * gw + ks) + 2 * t;
                    qa[ks][0] = r < H ? __ldg(q32 + (r * kRowDim + d0) / 2) : 0u;
                    qa[ks][1] = r + 8 < H ? __ldg(q32 + ((r + 8) * kRowDim + d0) / 2) : 0u;
                    qa[ks][2] = r < H ? __ldg(q32 + (r * kRowDim + d0 + 8) / 2) : 0u;
                    qa[ks][3] = r + 8 < H ? __ldg(q32 + ((r + 8) * kRowDim + d0 + 8) / 2) : 0u;
                }
            }
#pragma unroll 1
            for (int j = 0; j < n_tiles; ++j) {
                const int par = j & 1, stage = j & (kLfStages - 1);
                const bool tr = j >= 4 && j <= 5 && gt == 0;
                lf_mark(p.trace, tr && j == 4, 0);
                named_sync(kLfBarData + par, 256);          // the tile's rows (and corrections) have landed
                lf_mark(p.trace, tr && j == 4, 1);
                const uint32_t tile_addr = smem_base + stage * kTileBytes;
                const float *bias_s = bias_all + stage * kTileRows * kBiasPitch;
                const int nv = min(kTileRows, s_hi - (s_lo + kTileRows * j));
                float x[4][4];
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) x[nt][0] = x[nt][1] = x[nt][2] = x[nt][3] = 0.f;
                {
                    // all of the warp's key fragments first (the loads pipeline; an MMA right behind its own
                    // load would wait out the load's latency every time), then the 36 MMAs
                    uint32_t kb[9][2][4];
#pragma unroll
                    for (int ks = 0; ks < 9; ++ks) {
#pragma unroll
                        for (int ntp = 0; ntp < 2; ++ntp) {
                            const int row = 16 * ntp + ((lane >> 4) << 3) + (lane & 7);
                            const int chunk = 18 * gw + 2 * ks + ((lane >> 3) & 1);
                            ldmatrix_x4(kb[ks][ntp][0], kb[ks][ntp][1], kb[ks][ntp][2], kb[ks][ntp][3],
                                        tile_addr + row * kRowBytes + ((chunk ^ (lane & 7)) << 4));
                        }
                    }
#pragma unroll
                    for (int ks = 0; ks < 9; ++ks) {
#pragma unroll
                        for (int ntp = 0; ntp < 2; ++ntp) {
                            mma_bf16(x[2 * ntp], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], kb[ks][ntp][0], kb[ks][ntp][1]);
                            mma_bf16(x[2 * ntp + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], kb[ks][ntp][2], kb[ks][ntp][3]);
                        }
                    }
                }
                float4 *xch = xch_all + par * (4 * 4 * 32);
                lf_mark(p.trace, tr && j == 4, 2);
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) xch[(gw * 4 + nt) * 32 + lane] = make_float4(x[nt][0], x[nt][1], x[nt][2], x[nt][3]);
                named_sync(kLfBarS, 128);
                lf_mark(p.trace, tr && j == 4, 3);
                // from here on the warp owns rows 8 gw .. 8 gw + 7 of the tile: its four values per lane are
                // heads r (y0, y1) and r + 8 (y2, y3) for rows 8 gw + 2 t and + 1
                float y0, y1, y2, y3;
                {
                    float4 sacc = xch[gw * 32 + lane];
#pragma unroll
                    for (int w = 1; w < 4; ++w) {
                        const float4 v = xch[(w * 4 + gw) * 32 + lane];
                        sacc.x += v.x; sacc.y += v.y; sacc.z += v.z; sacc.w += v.w;
                    }
                    const int row = 8 * gw + 2 * t;
                    const float b00 = kAll ? 0.f : bias_s[row * kBiasPitch + r], b01 = kAll ? 0.f : bias_s[(row + 1) * kBiasPitch + r];
                    const float b10 = kAll ? 0.f : bias_s[row * kBiasPitch + r + 8], b11 = kAll ? 0.f : bias_s[(row + 1) * kBiasPitch + r + 8];
                    y0 = row < nv ? fmaf(sacc.x, p.qk_scale_log2, b00) : -CUDART_INF_F;
                    y1 = row + 1 < nv ? fmaf(sacc.y, p.qk_scale_log2, b01) : -CUDART_INF_F;
                    y2 = row < nv ? fmaf(sacc.z, p.qk_scale_log2, b10) : -CUDART_INF_F;
                    y3 = row + 1 < nv ? fmaf(sacc.w, p.qk_scale_log2, b11) : -CUDART_INF_F;
                }
                float mx0 = fmaxf(y0, y1), mx1 = fmaxf(y2, y3);
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 1));
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 2));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 1));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 2));
                float *mxw = reinterpret_cast<float *>(xch_all) + 2 * (4 * 4 * 32) * 4 + par * 64;   // [parity][4 warps][16 heads]
                if (t == 0) {
                    mxw[gw * 16 + r] = mx0;
                    mxw[gw * 16 + r + 8] = mx1;
                }
                named_sync(kLfBarS2, 128);
                mx0 = fmaxf(fmaxf(mxw[r], mxw[16 + r]), fmaxf(mxw[32 + r], mxw[48 + r]));
                mx1 = fmaxf(fmaxf(mxw[r + 8], mxw[16 + r + 8]), fmaxf(mxw[32 + r + 8], mxw[48 + r + 8]));
                const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                const float mu0 = mn0 == -CUDART_INF_F ? 0.f : mn0, mu1 = mn1 == -CUDART_INF_F ? 0.f : mn1;
                const float a0 = ex2(m0 - mu0), a1 = ex2(m1 - mu1);
                m0 = mn0;
                m1 = mn1;
                y0 = ex2(y0 - mu0);
                y1 = ex2(y1 - mu0);
                y2 = ex2(y2 - mu1);
                y3 = ex2(y3 - mu1);
                l0 = l0 * a0 + y0 + y1;                     // the warp's rows only: the four warps' sums are added at the end
                l1 = l1 * a1 + y2 + y3;
                {
                    // P as the A fragments of P V: n-tile gw is registers (gw / 2) * 4 + (gw % 2) * 2 and + 1 of a lane
                    uint32_t *pb = p_all + par * (16 * 32);
                    const int reg = (gw >> 1) * 4 + (gw & 1) * 2;
                    const uint32_t h0 = pack_bf16(y0, y1), h1 = pack_bf16(y2, y3);
                    pb[reg * 32 + lane] = h0;
                    pb[(reg + 1) * 32 + lane] = h1;
                    pb[(8 + reg) * 32 + lane] = pack_bf16(y0 - bf16_lo(h0), y1 - bf16_hi(h0));
                    pb[(8 + reg + 1) * 32 + lane] = pack_bf16(y2 - bf16_lo(h1), y3 - bf16_hi(h1));
                    if (gw == 0 && t == 0) {
                        alpha_all[par * 16 + r] = a0;
                        alpha_all[par * 16 + r + 8] = a1;
                    }
                }
                named_arrive(kLfBarP + par, 256);
                lf_mark(p.trace, tr && j == 4, 4);
                lf_mark(p.trace, tr && j == 5, 5);
            }
            l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 1);
            l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 2);
            l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 1);
            l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 2);
            if (t == 0) {
                if (gw == 0) { ml[r] = m0; ml[r + 8] = m1; }
                ml[16 + gw * 16 + r] = l0;                  // [4 warps][16 heads]
                ml[16 + gw * 16 + r + 8] = l1;
            }
            __syncthreads();                                // m and l are in shared memory
        } else {
            // ================= copies and O += P V =================
            float o[16][4];                                 // 16 heads x the warp's 128 value columns
#pragma unroll
            for (int j2 = 0; j2 < 16; ++j2) o[j2][0] = o[j2][1] = o[j2][2] = o[j2][3] = 0.f;
            const int2 *line = kAll ? nullptr : p.row_meta + row0 + (int64_t)b * p.suffix_cap;
            const float *bias_g = kAll ? nullptr : p.seg_bias + (size_t)b * p.seg_cap * kHeads;
            // source rows (and segments) of this thread's two rows of tile j, rows gt / 8 and gt / 8 + 16; -1: no row
            auto load_meta = [&](int j) -> int4 {
                int4 m = make_int4(-1, 0, -1, 0);
                if (j >= n_tiles) return m;
                const int pos = s_lo + kTileRows * j + (gt >> 3);
                if (kAll) {
                    if (pos < s_hi) m.x = pos < N ? (int)(row0 + pos) : (int)(kSrcSuffix | (uint32_t)(b * p.suffix_cap + pos - N));
                    if (pos + 16 < s_hi)
                        m.z = pos + 16 < N ? (int)(row0 + pos + 16) : (int)(kSrcSuffix | (uint32_t)(b * p.suffix_cap + pos + 16 - N));
                    return m;
                }
                if (pos < s_hi) { const int2 v = __ldcg(line + pos); m.x = v.x; m.y = v.y; }
                if (pos + 16 < s_hi) { const int2 v = __ldcg(line + pos + 16); m.z = v.x; m.w = v.y; }
                return m;
            };
            // eight threads copy a row, 128 bytes per instruction (one line of shared memory: the swizzle only
            // permutes pieces inside it); rows past the share's end are zero-filled
            auto issue = [&](int j, int4 meta) {
                if (j < n_tiles) {
                    const int jl = gt & 7, stage = j & (kLfStages - 1);
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const int i = (gt >> 3) + 16 * half;
                        const int msrc = half ? meta.z : meta.x, mseg = half ? meta.w : meta.y;
                        const bool valid = msrc != -1;
                        const uint32_t src = (uint32_t)msrc;
                        const uint4 *g = !valid ? rows_g
                                                : ((src & kSrcSuffix) ? suffix_g + (size_t)(src & 0x7FFFFFFFu) * kRowChunks
                                                                      : rows_g + (size_t)src * kRowChunks);
                        const uint32_t dst = smem_base + stage * kTileBytes + i * kRowBytes + ((jl ^ (i & 7)) << 4);
                        const int bytes = valid ? 16 : 0;
#pragma unroll
                        for (int c = 0; c < kRowChunks / 8; ++c) cp_async16(dst + c * 128, g + 8 * c + jl, bytes);
                        if (!kAll && jl < 4) {
                            const uint32_t bdst = smem_base + kLfOffBias + (stage * kTileRows * kBiasPitch + i * kBiasPitch + 4 * jl) * 4;
                            cp_async16(bdst, valid ? bias_g + (size_t)mseg * kHeads + 4 * jl : reinterpret_cast<const float *>(rows_g), bytes);
                        }
                    }
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
            };
#pragma unroll
            for (int j = 0; j < kLfStages; ++j) issue(j, load_meta(j));
            asm volatile("cp.async.wait_group 3;" ::: "memory");
            named_arrive(kLfBarData, 256);                  // tile 0 is there
            int4 meta_next = load_meta(kLfStages);
#pragma unroll 1
            for (int j = 0; j < n_tiles; ++j) {
                const int par = j & 1;
                const int4 meta_cur = meta_next;            // of the tile issued at the end of this round
                meta_next = load_meta(j + kLfStages + 1);
                const bool tr = j == 4 && gt == 0;
                lf_mark(p.trace, tr, 6);
                if (j + 1 < n_tiles) {                      // tile j + 1 was requested three rounds ago: tell the S warps
                    asm volatile("cp.async.wait_group 2;" ::: "memory");
                    named_arrive(kLfBarData + (par ^ 1), 256);
                }
                lf_mark(p.trace, tr, 7);
                named_sync(kLfBarP + par, 256);             // P of tile j is there
                lf_mark(p.trace, tr, 8);
                uint32_t pf[16];
                const uint32_t *pb = p_all + par * (16 * 32);
#pragma unroll
                for (int i = 0; i < 16; ++i) pf[i] = pb[i * 32 + lane];
                const float a0 = alpha_all[par * 16 + r], a1 = alpha_all[par * 16 + r + 8];
                if (__any_sync(0xFFFFFFFFu, a0 != 1.f || a1 != 1.f)) {        // most tiles leave the maxima where they were
#pragma unroll
                    for (int j2 = 0; j2 < 16; ++j2) { o[j2][0] *= a0; o[j2][1] *= a0; o[j2][2] *= a1; o[j2][3] *= a1; }
                }
                const uint32_t tile_addr = smem_base + (j & (kLfStages - 1)) * kTileBytes;
                {
                    uint32_t vb[2][8][4];                   // V fragments of the 16 column tiles, both k-steps: all loads first
#pragma unroll
                    for (int ks2 = 0; ks2 < 2; ++ks2) {
#pragma unroll
                        for (int j2 = 0; j2 < 8; ++j2) {
                            const int mi = lane >> 3;
                            const int row = 16 * ks2 + ((mi & 1) << 3) + (lane & 7);
                            const int chunk = 16 * gw + 2 * j2 + (mi >> 1);
                            ldmatrix_x4_trans(vb[ks2][j2][0], vb[ks2][j2][1], vb[ks2][j2][2], vb[ks2][j2][3],
                                              tile_addr + row * kRowBytes + ((chunk ^ (lane & 7)) << 4));
                        }
                    }
#pragma unroll
                    for (int ks2 = 0; ks2 < 2; ++ks2) {
#pragma unroll
                        for (int term = 0; term < 2; ++term) {      // 16 independent accumulators per term
#pragma unroll
                            for (int j2 = 0; j2 < 8; ++j2) {
                                mma_bf16(o[2 * j2], pf[8 * term + 4 * ks2], pf[8 * term + 4 * ks2 + 1], pf[8 * term + 4 * ks2 + 2],
                                         pf[8 * term + 4 * ks2 + 3], vb[ks2][j2][0], vb[ks2][j2][1]);
                                mma_bf16(o[2 * j2 + 1], pf[8 * term + 4 * ks2], pf[8 * term + 4 * ks2 + 1], pf[8 * term + 4 * ks2 + 2],
                                         pf[8 * term + 4 * ks2 + 3], vb[ks2][j2][2], vb[ks2][j2][3]);
                            }
                        }
                    }
                }
                lf_mark(p.trace, tr, 9);
                named_sync(kLfBarV, 128);                   // every P V warp is done with this stage
                lf_mark(p.trace, tr, 10);
                issue(j + kLfStages, meta_cur);
                lf_mark(p.trace, tr, 11);
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncthreads();                                // m and l are in shared memory
            const float M0 = ml[r], M1 = ml[r + 8];
            float *out0 = p.partials + ((size_t)(blockIdx.x + b) * kHeads + r) * kLatPartialStride;
            float *out1 = out0 + 8 * kLatPartialStride;
            if (gw == 0 && t == 0) {
                out0[0] = M0;
                out0[1] = ml[16 + r] + ml[32 + r] + ml[48 + r] + ml[64 + r];
                out1[0] = M1;
                out1[1] = ml[16 + r + 8] + ml[32 + r + 8] + ml[48 + r + 8] + ml[64 + r + 8];
            }
#pragma unroll
            for (int j2 = 0; j2 < 16; ++j2) {
                const int col = 4 + 128 * gw + 8 * j2 + 2 * t;
                *reinterpret_cast<float2 *>(out0 + col) = make_float2(o[j2][0], o[j2][1]);
                *reinterpret_cast<float2 *>(out1 + col) = make_float2(o[j2][2], o[j2][3]);
            }
        }
        __syncthreads();                                    // the share is done: shared memory may be reused
    }
}

}  // namespace

#include "latent_tc.cuh"

namespace {

// One block per (head, sequence): out = sum_c w_c acc_c / sum_c w_c l_c over the blocks that read
// rows of the sequence, w_c = 2^(m_c - max m). Four thread groups take every fourth partial; thread
// i of a group owns value columns 4 i .. 4 i + 3; the groups' sums meet in shared memory.
constexpr int kLmThreads = 512;
__global__ void __launch_bounds__(kLmThreads)
latent_merge_kernel(const float *partials, const uint32_t *pair_prefix, int n_seqs, int n_heads, int grid, float *out, int32_t *status)
{
    __shared__ float red[kLmThreads / 32];
    __shared__ float4 part_acc[3][128];
    __shared__ float part_l[3][128];
    const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, part = tid >> 7, col = tid & 127;
    const uint32_t total = pair_prefix[n_seqs], per = (total + grid - 1) / grid;
    const uint32_t lo = pair_prefix[b], hi = pair_prefix[b + 1];
    const int c_lo = (int)(lo / per), c_hi = hi > lo ? (int)((hi - 1) / per) : c_lo - 1;
    const float *base = partials + ((size_t)b * kHeads + h) * kLatPartialStride;      // slot c + b
    const size_t slot = (size_t)kHeads * kLatPartialStride;
    float M = -CUDART_INF_F;
    for (int c = c_lo + tid; c <= c_hi; c += kLmThreads) M = fmaxf(M, __ldcg(base + c * slot));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, o));
    if ((tid & 31) == 0) red[tid >> 5] = M;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kLmThreads / 32; ++w) M = fmaxf(M, red[w]);
    const float Mu = M == -CUDART_INF_F ? 0.f : M;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
    for (int c = c_lo + part; c <= c_hi; c += 8) {
        const float *p0 = base + c * slot, *p1 = p0 + 4 * slot;
        const bool two = c + 4 <= c_hi;
        const float m0 = __ldcg(p0), l0 = __ldcg(p0 + 1);
        const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(p0 + 4) + col);
        const float m1 = two ? __ldcg(p1) : -CUDART_INF_F, l1 = two ? __ldcg(p1 + 1) : 0.f;
        const float4 v1 = two ? __ldcg(reinterpret_cast<const float4 *>(p1 + 4) + col) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float w0 = ex2(m0 - Mu), w1 = ex2(m1 - Mu);
        L += w0 * l0 + w1 * l1;
        acc.x += w0 * v0.x + w1 * v1.x;
        acc.y += w0 * v0.y + w1 * v1.y;
        acc.z += w0 * v0.z + w1 * v1.z;
        acc.w += w0 * v0.w + w1 * v1.w;
    }
    if (part > 0) { part_acc[part - 1][col] = acc; part_l[part - 1][col] = L; }
    __syncthreads();
    if (part == 0) {
#pragma unroll
        for (int g = 0; g < 3; ++g) {
            const float4 v = part_acc[g][col];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            L += part_l[g][col];
        }
        const float inv = 1.f / L;
        const float4 res = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
        reinterpret_cast<float4 *>(out + ((size_t)b * n_heads + h) * kLatDim)[col] = res;
        if (status != nullptr && !(isfinite(res.x) && isfinite(res.y) && isfinite(res.z) && isfinite(res.w))) atomicOr(status, 1);
    }
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------
namespace {

inline size_t lat_align(size_t x) { return (x + 255) / 256 * 256; }
inline bool lat_misaligned(const void *p, size_t a) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) % a) != 0; }

int check_latent_geom(const santapp_latent_geom *g)
{
    if (!g) return SANTAPP_ERR_INVALID_ARG;
    if (g->n_seqs < 1 || g->n_heads < 1 || g->parent_size < 1 || g->reps_per_parent < 1) return SANTAPP_ERR_INVALID_ARG;
    if (g->parent_size % g->reps_per_parent != 0) return SANTAPP_ERR_INVALID_ARG;
    if (g->n_heads > kHeads || g->parent_size > kMaxP || g->n_seqs > kMaxLatentSeqs) return SANTAPP_ERR_UNSUPPORTED;
    return SANTAPP_OK;
}

int latent_teams_in_sequence(int N, int P, int R)
{
    const int full = N / P, tail = N % P;
    return full * (R < P ? R : P) + (tail ? (R < tail ? R : tail) : 0);
}

int check_latent_teams(const santapp_latent_geom *g, const santapp_latent_teams *t)
{
    if (!t) return SANTAPP_ERR_INVALID_ARG;
    if (!t->rows_packed || !t->rep_rows || !t->team_row_start || !t->seq_row_off || !t->seq_team_off || !t->rep_abs_max)
        return SANTAPP_ERR_INVALID_ARG;
    if (lat_misaligned(t->rows_packed, 16) || lat_misaligned(t->rep_rows, 32) || lat_misaligned(t->team_row_start, 4)
        || lat_misaligned(t->row_token, 4) || lat_misaligned(t->seq_row_off, 8) || lat_misaligned(t->seq_team_off, 8)
        || lat_misaligned(t->rep_abs_max, 4))
        return SANTAPP_ERR_INVALID_ARG;
    if (t->rows_total < g->n_seqs || t->teams_total < g->n_seqs || t->max_teams_per_seq < 1) return SANTAPP_ERR_INVALID_ARG;
    if (t->rows_total >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    if (t->max_teams_per_seq > kMaxTeamsPerSeq) return SANTAPP_ERR_UNSUPPORTED;
    return SANTAPP_OK;
}

LatentView make_latent_view(const santapp_latent_geom *g, const santapp_latent_teams *t)
{
    LatentView lv;
    lv.n_seqs = g->n_seqs;
    lv.n_heads = g->n_heads;
    lv.seq_row_off = t->seq_row_off;
    lv.seq_team_off = t->seq_team_off;
    lv.rows_total = t->rows_total;
    lv.teams_total = t->teams_total;
    return lv;
}

// Workspace of the decode calls. Offsets in bytes.
struct LatentLayout {
    size_t y32, sel_team, sel_logc, sel_rows, row_meta, seg_bias, pair_rows, pair_prefix, partials, total;
    int seg_cap, grid;
    int64_t y_stride;
};

LatentLayout latent_layout(const santapp_latent_geom *g, const santapp_latent_teams *t, int K, int suffix_cap, bool dense)
{
    LatentLayout L;
    L.grid = attend_grid_size();
    int64_t cap = (int64_t)g->n_heads * K;
    if (cap > t->max_teams_per_seq) cap = t->max_teams_per_seq;
    L.seg_cap = (int)cap + 1;
    L.y_stride = score_row_stride(t->max_teams_per_seq);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = lat_align(off + bytes); return o; };
    const size_t heads = (size_t)g->n_seqs * g->n_heads;
    L.y32 = take(dense ? 0 : sizeof(float) * (size_t)g->n_heads * g->n_seqs * (size_t)L.y_stride);
    L.sel_team = take(dense ? 0 : sizeof(int32_t) * heads * K);
    L.sel_logc = take(dense ? 0 : sizeof(float) * heads * K);
    L.sel_rows = take(dense ? 0 : sizeof(int2) * heads * K);
    L.row_meta = take(dense ? 0 : sizeof(int2) * ((size_t)t->rows_total + (size_t)g->n_seqs * suffix_cap));
    L.seg_bias = take(dense ? 0 : sizeof(float) * (size_t)g->n_seqs * L.seg_cap * kHeads);
    L.pair_rows = take(sizeof(int32_t) * (size_t)g->n_seqs);
    L.pair_prefix = take(sizeof(uint32_t) * ((size_t)g->n_seqs + 1));
    L.partials = take(sizeof(float) * ((size_t)L.grid + g->n_seqs) * kHeads * kLatPartialStride);
    L.total = off;
    return L;
}

int latent_attend_and_merge(const santapp_latent_geom *geom, const santapp_latent_teams *teams, const LatentLayout &L, char *ws,
                            const void *q, const void *suffix_rows, const int32_t *suffix_len_dev, int suffix_cap, float scale,
                            float *out, int32_t *status, bool dense, int mask, int &launches, cudaStream_t s,
                            unsigned long long *trace = nullptr)
{
    LatentAttendParams ap;
    ap.lv = make_latent_view(geom, teams);
    ap.rows_packed = static_cast<const uint16_t *>(teams->rows_packed);
    ap.suffix_rows = static_cast<const uint16_t *>(suffix_rows);
    ap.q = static_cast<const uint16_t *>(q);
    ap.row_meta = reinterpret_cast<const int2 *>(ws + L.row_meta);
    ap.seg_bias = reinterpret_cast<const float *>(ws + L.seg_bias);
    ap.pair_rows = reinterpret_cast<const int32_t *>(ws + L.pair_rows);
    ap.suffix_len = suffix_cap > 0 ? suffix_len_dev : nullptr;
    ap.suffix_cap = suffix_cap;
    ap.seg_cap = L.seg_cap;
    ap.qk_scale_log2 = (float)((double)scale * 1.4426950408889634);
    ap.partials = reinterpret_cast<float *>(ws + L.partials);
    ap.pair_prefix = reinterpret_cast<uint32_t *>(ws + L.pair_prefix);
    ap.trace = trace;
    cudaError_t err;
    if (mask & SANTAPP_STAGE_ATTEND) {
        static std::atomic<unsigned long long> done_tc_all, done_tc_sel;
        // The tcgen05 variant (latent_tc.cuh) computes the same thing on the 5th-generation tensor cores; it is
        // slower here (a tcgen05.mma of N = 16 columns costs as much as one of 64, and one thread issues 68 of
        // them per 64 rows), so the mma.sync kernel is the default and the other is chosen by the environment
        // (SANTAPP_LATENT_ATTEND=tcgen05).
        const char *which = getenv("SANTAPP_LATENT_ATTEND");
        const bool tc = which != nullptr && strcmp(which, "tcgen05") == 0;
        static std::atomic<unsigned long long> done_sp_all, done_sp_sel;
        if (!tc) {
            if (dense) {
                if ((err = ensure_dynamic_smem((const void *)latent_attend_kernel<true>, kLfSmemBytes, done_sp_all)) != cudaSuccess)
                    return note_cuda_failure(err, "latent attend attribute");
                err = launch_kernel(latent_attend_kernel<true>, dim3(L.grid), dim3(kLfThreads), kLfSmemBytes, s, ap);
            } else {
                if ((err = ensure_dynamic_smem((const void *)latent_attend_kernel<false>, kLfSmemBytes, done_sp_sel)) != cudaSuccess)
                    return note_cuda_failure(err, "latent attend attribute");
                err = launch_kernel(latent_attend_kernel<false>, dim3(L.grid), dim3(kLfThreads), kLfSmemBytes, s, ap);
            }
        } else if (dense) {
            if ((err = ensure_dynamic_smem((const void *)latent_attend_tc_kernel<true>, kTcSmemBytes, done_tc_all)) != cudaSuccess)
                return note_cuda_failure(err, "latent attend attribute");
            err = launch_kernel(latent_attend_tc_kernel<true>, dim3(L.grid), dim3(kTcThreads), kTcSmemBytes, s, ap, status);
        } else {
            if ((err = ensure_dynamic_smem((const void *)latent_attend_tc_kernel<false>, kTcSmemBytes, done_tc_sel)) != cudaSuccess)
                return note_cuda_failure(err, "latent attend attribute");
            err = launch_kernel(latent_attend_tc_kernel<false>, dim3(L.grid), dim3(kTcThreads), kTcSmemBytes, s, ap, status);
        }
        if (err != cudaSuccess) return note_cuda_failure(err, "latent attend launch");
        ++launches;
    }
    if (mask & SANTAPP_STAGE_MERGE) {
        err = launch_kernel(latent_merge_kernel, dim3(geom->n_heads, geom->n_seqs), dim3(kLmThreads), 0, s,
                            (const float *)ap.partials, (const uint32_t *)ap.pair_prefix, geom->n_seqs, geom->n_heads, L.grid, out,
                            status);
        if (err != cudaSuccess) return note_cuda_failure(err, "latent merge launch");
        ++launches;
    }
    return SANTAPP_OK;
}

}  // namespace

extern "C" {

int santapp_latent_sizes(const santapp_latent_geom *geom, const int32_t *prompt_len_host, santapp_sizes *out)
{
    const int rc = check_latent_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if (!prompt_len_host || !out) return SANTAPP_ERR_INVALID_ARG;
    int64_t rows = 0, tms = 0;
    int max_t = 0, max_r = 0;
    for (int b = 0; b < geom->n_seqs; ++b) {
        const int N = prompt_len_host[b];
        if (N < 1) return SANTAPP_ERR_INVALID_ARG;
        const int M = latent_teams_in_sequence(N, geom->parent_size, geom->reps_per_parent);
        rows += N;
        tms += M;
        if (M > max_t) max_t = M;
        if (N > max_r) max_r = N;
    }
    if (rows >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    if (max_t > kMaxTeamsPerSeq) return SANTAPP_ERR_UNSUPPORTED;
    out->rows_total = rows;
    out->teams_total = tms;
    out->max_teams_per_seq = max_t;
    out->max_rows_per_seq = max_r;
    out->team_row_start_elems = tms + geom->n_seqs;
    out->build_workspace_bytes = lat_align((size_t)rows);
    return SANTAPP_OK;
}

int santapp_latent_build_teams(const santapp_latent_geom *geom, const int32_t *prompt_len_host, const void *rows_prompt,
                               santapp_latent_teams *teams, void *workspace, size_t workspace_bytes, santapp_stream stream)
{
    santapp_sizes sz;
    const int rc = santapp_latent_sizes(geom, prompt_len_host, &sz);
    if (rc != SANTAPP_OK) return rc;
    if (!rows_prompt || !teams || !workspace) return SANTAPP_ERR_INVALID_ARG;
    if (!teams->rows_packed || !teams->rep_rows || !teams->team_row_start || !teams->row_token || !teams->seq_row_off
        || !teams->seq_team_off || !teams->rep_abs_max)
        return SANTAPP_ERR_INVALID_ARG;
    if (lat_misaligned(rows_prompt, 16) || lat_misaligned(workspace, 16) || lat_misaligned(teams->rows_packed, 16)
        || lat_misaligned(teams->rep_rows, 32) || lat_misaligned(teams->team_row_start, 4) || lat_misaligned(teams->row_token, 4)
        || lat_misaligned(teams->seq_row_off, 8) || lat_misaligned(teams->seq_team_off, 8) || lat_misaligned(teams->rep_abs_max, 4))
        return SANTAPP_ERR_INVALID_ARG;
    if (workspace_bytes < sz.build_workspace_bytes) return SANTAPP_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    std::vector<int64_t> offs(2 * ((size_t)geom->n_seqs + 1));
    int64_t *row_off = offs.data(), *team_off = offs.data() + geom->n_seqs + 1;
    row_off[0] = team_off[0] = 0;
    int max_parents = 0;
    for (int b = 0; b < geom->n_seqs; ++b) {
        const int N = prompt_len_host[b];
        row_off[b + 1] = row_off[b] + N;
        team_off[b + 1] = team_off[b] + latent_teams_in_sequence(N, geom->parent_size, geom->reps_per_parent);
        max_parents = std::max(max_parents, (N + geom->parent_size - 1) / geom->parent_size);
    }
    const size_t ob = sizeof(int64_t) * ((size_t)geom->n_seqs + 1);
    cudaError_t err = cudaMemcpyAsync(teams->seq_row_off, row_off, ob, cudaMemcpyHostToDevice, s);
    if (err != cudaSuccess) return note_cuda_failure(err, "copy seq_row_off");
    err = cudaMemcpyAsync(teams->seq_team_off, team_off, ob, cudaMemcpyHostToDevice, s);
    if (err != cudaSuccess) return note_cuda_failure(err, "copy seq_team_off");
    teams->rows_total = sz.rows_total;
    teams->teams_total = sz.teams_total;
    teams->max_teams_per_seq = sz.max_teams_per_seq;
    teams->max_rows_per_seq = sz.max_rows_per_seq;

    LatentBuildParams p;
    p.lv = make_latent_view(geom, teams);
    p.parent_size = geom->parent_size;
    p.reps = geom->reps_per_parent;
    p.teams_per_full_parent = std::min(geom->reps_per_parent, geom->parent_size);
    p.rows_prompt = static_cast<const uint16_t *>(rows_prompt);
    p.rows_packed = static_cast<uint16_t *>(teams->rows_packed);
    p.rep_rows = static_cast<uint16_t *>(teams->rep_rows);
    p.team_row_start = teams->team_row_start;
    p.row_token = teams->row_token;
    p.rep_abs_max = teams->rep_abs_max;
    p.owner = static_cast<uint8_t *>(workspace);
    p.max_parents_per_seq = max_parents;
    const dim3 grid(max_parents, geom->n_seqs);
    if ((err = launch_kernel(latent_build_parent_kernel, grid, dim3(kLbThreads), 0, s, p)) != cudaSuccess)
        return note_cuda_failure(err, "latent build launch");
    if ((err = launch_kernel(latent_scan_kernel, dim3(geom->n_seqs), dim3(256), 0, s, p)) != cudaSuccess)
        return note_cuda_failure(err, "latent scan launch");
    if ((err = launch_kernel(latent_pack_kernel, grid, dim3(kLbThreads), 0, s, p)) != cudaSuccess)
        return note_cuda_failure(err, "latent pack launch");
    return SANTAPP_OK;
}

size_t santapp_latent_decode_workspace_bytes(const santapp_latent_geom *geom, const santapp_latent_teams *teams, int32_t n_sample,
                                             int32_t suffix_cap)
{
    if (check_latent_geom(geom) != SANTAPP_OK || !teams || n_sample < 1 || n_sample > kLatMaxSample || suffix_cap < 0) return 0;
    return latent_layout(geom, teams, n_sample, suffix_cap, false).total;
}

size_t santapp_latent_dense_workspace_bytes(const santapp_latent_geom *geom, const santapp_latent_teams *teams)
{
    if (check_latent_geom(geom) != SANTAPP_OK || !teams) return 0;
    return latent_layout(geom, teams, 1, 0, true).total;
}

int santapp_latent_decode_attn(const santapp_latent_geom *geom, const santapp_latent_teams *teams, const void *q,
                               const void *suffix_rows, const int32_t *suffix_len_dev, int32_t suffix_cap, int32_t n_sample,
                               uint64_t seed, uint32_t step, const uint32_t *step_dev, uint32_t stream_base, float scale,
                               float *out, const santapp_debug *dbg, void *workspace, size_t workspace_bytes,
                               santapp_stream stream)
{
    note_launch_count(0);
    int rc = check_latent_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if ((rc = check_latent_teams(geom, teams)) != SANTAPP_OK) return rc;
    if (!q || !out || !workspace) return SANTAPP_ERR_INVALID_ARG;
    if (lat_misaligned(q, 16) || lat_misaligned(out, 16) || lat_misaligned(workspace, 16) || lat_misaligned(suffix_rows, 16)
        || lat_misaligned(suffix_len_dev, 4))
        return SANTAPP_ERR_INVALID_ARG;
    if (n_sample < 1 || suffix_cap < 0) return SANTAPP_ERR_INVALID_ARG;
    if (n_sample > kLatMaxSample) return SANTAPP_ERR_UNSUPPORTED;
    if (suffix_cap > 0 && suffix_len_dev && !suffix_rows) return SANTAPP_ERR_INVALID_ARG;
    if (!(scale > 0.f) || isinf(scale)) return SANTAPP_ERR_INVALID_ARG;
    if ((int64_t)geom->n_seqs * (int64_t)suffix_cap + teams->rows_total >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    const LatentLayout L = latent_layout(geom, teams, n_sample, suffix_cap, false);
    if (workspace_bytes < L.total) return SANTAPP_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(workspace);
    const int mask = current_stage_mask();
    int launches = 0;
    cudaError_t err;
    int32_t *status = dbg ? dbg->status : nullptr;
    if (status) {
        if ((err = cudaMemsetAsync(status, 0, sizeof(int32_t), s)) != cudaSuccess) return note_cuda_failure(err, "clear status");
    }
    const LatentView lv = make_latent_view(geom, teams);

    if (mask & SANTAPP_STAGE_ROUTE) {
        LatentScoreParams sp;
        sp.lv = lv;
        sp.rep_rows = static_cast<const uint16_t *>(teams->rep_rows);
        sp.team_row_start = teams->team_row_start;
        sp.q = static_cast<const uint16_t *>(q);
        sp.y32 = reinterpret_cast<float *>(ws + L.y32);
        sp.y_stride = L.y_stride;
        sp.n_sample = n_sample;
        sp.seed_lo = (uint32_t)(seed & 0xFFFFFFFFull);
        sp.seed_hi = (uint32_t)(seed >> 32);
        sp.step = step;
        sp.step_dev = step_dev;
        sp.stream_base = stream_base;
        sp.scale = scale;
        // as many tiles per warp as it takes for all blocks to be resident at once (two per SM)
        const long long blocks1 = (long long)((teams->max_teams_per_seq + kLsTeamsPerBlock - 1) / kLsTeamsPerBlock) * geom->n_seqs;
        const long long slots = 2ll * attend_grid_size();
        sp.tiles_per_warp = (int)std::min<long long>(std::max<long long>((blocks1 + slots - 1) / slots, 1), 64);
        const dim3 grid((teams->max_teams_per_seq + kLsTeamsPerBlock * sp.tiles_per_warp - 1) / (kLsTeamsPerBlock * sp.tiles_per_warp),
                        geom->n_seqs);
        if ((err = launch_kernel(latent_score_kernel, grid, dim3(kLsThreads), 0, s, sp)) != cudaSuccess)
            return note_cuda_failure(err, "latent score launch");
        ++launches;
    }
    if (mask & SANTAPP_STAGE_SELECT) {
        PlanInputs in = {};
        in.bv.n_seqs = geom->n_seqs;
        in.bv.n_q = geom->n_heads;
        in.bv.n_kv = 1;
        in.bv.group = geom->n_heads;
        in.bv.seq_row_off = teams->seq_row_off;
        in.bv.seq_team_off = teams->seq_team_off;
        in.bv.team_count = nullptr;
        in.bv.rows_total = teams->rows_total;
        in.bv.teams_total = teams->teams_total;
        in.bv.elem = 0;
        in.y32 = reinterpret_cast<const float *>(ws + L.y32);
        in.y_stride = L.y_stride;
        in.rep_keys = static_cast<const uint16_t *>(teams->rep_rows);
        in.team_row_start = teams->team_row_start;
        in.rep_abs_max = teams->rep_abs_max;
        in.q = static_cast<const uint16_t *>(q);
        in.n_sample = n_sample;
        in.seed_lo = (uint32_t)(seed & 0xFFFFFFFFull);
        in.seed_hi = (uint32_t)(seed >> 32);
        in.step = step;
        in.step_dev = step_dev;
        in.stream_base = stream_base;
        in.scale = (double)scale;
        in.suffix_len = suffix_cap > 0 ? suffix_len_dev : nullptr;
        in.suffix_cap = suffix_cap;
        in.sel_team = reinterpret_cast<int32_t *>(ws + L.sel_team);
        in.sel_logc = reinterpret_cast<float *>(ws + L.sel_logc);
        in.sel_rows = reinterpret_cast<int2 *>(ws + L.sel_rows);
        in.status = status;
        in.dbg_sel_idx = dbg ? dbg->sel_idx : nullptr;
        in.dbg_sel_logc = dbg ? dbg->sel_logc : nullptr;
        in.dbg_tau = dbg ? dbg->tau : nullptr;
        in.dbg_union_rows = nullptr;
        in.trace = dbg ? reinterpret_cast<unsigned long long *>(dbg->trace) : nullptr;
        const int n_heads = geom->n_seqs * geom->n_heads;
        if (n_heads <= L.grid) err = launch_kernel(latent_select_kernel<512>, dim3(n_heads), dim3(512), 0, s, in);
        else                   err = launch_kernel(latent_select_kernel<256>, dim3(n_heads), dim3(256), 0, s, in);
        if (err != cudaSuccess) return note_cuda_failure(err, "latent select launch");
        ++launches;

        LatentPlanParams pp;
        pp.lv = lv;
        pp.sel_team = in.sel_team;
        pp.sel_logc = in.sel_logc;
        pp.sel_rows = in.sel_rows;
        pp.suffix_len = in.suffix_len;
        pp.suffix_cap = suffix_cap;
        pp.n_sample = n_sample;
        pp.seg_cap = L.seg_cap;
        pp.row_meta = reinterpret_cast<int2 *>(ws + L.row_meta);
        pp.seg_bias = reinterpret_cast<float *>(ws + L.seg_bias);
        pp.pair_rows = reinterpret_cast<int32_t *>(ws + L.pair_rows);
        pp.dbg_sel_idx = in.dbg_sel_idx;
        pp.dbg_sel_logc = in.dbg_sel_logc;
        pp.dbg_tau = in.dbg_tau;
        pp.dbg_union_rows = dbg ? dbg->union_rows : nullptr;
        static std::atomic<unsigned long long> done_plan;
        if ((err = ensure_dynamic_smem((const void *)latent_plan_kernel, (int)sizeof(LatentPlanSmem), done_plan)) != cudaSuccess)
            return note_cuda_failure(err, "latent plan attribute");
        if ((err = launch_kernel(latent_plan_kernel, dim3(geom->n_seqs), dim3(kLpThreads), sizeof(LatentPlanSmem), s, pp)) != cudaSuccess)
            return note_cuda_failure(err, "latent plan launch");
        ++launches;
    }
    rc = latent_attend_and_merge(geom, teams, L, ws, q, suffix_rows, suffix_len_dev, suffix_cap, scale, out, status, false, mask,
                                 launches, s, dbg ? reinterpret_cast<unsigned long long *>(dbg->trace) : nullptr);
    note_launch_count(launches);
    return rc;
}

int santapp_latent_dense_decode_attn(const santapp_latent_geom *geom, const santapp_latent_teams *teams, const void *q,
                                     const void *suffix_rows, const int32_t *suffix_len_dev, int32_t suffix_cap, float scale,
                                     float *out, void *workspace, size_t workspace_bytes, santapp_stream stream)
{
    note_launch_count(0);
    int rc = check_latent_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if ((rc = check_latent_teams(geom, teams)) != SANTAPP_OK) return rc;
    if (!q || !out || !workspace) return SANTAPP_ERR_INVALID_ARG;
    if (lat_misaligned(q, 16) || lat_misaligned(out, 16) || lat_misaligned(workspace, 16) || lat_misaligned(suffix_rows, 16)
        || lat_misaligned(suffix_len_dev, 4))
        return SANTAPP_ERR_INVALID_ARG;
    if (suffix_cap < 0) return SANTAPP_ERR_INVALID_ARG;
    if (suffix_cap > 0 && suffix_len_dev && !suffix_rows) return SANTAPP_ERR_INVALID_ARG;
    if (!(scale > 0.f) || isinf(scale)) return SANTAPP_ERR_INVALID_ARG;
    if ((int64_t)geom->n_seqs * (int64_t)suffix_cap + teams->rows_total >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    const LatentLayout L = latent_layout(geom, teams, 1, 0, true);
    if (workspace_bytes < L.total) return SANTAPP_ERR_WORKSPACE_TOO_SMALL;
    int launches = 0;
    rc = latent_attend_and_merge(geom, teams, L, static_cast<char *>(workspace), q, suffix_rows, suffix_len_dev, suffix_cap, scale,
                                 out, nullptr, true, SANTAPP_STAGE_ATTEND | SANTAPP_STAGE_MERGE, launches,
                                 static_cast<cudaStream_t>(stream));
    note_launch_count(launches);
    return rc;
}

}  // extern "C"
