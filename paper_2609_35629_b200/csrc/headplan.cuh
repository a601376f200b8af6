// Sampling of one query head (Algorithm 1: Gumbel-top-K over the perturbed routing scores and the
// conditional inclusion correction of Eq. method-inclusion), as a block-wide device function.
//
// The scorer leaves fp32 perturbed scores Y32 for every (head, team) and the inputs of a bound E on
// |Y32 - Y| against the exact fp64 score Y. The sample must be the fp64 one, so:
//   1. the block reads the head's whole score row once (each thread keeps its scores in registers)
//      and finds a lower bound t on the (K+1)-st largest Y32 from a histogram of the scores;
//   2. every team with Y32 >= t - 2E is a candidate: that set contains the K+1 largest exact
//      scores (if K+1 teams have Y32 >= t they have Y >= t - E, so the (K+1)-st largest Y is at
//      least t - E, and a team with Y above that has Y32 >= t - 2E);
//   3. the candidates are re-evaluated exactly in fp64 (dot product of the 16-bit values, log n_g,
//      Gumbel from the same Philox word) and ranked by (Y descending, team id ascending);
//   4. the K largest are the sample, the next one is tau, c_g = 1 - exp(-exp(phi_g - tau)).
// At most kCandCap candidates are held at a time; when more qualify the teams are walked in ranges
// of kCandCap with a running top-(K+1) list, so any number of candidates fits in shared memory.
// Output per head: the K sampled team ids in descending Y, log c_g and the packed row range of each.
#pragma once

#include <math_constants.h>

#include <stddef.h>

#include "common.cuh"

namespace santapp {

constexpr int kMaxHeadWarps = 32;        // blocks of up to 1024 threads
constexpr int kCandCap = 512;           // candidates refined at a time
constexpr int kListCap = 260;           // running top list: K + 1 <= 257 entries (+ pad); K <= 128 for K/V rows, <= 256 for shared-latent rows
constexpr int kDotLanes = 8;            // threads that share one candidate's dot product
constexpr int kWindow = 255;            // histogram bins per pass of the bound

// kDim: values per routing key (128 for K rows, 576 for shared-latent rows); a multiple of 64.
template <int kDim>
struct alignas(16) HeadSmemT {
    double q64[kDotLanes][kDim / kDotLanes + 2];   // query in fp64: [slice of kDim / 8 dims][+ pad] (pad: conflict-free LDS.128)
    double cand_y[kCandCap + 2];        // dot products, then exact Y; read in pairs
    double cand_phi[kCandCap];          // log n_g, then phi_g
    double cand_g[kCandCap];            // Gumbel term
    double list_y[2][kListCap];
    double list_phi[2][kListCap];
    int list_id[2][kListCap];
    int cand_id[kCandCap];
    int2 cand_rows[kCandCap];           // first packed row (local to the sequence) and size of the candidate's team
    int2 list_rows[2][kListCap];
    int hist[256];
    float red_max[kMaxHeadWarps], red_sum[kMaxHeadWarps];
    int n_cand, bound_bin, bound_below, bound_total;
    uint32_t taken[(kListCap + 31) / 32];   // ranks handed out by the integer ranking pass
    int need_exact;                     // two entries met on one rank: rank again on whole scores
};
using HeadSmem = HeadSmemT<kHeadDim>;
static_assert(offsetof(HeadSmemT<128>, cand_g) % 16 == 0 && offsetof(HeadSmemT<576>, cand_g) % 16 == 0,
              "the ranking pass reads the keys kept in cand_g sixteen bytes at a time");

// Guard on |Y32 - Y|: tensor-core accumulation of exact 16-bit products in fp32 (relative to the sum
// of magnitudes, bounded by scale * |q|_1 * max|l|), plus the fp32 logarithm and Gumbel terms.
__device__ __forceinline__ float score_guard(double scale, double q_l1, float k_abs_max)
{
    return (float)(2.5e-4 * scale * q_l1 * (double)k_abs_max + 1e-3);
}

// Global histogram bin of a score below the top: floor((top - v) * 4), saturated (the same in every pass).
__device__ __forceinline__ int score_bin(float top, float v)
{
    const float d = (top - v) * 4.f;
    return d >= 1073741824.f ? (1 << 30) : (int)d;
}

// Block: sample of head hq = (sequence, query head). All kT threads call; the first half of the
// block's warps compute dot products, the second half the Gumbel terms. Nothing is done (and
// nothing written) when K >= M: every team is then read with c = 1 and nothing is drawn.
// kScoreRegs: 16-byte pieces of the score row a thread keeps in registers.
template <int kT, int kScoreRegs, bool kHalf, int kDim = kHeadDim>
__device__ __forceinline__ void select_head(const PlanInputs &in, int hq, HeadSmemT<kDim> &sm)
{
    static_assert(kDim % 64 == 0, "eight lanes share a key, each takes whole 16-byte pieces");
    constexpr bool kAllDot = kDim > 128;
    constexpr int kHeadWarps = kT / 32, kDotWarps = kAllDot ? kHeadWarps : kHeadWarps / 2;
    constexpr int kSlice = kDim / kDotLanes;                          // dims per lane of a dot product
    constexpr int kPieces = kSlice / 8;                               // 16-byte pieces per lane
    constexpr int kQRegs = (kDim + kT - 1) / kT;                      // query values a thread converts
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = hq / in.bv.n_q, hh = hq - b * in.bv.n_q;            // hh = j * G + h
    const int j = hh / in.bv.group;

    // ---- the head's scores (registers), the query in fp64, |q|_1, the largest score ----
    // piece tid + i * kT of the row, for i < kScoreRegs, lives in yv[i]; rows longer than that are
    // read again from global memory in every pass (L2 hits). The row's address needs no table, so
    // these loads leave before anything else; what lies behind the pair's last team is masked later.
    const float *y32 = in.y32 + ((size_t)hh * in.bv.n_seqs + b) * in.y_stride;             // 16-byte aligned
    const float4 *y4 = reinterpret_cast<const float4 *>(y32);
    const int n4_row = (int)(in.y_stride >> 2);
    float4 yv[kScoreRegs];
    const float4 kNone = make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
#pragma unroll
    for (int i = 0; i < kScoreRegs; ++i) {
        const int at = tid + i * kT;
        yv[i] = at < n4_row ? __ldcg(y4 + at) : kNone;
    }
    float q_val[kQRegs];
#pragma unroll
    for (int i = 0; i < kQRegs; ++i)
        q_val[i] = tid + i * kT < kDim ? elem_to_float<kHalf>(in.q[(size_t)hq * kDim + tid + i * kT]) : 0.f;
    const float k_abs_max = in.rep_abs_max[(size_t)j * in.bv.n_seqs + b];

    const int64_t team0 = in.bv.seq_team_off[b];
    const int M = pair_team_count(in.bv, b, j);
    const int K = in.n_sample;
    if (K >= M) return;
    trace_mark(in.trace, 1, 7);
    const uint32_t step = in.step + (in.step_dev ? *in.step_dev : 0u);
    const uint16_t *rep = in.rep_keys + ((size_t)j * in.bv.teams_total + team0) * kDim;
    const int32_t *csr = in.team_row_start + (size_t)j * (in.bv.teams_total + in.bv.n_seqs) + team0 + b;
    const int n4 = (M + 3) >> 2;                                      // 16-byte pieces that hold teams
    const int need = K + 1;

    // f(x, team, valid) for every score slot this thread owns, the same number of calls in every
    // thread of the block (so f may use warp-wide votes); x = -inf where valid is false
    auto each_score = [&](auto &&f) {
#pragma unroll
        for (int i = 0; i < kScoreRegs; ++i) {
            if (4 * i * kT >= M) break;                               // the same for every thread: no team in this piece or later ones
            const int at = tid + i * kT;
            const float4 v = yv[i];
            f(4 * at < M ? v.x : -CUDART_INF_F, 4 * at, 4 * at < M);
            f(4 * at + 1 < M ? v.y : -CUDART_INF_F, 4 * at + 1, 4 * at + 1 < M);
            f(4 * at + 2 < M ? v.z : -CUDART_INF_F, 4 * at + 2, 4 * at + 2 < M);
            f(4 * at + 3 < M ? v.w : -CUDART_INF_F, 4 * at + 3, 4 * at + 3 < M);
        }
        for (int base = kScoreRegs * kT; base < n4; base += kT) {
            const int at = base + tid;
            const float4 v = at < n4 ? __ldcg(y4 + at) : kNone;
            f(4 * at < M ? v.x : -CUDART_INF_F, 4 * at, 4 * at < M);
            f(4 * at + 1 < M ? v.y : -CUDART_INF_F, 4 * at + 1, 4 * at + 1 < M);
            f(4 * at + 2 < M ? v.z : -CUDART_INF_F, 4 * at + 2, 4 * at + 2 < M);
            f(4 * at + 3 < M ? v.w : -CUDART_INF_F, 4 * at + 3, 4 * at + 3 < M);
        }
    };
    {
        float a = 0.f, top = -CUDART_INF_F;
#pragma unroll
        for (int i = 0; i < kQRegs; ++i) a += fabsf(q_val[i]);
        each_score([&](float x, int, bool) { top = fmaxf(top, x); });
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
            top = fmaxf(top, __shfl_xor_sync(0xFFFFFFFFu, top, o));
        }
        trace_mark(in.trace, 1, 8);
        __syncthreads();                                              // the shared structure is free (block reuse)
#pragma unroll
        for (int i = 0; i < kQRegs; ++i) {
            const int d = tid + i * kT;
            if (d < kDim) sm.q64[d / kSlice][d % kSlice] = (double)q_val[i];
        }
        if (lane == 0) { sm.red_sum[warp] = a; sm.red_max[warp] = top; }
        if (tid == 0) sm.n_cand = 0;
        for (int i = tid; i < 256; i += kT) sm.hist[i] = 0;
    }
    __syncthreads();
    trace_mark(in.trace, 1, 2);
    float q_l1 = 0.f, top = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < kHeadWarps; ++w) { q_l1 += sm.red_sum[w]; top = fmaxf(top, sm.red_max[w]); }
    const float guard = score_guard(in.scale, (double)q_l1 * 1.001, k_abs_max);

    // ---- 1. lower bound on the need-th largest score ----
    // Counted are the maxima of groups of 16 teams (of 4 teams, or single scores, when there are
    // too few groups to find `need` of them): `need` group maxima above an edge are `need`
    // distinct teams above it. A maximum v falls in global bin floor((top - v) * 4); one pass counts
    // a window of 255 bins (bin 255 of the table counts everything below the window). The first bin
    // at which the running count reaches `need` gives the edge. Windows further down are visited
    // only when outliers at the top leave the first one short.
    const int level = (M >> 4) >= 2 * need ? 2 : (n4 >= 2 * need ? 1 : 0);
    float t_lb = -CUDART_INF_F;
    {
        int above = 0;
        for (int win = 0; win < 16 * kWindow; win += kWindow) {      // 1020 units below the top, then give up
            if (win > 0) {
                __syncthreads();
                for (int i = tid; i < 256; i += kT) sm.hist[i] = 0;
                __syncthreads();
            }
            auto count = [&](float x) {
                const int gb = score_bin(top, x);
                if (gb >= win) atomicAdd(&sm.hist[min(gb - win, kWindow)], 1);
            };
            float grp = -CUDART_INF_F;
            bool any = false;
            each_score([&](float x, int team, bool valid) {
                if (level == 0) {
                    if (valid) count(x);
                } else {
                    grp = fmaxf(grp, x);
                    any = any || valid;
                    if ((team & 3) == 3) {                            // the piece is complete
                        if (level == 2) {                             // four neighbouring lanes hold one group of 16
                            grp = fmaxf(grp, __shfl_xor_sync(0xFFFFFFFFu, grp, 1));
                            grp = fmaxf(grp, __shfl_xor_sync(0xFFFFFFFFu, grp, 2));
                            any = __shfl_sync(0xFFFFFFFFu, (int)any, lane & ~3) != 0 && (lane & 3) == 0;
                        }
                        if (any) count(grp);
                        grp = -CUDART_INF_F;
                        any = false;
                    }
                }
            });
            trace_mark(in.trace, 1, 9);
            __syncthreads();
            trace_mark(in.trace, 1, 10);
            if (warp == 0) {
                // lane l owns bins 8 l .. 8 l + 7 of the window; bin 255 holds everything below it
                int local[8], sum = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) { local[i] = sm.hist[lane * 8 + i]; sum += local[i]; }
                int incl = sum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += t;
                }
                int bin = 256, acc = above + incl - sum;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    acc += local[i];
                    if (acc >= need && bin == 256) bin = lane * 8 + i;
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) bin = min(bin, __shfl_xor_sync(0xFFFFFFFFu, bin, o));
                if (lane == 31) { sm.bound_bin = bin; sm.bound_below = local[7]; sm.bound_total = incl; }
            }
            trace_mark(in.trace, 1, 11);
            __syncthreads();
            const int bin = sm.bound_bin, below_all = sm.bound_below, total = sm.bound_total;
            if (bin < kWindow) {                                    // lower edge, minus the rounding of the binning
                t_lb = top - (float)(win + bin + 1) * 0.25f * (1.f + 1e-6f) - 1e-4f;
                break;
            }
            if (below_all == 0) break;
            above += total - below_all;
        }
    }
    const float t_lo = t_lb - 2.f * guard;
    trace_mark(in.trace, 1, 3);

    // ---- 2. candidates: teams whose score reaches t_lo; a warp reserves its slots with one atomic ----
    {
        int cnt = 0;
        each_score([&](float x, int, bool valid) { cnt += __popc(__ballot_sync(0xFFFFFFFFu, valid && x >= t_lo)); });
        int base = 0;
        if (lane == 0 && cnt > 0) base = atomicAdd(&sm.n_cand, cnt);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        each_score([&](float x, int team, bool valid) {
            const bool mine = valid && x >= t_lo;
            const uint32_t votes = __ballot_sync(0xFFFFFFFFu, mine);
            if (mine) {
                const int slot = base + __popc(votes & ((1u << lane) - 1u));
                if (slot < kCandCap) sm.cand_id[slot] = team;
            }
            base += __popc(votes);
        });
    }
    __syncthreads();
    trace_mark(in.trace, 1, 4);
    const bool fits = sm.n_cand <= kCandCap;
    const int n_ranges = fits ? 1 : (M + kCandCap - 1) / kCandCap;

    int cur = 0, n_list = 0;
    for (int r = 0; r < n_ranges; ++r) {
        if (!fits) {                                                  // teams [r, r + 1) * kCandCap
            __syncthreads();
            if (tid == 0) sm.n_cand = 0;
            __syncthreads();
            for (int t = r * kCandCap + tid; t < min(M, (r + 1) * kCandCap); t += kT) {
                if (__ldcg(y32 + t) >= t_lo) sm.cand_id[atomicAdd(&sm.n_cand, 1)] = t;       // at most kCandCap teams in a range
            }
            __syncthreads();
        }
        const int n_cand = sm.n_cand;

        // ---- 3a. exact terms: dot products on the first half of the warps (8 lanes per candidate, kDim / 8 dims each),
        //          log n_g and the Gumbel term on the other warps (one thread per candidate) ----
        // Long keys (kAllDot): every warp takes part in the dot products (their round trips to memory
        // are the longest chain of the kernel), then every thread takes a candidate's other terms.
        if (kAllDot || warp < kDotWarps) {
            const int sub = lane & (kDotLanes - 1);
            const double *qs = sm.q64[sub];
            // a few candidates per thread group at a time: all their key pieces are requested before
            // the first product, so a chunk costs one memory round trip
            constexpr int kPerPass = kDotWarps * 32 / kDotLanes, kChunk = kPieces > 2 ? 1 : (kT >= 512 ? 2 : 4);
            for (int c0 = 0; c0 < n_cand; c0 += kPerPass * kChunk) {
                uint4 w[kChunk][kPieces];
#pragma unroll
                for (int u = 0; u < kChunk; ++u) {
                    const int cand = c0 + u * kPerPass + (tid >> 3);
                    if (cand < n_cand) {
                        const uint4 *kr = reinterpret_cast<const uint4 *>(rep + (size_t)sm.cand_id[cand] * kDim) + sub * kPieces;
#pragma unroll
                        for (int pc = 0; pc < kPieces; ++pc) w[u][pc] = __ldg(kr + pc);
                    } else {
#pragma unroll
                        for (int pc = 0; pc < kPieces; ++pc) w[u][pc] = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
#pragma unroll
                for (int u = 0; u < kChunk; ++u) {
                    const int cand = c0 + u * kPerPass + (tid >> 3);
                    double d0 = 0.0, d1 = 0.0;                        // even and odd dims of the slice, in order
#pragma unroll
                    for (int pc = 0; pc < kPieces; ++pc) {
                        const uint4 wv = w[u][pc];
                        d0 = fma((double)elem_lo<kHalf>(wv.x), qs[8 * pc + 0], d0);
                        d1 = fma((double)elem_hi<kHalf>(wv.x), qs[8 * pc + 1], d1);
                        d0 = fma((double)elem_lo<kHalf>(wv.y), qs[8 * pc + 2], d0);
                        d1 = fma((double)elem_hi<kHalf>(wv.y), qs[8 * pc + 3], d1);
                        d0 = fma((double)elem_lo<kHalf>(wv.z), qs[8 * pc + 4], d0);
                        d1 = fma((double)elem_hi<kHalf>(wv.z), qs[8 * pc + 5], d1);
                        d0 = fma((double)elem_lo<kHalf>(wv.w), qs[8 * pc + 6], d0);
                        d1 = fma((double)elem_hi<kHalf>(wv.w), qs[8 * pc + 7], d1);
                    }
                    double d = d0 + d1;
                    d += __shfl_xor_sync(0xFFFFFFFFu, d, 1);
                    d += __shfl_xor_sync(0xFFFFFFFFu, d, 2);
                    d += __shfl_xor_sync(0xFFFFFFFFu, d, 4);
                    if (cand < n_cand && sub == 0) sm.cand_y[cand] = d;
                }
            }
        }
        if (kAllDot || warp >= kDotWarps) {
            for (int i = kAllDot ? tid : tid - kDotWarps * 32; i < n_cand; i += kAllDot ? kT : kT - kDotWarps * 32) {
                const int id = sm.cand_id[i];
                const int r_lo = csr[id];
                const int n_g = csr[id + 1] - r_lo;
                sm.cand_rows[i] = make_int2(r_lo, n_g);
                const uint4 words = philox4x32_10(
                    make_uint4((uint32_t)id >> 2, step, (uint32_t)hh, in.stream_base + (uint32_t)b), in.seed_lo, in.seed_hi);
                sm.cand_g[i] = gumbel_from_word(pick_word(words, id & 3));
                sm.cand_phi[i] = log((double)n_g);
            }
        }
        __syncthreads();
        trace_mark(in.trace, 1, 5);
        for (int i = tid; i < n_cand; i += kT) {
            const double phi = sm.cand_phi[i] + sm.cand_y[i] * in.scale;
            sm.cand_phi[i] = phi;
            sm.cand_y[i] = phi + sm.cand_g[i];
        }
        __syncthreads();

        // ---- 3b. merge with the running list: keep the K + 1 largest by (Y descending, id ascending) ----
        // Ranking is all comparisons, and the count of them is what this step costs. First pass, on
        // integers: every entry (list, then candidates) gets the upper half of its score's integer
        // key (same order as the score); a thread holds one entry and walks all keys, four per
        // broadcast load, counting the larger ones. Two entries whose scores agree in the upper half
        // of the key land on the same rank; the second one to arrive sees the rank taken and asks for
        // the exact pass below, which ranks on whole scores and ids as the paper's order says.
        const int n_all = n_list + n_cand;
        uint32_t *key_hi = reinterpret_cast<uint32_t *>(sm.cand_g);   // (the Gumbel terms are used up)
        const int n_pad = (n_all + 3) & ~3;
        for (int e = tid; e < n_pad; e += kT) {
            uint32_t h = 0u;                                          // padding: below every key
            if (e < n_all) h = (uint32_t)(sortable_key(e < n_list ? sm.list_y[cur][e] : sm.cand_y[e - n_list]) >> 32);
            key_hi[e] = h;
        }
        if (tid < (kListCap + 31) / 32) sm.taken[tid] = 0u;
        if (tid == 0) sm.need_exact = 0;
        __syncthreads();
        for (int e = tid; e < n_all; e += kT) {
            const uint32_t yh = key_hi[e];
            int rank = 0;
#pragma unroll 2
            for (int a = 0; a < n_pad; a += 4) {
                const uint4 w = *reinterpret_cast<const uint4 *>(key_hi + a);
                rank += (w.x > yh) + (w.y > yh) + (w.z > yh) + (w.w > yh);
            }
            if (rank <= K) {
                const uint32_t bit = 1u << (rank & 31);
                if (atomicOr(&sm.taken[rank >> 5], bit) & bit) sm.need_exact = 1;
                else if (e < n_list) {
                    sm.list_y[cur ^ 1][rank] = sm.list_y[cur][e];
                    sm.list_phi[cur ^ 1][rank] = sm.list_phi[cur][e];
                    sm.list_id[cur ^ 1][rank] = sm.list_id[cur][e];
                    sm.list_rows[cur ^ 1][rank] = sm.list_rows[cur][e];
                } else {
                    sm.list_y[cur ^ 1][rank] = sm.cand_y[e - n_list];
                    sm.list_phi[cur ^ 1][rank] = sm.cand_phi[e - n_list];
                    sm.list_id[cur ^ 1][rank] = sm.cand_id[e - n_list];
                    sm.list_rows[cur ^ 1][rank] = sm.cand_rows[e - n_list];
                }
            }
        }
        __syncthreads();
        if (sm.need_exact) {
            // eight lanes share an entry: each counts the entries ahead of it in its share of the scores
            const int sub = lane & 7;
            for (int e0 = 0; e0 < n_all; e0 += kT / 8) {                  // uniform trip count: the votes below are warp-wide
                const int e = e0 + (tid >> 3);
                const bool live = e < n_all;
                double y = 0.0, phi = 0.0;
                int id = 0;
                int2 rows = make_int2(0, 0);
                if (live) {
                    if (e < n_list) { y = sm.list_y[cur][e]; phi = sm.list_phi[cur][e]; id = sm.list_id[cur][e]; rows = sm.list_rows[cur][e]; }
                    else { y = sm.cand_y[e - n_list]; phi = sm.cand_phi[e - n_list]; id = sm.cand_id[e - n_list]; rows = sm.cand_rows[e - n_list]; }
                }
                // rank = entries ahead of this one (larger score, or the same score and a smaller id);
                // ids are looked at only when some other entry has exactly the same score
                int rank = 0, same = 0;
                if (live) {
                    for (int a = sub; a < n_list; a += 8) {
                        const double w = sm.list_y[cur][a];
                        rank += (w > y);
                        same += (w == y);
                    }
                    for (int a = sub; a < n_cand; a += 8) {
                        const double w = sm.cand_y[a];
                        rank += (w > y);
                        same += (w == y);
                    }
                }
                same += __shfl_xor_sync(0xFFFFFFFFu, same, 1);
                same += __shfl_xor_sync(0xFFFFFFFFu, same, 2);
                same += __shfl_xor_sync(0xFFFFFFFFu, same, 4);
                if (live && same > 1) {
                    for (int a = sub; a < n_list; a += 8) rank += (sm.list_y[cur][a] == y && sm.list_id[cur][a] < id);
                    for (int a = sub; a < n_cand; a += 8) rank += (sm.cand_y[a] == y && sm.cand_id[a] < id);
                }
                rank += __shfl_xor_sync(0xFFFFFFFFu, rank, 1);
                rank += __shfl_xor_sync(0xFFFFFFFFu, rank, 2);
                rank += __shfl_xor_sync(0xFFFFFFFFu, rank, 4);
                if (live && sub == 0 && rank <= K) {
                    sm.list_y[cur ^ 1][rank] = y;
                    sm.list_phi[cur ^ 1][rank] = phi;
                    sm.list_id[cur ^ 1][rank] = id;
                    sm.list_rows[cur ^ 1][rank] = rows;
                }
            }
        }
        n_list = min(K + 1, n_list + n_cand);
        cur ^= 1;
        __syncthreads();
    }

    trace_mark(in.trace, 1, 6);
    // ---- 4. corrections ----
    // Fewer than K + 1 ranked teams can only mean scores that do not compare (non-finite inputs):
    // the sample is completed with the first teams so that every index handed on is valid, and
    // the status word says so.
    const bool short_list = n_list < K + 1;
    const double tau = short_list ? __longlong_as_double(0x7FF8000000000000ll) : sm.list_y[cur][K];
    if (short_list && tid == 0 && in.status) atomicOr(in.status, 2);
    for (int a = tid; a < K; a += kT) {
        int id;
        float logc;
        int2 rows;
        if (a < n_list && !short_list) {
            // c = 1 - exp(-exp(phi - tau)), in fp32 from the exact difference: log c changes by at most
            // the error of its argument x = phi - tau (slope <= 1), |x| < 64, so the result is within
            // a few 1e-6 of the fp64 value, the order of its own rounding to fp32
            const float x = (float)(sm.list_phi[cur][a] - tau);
            logc = logf(-expm1f(-expf(x)));
            id = sm.list_id[cur][a];
            rows = sm.list_rows[cur][a];
        } else {
            id = a;                                                       // K < M: a valid team
            logc = 0.f;
            rows = make_int2(csr[a], csr[a + 1] - csr[a]);
        }
        in.sel_team[(size_t)hq * K + a] = id;
        in.sel_logc[(size_t)hq * K + a] = logc;
        in.sel_rows[(size_t)hq * K + a] = rows;
        if (in.dbg_sel_idx) in.dbg_sel_idx[(size_t)hq * K + a] = id;
        if (in.dbg_sel_logc) in.dbg_sel_logc[(size_t)hq * K + a] = logc;
    }
    if (tid == 0 && in.dbg_tau) in.dbg_tau[hq] = tau;
}

}  // namespace santapp
