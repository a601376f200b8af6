// Sampling and read plan of one (sequence, KV head) pair, as a block-wide device function
// (Algorithm 1: Gumbel-top-K over the perturbed routing scores, the conditional inclusion
// correction of Eq. method-inclusion, and the GQA union of the heads' selections).
//
// The scorer leaves fp32 perturbed scores Y32 for every (head, team) together with a bound E on
// |Y32 - Y| against the exact fp64 score Y. The sample must be the fp64 one, so per head:
//   1. a lower bound t on the (K+1)-st largest Y32 (from the maxima of 16-team blocks);
//   2. every team with Y32 >= t - 2E is a candidate: that set contains the K+1 largest exact
//      scores (if K+1 teams have Y32 >= t they have Y >= t - E, so the (K+1)-st largest Y is at
//      least t - E, and a team with Y above that has Y32 >= t - 2E);
//   3. the candidates are re-evaluated exactly in fp64 (dot product of bf16 values, log n_g,
//      Gumbel from the same Philox word) and ranked by (Y descending, team id ascending);
//   4. the K largest are the sample, the next one is tau, c_g = 1 - exp(-exp(phi_g - tau)).
// Candidates are processed at most kCandCap at a time with a running top-(K+1) list, so any
// number of candidates is handled in bounded shared memory.
// The plan is the union of the heads' samples in team order with head masks, per-head
// log2(e) * log c_g, segment row prefix, and the exact suffix as a last segment.
#pragma once

#include <math_constants.h>

#include "common.cuh"

namespace santapp {

constexpr int kPlanThreads = 384;       // block size of every kernel that builds a pair plan
constexpr int kPlanWarps = kPlanThreads / 32;
constexpr int kCandCap = 512;           // candidates of one head refined at a time
constexpr int kListCap = 132;           // running top list: K + 1 <= 129 entries
constexpr int kEntCap = 1024;           // G * K entries of a plan
constexpr int kSegMax = 1025;           // segments of a plan (entries + suffix)
constexpr int kBitmapWords = kMaxTeamsPerSeq / 32;

struct alignas(16) HeadScratch {
    int n_cand, n_list, n_ranges, range_len;
    float t_lo;                         // candidate threshold on Y32 (lower bound minus guard)
    float pad[3];
    int hist[256];                      // block maxima by distance from the largest, for the lower bound
    int cand_id[kCandCap];
    double cand_y[kCandCap + 2];          // read in pairs: an odd count is padded with -inf
    double cand_phi[kCandCap];
    int list_id[2][kListCap];
    double list_y[2][kListCap];
    double list_phi[2][kListCap];
};

template <int G>
struct alignas(16) PlanScratch {
    double q64[G][kHeadDim];
    HeadScratch head[G];
    int ent_key[kEntCap];               // team * 8 + head
    float ent_logc[kEntCap];
    uint32_t bitmap[kBitmapWords];
    int wprefix[kBitmapWords];
    int seg_rows[kSegMax];
    int scan[33];
    double tau[kMaxGroup];
    int misc[8];
};

// Guard on |Y32 - Y|: tensor-core accumulation of exact bf16 products, fp32 log / Gumbel.
__device__ __forceinline__ float score_guard(double scale, double q_l1, float k_abs_max)
{
    return (float)(2.5e-4 * scale * q_l1 * (double)k_abs_max + 1e-3);
}

// Warp: lower bound on the `need`-th largest score of a head from the maxima of its 16-team
// blocks, by histograms: a block maximum v falls in global bin floor((top - v) * 4) counted down
// from the largest maximum `top`; one pass counts a window of 255 consecutive bins. The first
// bin at which the running count of block maxima reaches `need` has `need` distinct teams'
// scores above its lower edge, so that edge is at most the `need`-th largest score. Windows
// further down are visited only when an outlier at the top leaves the first one short.
// -inf when there are fewer than `need` blocks.
__device__ __forceinline__ float warp_lower_bound(const float *ym, int nblk, int need, int lane, int *hist)
{
    constexpr float kInvWidth = 4.f;
    constexpr int kWindow = 255;
    if (nblk < need) return -CUDART_INF_F;
    float top = -CUDART_INF_F;
    for (int i0 = lane; i0 < nblk; i0 += 128) {
        float v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = (i0 + 32 * k < nblk) ? __ldg(ym + i0 + 32 * k) : -CUDART_INF_F;
        top = fmaxf(top, fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3])));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) top = fmaxf(top, __shfl_xor_sync(0xFFFFFFFFu, top, o));
    int above = 0;                                             // maxima in the windows already passed
    for (int win = 0; win < 16 * kWindow; win += kWindow) {   // 1020 units below the top, then give up
#pragma unroll
        for (int i = 0; i < 8; ++i) hist[lane * 8 + i] = 0;
        __syncwarp();
        for (int i0 = lane; i0 < nblk; i0 += 128) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (i0 + 32 * k < nblk) {
                    const float d = (top - __ldg(ym + i0 + 32 * k)) * kInvWidth;   // cached by the first pass
                    const int gb = d >= 1073741824.f ? (1 << 30) : (int)d;         // global bin, the same in every pass
                    if (gb >= win) atomicAdd(&hist[min(gb - win, kWindow)], 1);
                }
            }
        }
        __syncwarp();
        // lane l owns bins 8 l .. 8 l + 7 of the window; bin 255 holds everything below it
        int local[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { local[i] = hist[lane * 8 + i]; sum += local[i]; }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        int bin = 256;                                         // first bin whose running count reaches need
        int acc = above + incl - sum;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            acc += local[i];
            if (acc >= need && bin == 256) bin = lane * 8 + i;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) bin = min(bin, __shfl_xor_sync(0xFFFFFFFFu, bin, o));
        const int below = __shfl_sync(0xFFFFFFFFu, local[7], 31);
        const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        __syncwarp();
        if (bin < kWindow)                                     // lower edge, minus the rounding of the binning
            return top - (float)(win + bin + 1) * (1.f / kInvWidth) * (1.f + 1e-6f) - 1e-4f;
        if (below == 0) break;
        above += total - below;
    }
    return -CUDART_INF_F;
}

// Warp: append the teams of blocks [blk_lo, blk_hi) with y >= t_lo to the head's candidate list
// (any order; the exact ranking does not depend on it). hs.n_cand counts every hit, also those
// beyond kCandCap, so the caller can tell an overflow.
__device__ __forceinline__ void warp_append_blocks(const float *y, const float *ym, int blk_lo, int blk_hi, int M, float t_lo,
                                          HeadScratch &hs, int lane)
{
    // four blocks per lane at a time: block maxima first, then the scores of the blocks that can
    // hold a candidate, all loads of a batch in flight together
    for (int blk0 = blk_lo + lane; blk0 < blk_hi; blk0 += 128) {
        bool hit[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) hit[k] = (blk0 + 32 * k < blk_hi) && (__ldg(ym + blk0 + 32 * k) >= t_lo);
        float v[4][16];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int g0 = (blk0 + 32 * k) * 16;
#pragma unroll
            for (int i = 0; i < 16; ++i) v[k][i] = (hit[k] && g0 + i < M) ? __ldg(y + g0 + i) : -CUDART_INF_F;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int g0 = (blk0 + 32 * k) * 16;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                if (hit[k] && g0 + i < M && v[k][i] >= t_lo) {
                    const int slot = atomicAdd(&hs.n_cand, 1);
                    if (slot < kCandCap) hs.cand_id[slot] = g0 + i;
                }
            }
        }
    }
}

// Warp: candidates of a whole head in two steps: the blocks whose maximum reaches t_lo are
// listed first (ballot compaction over the block maxima, which the bound left in cache), then
// the scores of the listed blocks are fetched as independent 16-byte loads, several per lane in
// flight. Returns false when more than kCandCap blocks qualify (the caller then walks ranges).
__device__ __forceinline__ bool warp_append_listed(const float *y, const float *ym, int nblk, int M, float t_lo,
                                                   HeadScratch &hs, int lane)
{
    int *blk_list = reinterpret_cast<int *>(hs.cand_y);        // free until the exact scores are written
    int n_blk = 0;
    for (int i0 = 0; i0 < nblk; i0 += 32) {
        const int blk = i0 + lane;
        const bool hit = blk < nblk && __ldg(ym + blk) >= t_lo;
        const unsigned m = __ballot_sync(0xFFFFFFFFu, hit);
        if (hit) {
            const int slot = n_blk + __popc(m & ((1u << lane) - 1u));
            if (slot < kCandCap) blk_list[slot] = blk;
        }
        n_blk += __popc(m);
    }
    if (n_blk > kCandCap) return false;
    __syncwarp();
    const int n_item = n_blk * 4;                              // (listed block, quarter of its 16 scores)
    for (int it0 = lane; it0 < n_item; it0 += 128) {
        float4 v[4];
        int g0[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int it = it0 + 32 * k;
            g0[k] = -1;
            if (it < n_item) {
                g0[k] = blk_list[it >> 2] * 16 + (it & 3) * 4;
                // rows of Y32 start at multiples of 4 teams only when team0 does; load scalars otherwise
                v[k].x = g0[k] < M ? __ldg(y + g0[k]) : -CUDART_INF_F;
                v[k].y = g0[k] + 1 < M ? __ldg(y + g0[k] + 1) : -CUDART_INF_F;
                v[k].z = g0[k] + 2 < M ? __ldg(y + g0[k] + 2) : -CUDART_INF_F;
                v[k].w = g0[k] + 3 < M ? __ldg(y + g0[k] + 3) : -CUDART_INF_F;
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (g0[k] < 0) continue;
            const float vv[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (g0[k] + i < M && vv[i] >= t_lo) {
                    const int slot = atomicAdd(&hs.n_cand, 1);
                    if (slot < kCandCap) hs.cand_id[slot] = g0[k] + i;
                }
            }
        }
    }
    return true;
}

// Block: plan of `pair` into shared-memory tables (seg_prefix[nseg+1], seg_row, seg_mask) and the
// pair's log c table in global memory (g_logc [kSegMax][8]). All threads call; blockDim.x ==
// kPlanThreads. Returns the number of segments in nseg_out and of rows in rows_out.
template <int G>
__device__ __forceinline__ void build_pair_plan(const PlanInputs &in, int pair, PlanScratch<G> &sc, int *seg_prefix, int *seg_row,
                                uint32_t *seg_mask, float *g_logc, int &nseg_out, int &rows_out, bool write_debug)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = pair / in.bv.n_kv, j = pair - b * in.bv.n_kv;
    const int64_t team0 = in.bv.seq_team_off[b];
    const int M = (int)(in.bv.seq_team_off[b + 1] - team0);
    const int64_t row0 = in.bv.seq_row_off[b];
    const int N = (int)(in.bv.seq_row_off[b + 1] - row0);
    const int K = in.n_sample;
    const int Ke = min(K, M);
    int t_suffix = 0;
    if (in.suffix_len != nullptr && in.suffix_cap > 0) t_suffix = max(0, min(in.suffix_len[b], in.suffix_cap));
    const uint32_t all_heads = (1u << G) - 1u;
    const float kLog2e = 1.4426950408889634f;
    const size_t head0 = (size_t)b * in.bv.n_q + (size_t)j * G;       // first query head of the pair

    __syncthreads();                                                  // scratch and tables are free
    if (Ke == M) {
        // every team is read with correction one; nothing is drawn
        if (tid == 0) {
            seg_prefix[0] = 0;
            seg_row[0] = (int32_t)row0;
            seg_mask[0] = all_heads;
            int nseg = 1, rows = N;
            if (t_suffix > 0) {
                seg_prefix[1] = rows;
                seg_row[1] = pair * in.suffix_cap;
                seg_mask[1] = all_heads | kSrcSuffix;
                rows += t_suffix;
                nseg = 2;
            }
            seg_prefix[nseg] = rows;
            sc.misc[0] = nseg;
            sc.misc[1] = rows;
            if (write_debug && in.dbg_union_rows) in.dbg_union_rows[pair] = N;
        }
        if (tid < 2 * kMaxGroup) g_logc[tid] = 0.f;
        if (write_debug) {
            for (int e = tid; e < G * K; e += kPlanThreads) {
                const int h = e / K, a = e - h * K;
                if (in.dbg_sel_idx) in.dbg_sel_idx[(head0 + h) * K + a] = a < M ? a : -1;
                if (in.dbg_sel_logc) in.dbg_sel_logc[(head0 + h) * K + a] = 0.f;
            }
            if (tid < G && in.dbg_tau) in.dbg_tau[head0 + tid] = __longlong_as_double(0x7FF8000000000000ll);
        }
        __threadfence_block();
        __syncthreads();
        nseg_out = sc.misc[0];
        rows_out = sc.misc[1];
        return;
    }

    const uint32_t step = in.step + (in.step_dev ? *in.step_dev : 0u);
    const uint16_t *rep = in.rep_keys + ((size_t)j * in.bv.teams_total + team0) * kHeadDim;
    const int32_t *csr = in.team_row_start + (size_t)j * (in.bv.teams_total + in.bv.n_seqs) + team0 + b;

    // ---- queries in fp64 (idle warps), guard per head and candidate thresholds (one warp per head) ----
    if (warp >= G) {
        for (int e = tid - 32 * G; e < G * kHeadDim; e += kPlanThreads - 32 * G)
            sc.q64[e >> 7][e & 127] = bf16_to_double(in.q[(head0 + (e >> 7)) * kHeadDim + (e & 127)]);
    } else {
        const int h = warp;
        HeadScratch &hs = sc.head[h];
        float l1 = 0.f;
        for (int d = lane; d < kHeadDim; d += 32) l1 += fabsf(bf16_to_float(in.q[(head0 + h) * kHeadDim + d]));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, o);
        const float guard = score_guard(in.scale, (double)l1 * 1.001, in.rep_abs_max[(size_t)j * in.bv.n_seqs + b]);
        const float *y = in.y32 + ((size_t)j * G + h) * in.bv.teams_total + team0;
        const float *ym = in.ymax + ((size_t)j * G + h) * in.ymax_stride + (team0 >> 4) + b;
        const int nblk = (M + 15) >> 4;
        const float t_lb = warp_lower_bound(ym, nblk, Ke + 1, lane, hs.hist);
        const float t_lo = t_lb - 2.f * guard;
        // candidates in one go if they fit, else ranges of kCandCap teams in the loop below
        if (lane == 0) hs.n_cand = 0;
        __syncwarp();
        const bool listed = warp_append_listed(y, ym, nblk, M, t_lo, hs, lane);
        __syncwarp();
        if (lane == 0) {
            const bool fits = listed && hs.n_cand <= kCandCap;
            hs.t_lo = t_lo;
            hs.n_list = 0;
            hs.range_len = fits ? M : kCandCap;
            hs.n_ranges = fits ? 1 : (M + kCandCap - 1) / kCandCap;
        }
    }
    __syncthreads();
    int n_iter = 1;
#pragma unroll
    for (int h = 0; h < G; ++h) n_iter = max(n_iter, sc.head[h].n_ranges);

    int cur = 0;                                                      // which list buffer is current
    for (int it = 0; it < n_iter; ++it) {
        // a. candidates of this range
        if (warp < G) {
            HeadScratch &hs = sc.head[warp];
            if (hs.n_ranges > 1 && it < hs.n_ranges) {
                const float *y = in.y32 + ((size_t)j * G + warp) * in.bv.teams_total + team0;
                const float *ym = in.ymax + ((size_t)j * G + warp) * in.ymax_stride + (team0 >> 4) + b;
                const int blk_lo = it * (kCandCap / 16), blk_hi = min((M + 15) >> 4, blk_lo + kCandCap / 16);
                if (lane == 0) hs.n_cand = 0;
                __syncwarp();
                warp_append_blocks(y, ym, blk_lo, blk_hi, M, hs.t_lo, hs, lane);
            } else if (it > 0 && lane == 0) {
                hs.n_cand = 0;                                     // single range: done in iteration 0
            }
        }
        __syncthreads();
        // b. exact scores of the candidates (all heads, one thread per candidate)
        int n_tot = 0, cand_off[G + 1];
#pragma unroll
        for (int h = 0; h < G; ++h) { cand_off[h] = n_tot; n_tot += sc.head[h].n_cand; }
        cand_off[G] = n_tot;
        for (int e = tid; e < n_tot; e += kPlanThreads) {
            int h = 0, off = 0;
#pragma unroll
            for (int hh = 1; hh < G; ++hh) {
                const bool ge = e >= cand_off[hh];
                h += ge;
                off = ge ? cand_off[hh] : off;
            }
            HeadScratch &hs = sc.head[h];
            const int i = e - off;
            const int id = hs.cand_id[i];
            const uint4 *kr = reinterpret_cast<const uint4 *>(rep + (size_t)id * kHeadDim);
            const double *qh = sc.q64[h];
            const int r_lo = csr[id], r_hi = csr[id + 1];
            uint4 kw[16];
#pragma unroll
            for (int c4 = 0; c4 < 16; ++c4) kw[c4] = __ldg(kr + c4);
            double d0 = 0.0, d1 = 0.0, d2 = 0.0, d3 = 0.0;            // four chains, summed at the end
#pragma unroll
            for (int c4 = 0; c4 < 16; ++c4) {
                const uint4 w = kw[c4];
                const double *qq = qh + c4 * 8;
                d0 = fma((double)bf16_lo(w.x), qq[0], d0);
                d1 = fma((double)bf16_hi(w.x), qq[1], d1);
                d2 = fma((double)bf16_lo(w.y), qq[2], d2);
                d3 = fma((double)bf16_hi(w.y), qq[3], d3);
                d0 = fma((double)bf16_lo(w.z), qq[4], d0);
                d1 = fma((double)bf16_hi(w.z), qq[5], d1);
                d2 = fma((double)bf16_lo(w.w), qq[6], d2);
                d3 = fma((double)bf16_hi(w.w), qq[7], d3);
            }
            const double dot = (d0 + d1) + (d2 + d3);
            const int n_g = r_hi - r_lo;
            const double phi = log((double)n_g) + dot * in.scale;
            const uint4 words = philox4x32_10(
                make_uint4((uint32_t)id >> 2, step, (uint32_t)(j * G + h), in.stream_base + (uint32_t)b),
                in.seed_lo, in.seed_hi);
            hs.cand_phi[i] = phi;
            hs.cand_y[i] = phi + gumbel_from_word(pick_word(words, id & 3));
            if (i == hs.n_cand - 1) hs.cand_y[i + 1] = -CUDART_INF;
        }
        __syncthreads();
        // c. merge with the running list: keep the Ke + 1 largest by (Y descending, id ascending)
        int ent_off[G + 1], e_tot = 0;
#pragma unroll
        for (int h = 0; h < G; ++h) { ent_off[h] = e_tot; e_tot += sc.head[h].n_list + sc.head[h].n_cand; }
        ent_off[G] = e_tot;
        for (int e = tid; e < e_tot; e += kPlanThreads) {
            int h = 0, off = 0;
#pragma unroll
            for (int hh = 1; hh < G; ++hh) {
                const bool ge = e >= ent_off[hh];
                h += ge;
                off = ge ? ent_off[hh] : off;
            }
            HeadScratch &hs = sc.head[h];
            const int i = e - off;
            const int nl = hs.n_list, nc = hs.n_cand;
            double y, phi;
            int id;
            if (i < nl) { y = hs.list_y[cur][i]; phi = hs.list_phi[cur][i]; id = hs.list_id[cur][i]; }
            else { y = hs.cand_y[i - nl]; phi = hs.cand_phi[i - nl]; id = hs.cand_id[i - nl]; }
            // rank = entries ahead in (Y descending, id ascending); scores are compared two at a
            // time, and ids are looked at only when some other entry has exactly the same score
            int rank = 0, same = 0;
            const double2 *ly = reinterpret_cast<const double2 *>(hs.list_y[cur]);
            const double2 *cy = reinterpret_cast<const double2 *>(hs.cand_y);
#pragma unroll 2
            for (int a = 0; a < (nl + 1) >> 1; ++a) {
                const double2 w = ly[a];
                rank += (w.x > y) + (w.y > y);
                same += (w.x == y) + (w.y == y);
            }
#pragma unroll 2
            for (int a = 0; a < (nc + 1) >> 1; ++a) {
                const double2 w = cy[a];
                rank += (w.x > y) + (w.y > y);
                same += (w.x == y) + (w.y == y);
            }
            if (same > 1) {
                for (int a = 0; a < nl; ++a) rank += (hs.list_y[cur][a] == y && hs.list_id[cur][a] < id);
                for (int a = 0; a < nc; ++a) rank += (hs.cand_y[a] == y && hs.cand_id[a] < id);
            }
            if (rank <= Ke) {
                hs.list_y[cur ^ 1][rank] = y;
                hs.list_phi[cur ^ 1][rank] = phi;
                hs.list_id[cur ^ 1][rank] = id;
            }
        }
        __syncthreads();
        if (tid < G) {
            const int n_new = min(Ke + 1, sc.head[tid].n_list + sc.head[tid].n_cand);
            sc.head[tid].n_list = n_new;
            sc.head[tid].list_y[cur ^ 1][n_new] = -CUDART_INF;
        }
        cur ^= 1;
        __syncthreads();
    }

    // ---- corrections, diagnostics, plan entries ----
    for (int e = tid; e < G * Ke; e += kPlanThreads) {
        const int h = e / Ke, a = e - h * Ke;
        const HeadScratch &hs = sc.head[h];
        const double tau = hs.list_y[cur][Ke];
        const double c = -expm1(-exp(hs.list_phi[cur][a] - tau));     // 1 - exp(-exp(phi - tau))
        const float logc = (float)log(c);
        const int id = hs.list_id[cur][a];
        sc.ent_key[e] = id * kMaxGroup + h;
        sc.ent_logc[e] = logc;
        if (write_debug) {
            if (in.dbg_sel_idx) in.dbg_sel_idx[(head0 + h) * K + a] = id;
            if (in.dbg_sel_logc) in.dbg_sel_logc[(head0 + h) * K + a] = logc;
            if (a == 0 && in.dbg_tau) in.dbg_tau[head0 + h] = tau;
        }
    }
    for (int i = tid; i < (M + 31) / 32; i += kPlanThreads) sc.bitmap[i] = 0u;
    for (int i = tid; i < kSegMax; i += kPlanThreads) seg_mask[i] = 0u;
    __syncthreads();
    const int E = G * Ke;
    for (int e = tid; e < E; e += kPlanThreads) {
        const int team = sc.ent_key[e] >> 3;
        atomicOr(&sc.bitmap[team >> 5], 1u << (team & 31));
    }
    __syncthreads();
    // word prefix of the bitmap -> segment index of a team = teams selected before it
    {
        const int n_words = (M + 31) / 32;
        const int per = (n_words + kPlanThreads - 1) / kPlanThreads;
        const int lo = min(tid * per, n_words), hi = min(lo + per, n_words);
        int sum = 0;
        for (int w = lo; w < hi; ++w) sum += __popc(sc.bitmap[w]);
        int total;
        int run = block_exclusive_scan(sum, sc.scan, total);
        for (int w = lo; w < hi; ++w) { sc.wprefix[w] = run; run += __popc(sc.bitmap[w]); }
        if (tid == 0) sc.misc[0] = total;                             // segments of the prompt
    }
    __syncthreads();
    const int nseg_prompt = sc.misc[0];
    for (int e = tid; e < E; e += kPlanThreads) {
        const int team = sc.ent_key[e] >> 3, h = sc.ent_key[e] & 7;
        const int seg = sc.wprefix[team >> 5] + __popc(sc.bitmap[team >> 5] & ((1u << (team & 31)) - 1u));
        atomicOr(&seg_mask[seg], 1u << h);
        g_logc[(size_t)seg * kMaxGroup + h] = kLog2e * sc.ent_logc[e];
        const int r_lo = csr[team];
        seg_row[seg] = (int32_t)(row0 + r_lo);                        // same value from every selecting head
        sc.seg_rows[seg] = csr[team + 1] - r_lo;
    }
    __syncthreads();
    {
        const int per = (nseg_prompt + kPlanThreads - 1) / kPlanThreads;
        const int lo = min(tid * per, nseg_prompt), hi = min(lo + per, nseg_prompt);
        int sum = 0;
        for (int s = lo; s < hi; ++s) sum += sc.seg_rows[s];
        int total;
        int run = block_exclusive_scan(sum, sc.scan, total);
        for (int s = lo; s < hi; ++s) { seg_prefix[s] = run; run += sc.seg_rows[s]; }
        if (tid == 0) {
            int nseg = nseg_prompt, rows = total;
            if (write_debug && in.dbg_union_rows) in.dbg_union_rows[pair] = total;
            if (t_suffix > 0) {
                seg_prefix[nseg] = rows;
                seg_row[nseg] = pair * in.suffix_cap;
                seg_mask[nseg] = all_heads | kSrcSuffix;
                rows += t_suffix;
                ++nseg;
            }
            seg_prefix[nseg] = rows;
            sc.misc[0] = nseg;
            sc.misc[1] = rows;
        }
        if (t_suffix > 0 && tid < kMaxGroup) g_logc[(size_t)nseg_prompt * kMaxGroup + tid] = 0.f;
    }
    __threadfence_block();
    __syncthreads();
    nseg_out = sc.misc[0];
    rows_out = sc.misc[1];
}

}  // namespace santapp
