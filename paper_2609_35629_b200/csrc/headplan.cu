// Sampling of one query head (Algorithm 1: Gumbel-top-K over the perturbed routing scores and the
// conditional inclusion correction of Eq. method-inclusion), one block per (sequence, query head).
//
// The scorer leaves fp32 perturbed scores Y32 for every (head, team), the maximum of every block
// of 16 teams, and the inputs of a bound E on |Y32 - Y| against the exact fp64 score Y. The
// sample must be the fp64 one, so:
//   1. a lower bound t on the (K+1)-st largest Y32, from a histogram of the block maxima;
//   2. every team with Y32 >= t - 2E is a candidate: that set contains the K+1 largest exact
//      scores (if K+1 teams have Y32 >= t they have Y >= t - E, so the (K+1)-st largest Y is at
//      least t - E, and a team with Y above that has Y32 >= t - 2E);
//   3. the candidates are re-evaluated exactly in fp64 (dot product of bf16 values, log n_g,
//      Gumbel from the same Philox word) and ranked by (Y descending, team id ascending);
//   4. the K largest are the sample, the next one is tau, c_g = 1 - exp(-exp(phi_g - tau)).
// At most kCandCap candidates are held at a time; when more qualify the teams are walked in ranges
// of kCandCap with a running top-(K+1) list, so any number of candidates fits in shared memory.
// Output per head: the K sampled team ids in descending Y, log c_g and the packed row range of each.
#include <math_constants.h>

#include "common.cuh"

namespace santapp {

namespace {

constexpr int kMaxHeadWarps = 8;         // blocks of 256 threads, or 128 when many heads share the GPU
constexpr int kCandCap = 512;           // candidates refined at a time
constexpr int kListCap = 132;           // running top list: K + 1 <= 129 entries (+ one pad)
constexpr int kDotLanes = 8;            // threads that share one candidate's dot product
constexpr int kWindow = 255;            // histogram bins per pass of the bound

struct alignas(16) HeadSmem {
    double q64[kDotLanes][18];          // query in fp64: [16-dim slice][16 + pad] (pad: conflict-free LDS.128)
    double cand_y[kCandCap + 2];        // block list (ints), then dot products, then exact Y; read in pairs
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
    int n_blk, n_cand, bound_bin, bound_below, bound_total;
};

// Guard on |Y32 - Y|: tensor-core accumulation of exact bf16 products in fp32 (relative to the sum of
// magnitudes, bounded by scale * |q|_1 * max|l|), plus the fp32 logarithm and Gumbel terms.
__device__ __forceinline__ float score_guard(double scale, double q_l1, float k_abs_max)
{
    return (float)(2.5e-4 * scale * q_l1 * (double)k_abs_max + 1e-3);
}

// The first half of the block's warps compute dot products, the second half the Gumbel terms.
template <int kHeadThreads, bool kHalf>
__global__ void __launch_bounds__(kHeadThreads, 1024 / kHeadThreads)
headplan_kernel(PlanInputs in)
{
    constexpr int kHeadWarps = kHeadThreads / 32, kDotWarps = kHeadWarps / 2;
    __shared__ HeadSmem sm;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hq = blockIdx.x;                                        // (sequence, query head)
    const int b = hq / in.bv.n_q, hh = hq - b * in.bv.n_q;            // hh = j * G + h
    const int j = hh / in.bv.group;
    const int64_t team0 = in.bv.seq_team_off[b];
    const int M = pair_team_count(in.bv, b, j);
    const int K = in.n_sample;
    if (K >= M) return;                                               // every team is read with c = 1: nothing is drawn

    const uint32_t step = in.step + (in.step_dev ? *in.step_dev : 0u);
    const uint16_t *rep = in.rep_keys + ((size_t)j * in.bv.teams_total + team0) * kHeadDim;
    const int32_t *csr = in.team_row_start + (size_t)j * (in.bv.teams_total + in.bv.n_seqs) + team0 + b;
    const float *y32 = in.y32 + (size_t)hh * in.bv.teams_total + team0;
    const float *ym = in.ymax + (size_t)hh * in.ymax_stride + (team0 >> 4) + b;
    const int nblk = (M + 15) >> 4;
    const int need = K + 1;

    // ---- query in fp64, |q|_1, largest block maximum ----
    {
        float a = 0.f, top = -CUDART_INF_F;
        if (tid < kHeadDim) {
            const float v = elem_to_float<kHalf>(in.q[(size_t)hq * kHeadDim + tid]);
            sm.q64[tid >> 4][tid & 15] = (double)v;
            a = fabsf(v);
        }
        for (int i = tid; i < nblk; i += kHeadThreads) top = fmaxf(top, __ldg(ym + i));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
            top = fmaxf(top, __shfl_xor_sync(0xFFFFFFFFu, top, o));
        }
        if (lane == 0) { sm.red_sum[warp] = a; sm.red_max[warp] = top; }
        if (tid == 0) { sm.n_blk = 0; sm.n_cand = 0; }
    }
    __syncthreads();
    float q_l1 = 0.f, top = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < kHeadWarps; ++w) { q_l1 += sm.red_sum[w]; top = fmaxf(top, sm.red_max[w]); }
    const float guard = score_guard(in.scale, (double)q_l1 * 1.001, in.rep_abs_max[(size_t)j * in.bv.n_seqs + b]);

    // ---- 1. lower bound on the need-th largest score from the block maxima ----
    // A maximum v falls in global bin floor((top - v) * 4); one pass counts a window of 255 bins.
    // The first bin at which the running count reaches `need` has `need` distinct teams' scores
    // above its lower edge. Windows further down are visited only when an outlier at the top
    // leaves the first one short. -inf when there are fewer than `need` blocks.
    float t_lb = -CUDART_INF_F;
    if (nblk >= need) {
        int above = 0;
        for (int win = 0; win < 16 * kWindow; win += kWindow) {      // 1020 units below the top, then give up
            for (int i = tid; i < 256; i += kHeadThreads) sm.hist[i] = 0;
            __syncthreads();
            for (int i = tid; i < nblk; i += kHeadThreads) {
                const float d = (top - __ldg(ym + i)) * 4.f;
                const int gb = d >= 1073741824.f ? (1 << 30) : (int)d;    // the same in every pass
                if (gb >= win) atomicAdd(&sm.hist[min(gb - win, kWindow)], 1);
            }
            __syncthreads();
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
            __syncthreads();
            const int bin = sm.bound_bin, below = sm.bound_below, total = sm.bound_total;
            if (bin < kWindow) {                                    // lower edge, minus the rounding of the binning
                t_lb = top - (float)(win + bin + 1) * 0.25f * (1.f + 1e-6f) - 1e-4f;
                break;
            }
            if (below == 0) break;
            above += total - below;
        }
    }
    const float t_lo = t_lb - 2.f * guard;

    // ---- 2. candidates: blocks whose maximum reaches t_lo, then their teams ----
    int *blk_list = reinterpret_cast<int *>(sm.cand_y);
    for (int i = tid; i < nblk; i += kHeadThreads) {
        if (__ldg(ym + i) >= t_lo) {
            const int slot = atomicAdd(&sm.n_blk, 1);
            if (slot < kCandCap) blk_list[slot] = i;
        }
    }
    __syncthreads();
    const int n_blk = sm.n_blk;
    if (n_blk <= kCandCap) {
        // (listed block, quarter of its 16 scores) items, two per thread in flight
        for (int it0 = tid; it0 < n_blk * 4; it0 += 2 * kHeadThreads) {
            float v[2][4];
            int g0[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int it = it0 + u * kHeadThreads;
                g0[u] = it < n_blk * 4 ? blk_list[it >> 2] * 16 + (it & 3) * 4 : M;
#pragma unroll
                for (int i = 0; i < 4; ++i) v[u][i] = g0[u] + i < M ? __ldg(y32 + g0[u] + i) : -CUDART_INF_F;
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (g0[u] + i < M && v[u][i] >= t_lo) {
                        const int slot = atomicAdd(&sm.n_cand, 1);
                        if (slot < kCandCap) sm.cand_id[slot] = g0[u] + i;
                    }
                }
            }
        }
    }
    __syncthreads();
    const bool fits = n_blk <= kCandCap && sm.n_cand <= kCandCap;
    const int n_ranges = fits ? 1 : (M + kCandCap - 1) / kCandCap;

    int cur = 0, n_list = 0;
    for (int r = 0; r < n_ranges; ++r) {
        if (!fits) {                                                  // teams [r, r + 1) * kCandCap
            __syncthreads();
            if (tid == 0) sm.n_cand = 0;
            __syncthreads();
            for (int t = r * kCandCap + tid; t < min(M, (r + 1) * kCandCap); t += kHeadThreads) {
                if (__ldg(y32 + t) >= t_lo) sm.cand_id[atomicAdd(&sm.n_cand, 1)] = t;
            }
            __syncthreads();
        }
        const int n_cand = sm.n_cand;

        // ---- 3a. exact terms: dot products on the first half of the warps (8 lanes per candidate, 16 dims each),
        //          log n_g and the Gumbel term on the other warps (one thread per candidate) ----
        if (warp < kDotWarps) {
            const int sub = lane & (kDotLanes - 1);
            const double *qs = sm.q64[sub];
            // four candidates per thread group at a time: all their key pieces are requested before
            // the first product, so a chunk costs one memory round trip
            constexpr int kPerPass = kDotWarps * 32 / kDotLanes, kChunk = 4;
            for (int c0 = 0; c0 < n_cand; c0 += kPerPass * kChunk) {
                uint4 w[kChunk][2];
#pragma unroll
                for (int u = 0; u < kChunk; ++u) {
                    const int cand = c0 + u * kPerPass + (tid >> 3);
                    if (cand < n_cand) {
                        const uint4 *kr = reinterpret_cast<const uint4 *>(rep + (size_t)sm.cand_id[cand] * kHeadDim) + sub * 2;
                        w[u][0] = __ldg(kr);
                        w[u][1] = __ldg(kr + 1);
                    } else {
                        w[u][0] = w[u][1] = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
#pragma unroll
                for (int u = 0; u < kChunk; ++u) {
                    const int cand = c0 + u * kPerPass + (tid >> 3);
                    const uint4 w0 = w[u][0], w1 = w[u][1];
                    double d0 = 0.0, d1 = 0.0;
                    d0 = fma((double)elem_lo<kHalf>(w0.x), qs[0], d0);
                    d1 = fma((double)elem_hi<kHalf>(w0.x), qs[1], d1);
                    d0 = fma((double)elem_lo<kHalf>(w0.y), qs[2], d0);
                    d1 = fma((double)elem_hi<kHalf>(w0.y), qs[3], d1);
                    d0 = fma((double)elem_lo<kHalf>(w0.z), qs[4], d0);
                    d1 = fma((double)elem_hi<kHalf>(w0.z), qs[5], d1);
                    d0 = fma((double)elem_lo<kHalf>(w0.w), qs[6], d0);
                    d1 = fma((double)elem_hi<kHalf>(w0.w), qs[7], d1);
                    d0 = fma((double)elem_lo<kHalf>(w1.x), qs[8], d0);
                    d1 = fma((double)elem_hi<kHalf>(w1.x), qs[9], d1);
                    d0 = fma((double)elem_lo<kHalf>(w1.y), qs[10], d0);
                    d1 = fma((double)elem_hi<kHalf>(w1.y), qs[11], d1);
                    d0 = fma((double)elem_lo<kHalf>(w1.z), qs[12], d0);
                    d1 = fma((double)elem_hi<kHalf>(w1.z), qs[13], d1);
                    d0 = fma((double)elem_lo<kHalf>(w1.w), qs[14], d0);
                    d1 = fma((double)elem_hi<kHalf>(w1.w), qs[15], d1);
                    double d = d0 + d1;
                    d += __shfl_xor_sync(0xFFFFFFFFu, d, 1);
                    d += __shfl_xor_sync(0xFFFFFFFFu, d, 2);
                    d += __shfl_xor_sync(0xFFFFFFFFu, d, 4);
                    if (cand < n_cand && sub == 0) sm.cand_y[cand] = d;
                }
            }
        } else {
            for (int i = tid - kDotWarps * 32; i < n_cand; i += kHeadThreads - kDotWarps * 32) {
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
        for (int i = tid; i < n_cand; i += kHeadThreads) {
            const double phi = sm.cand_phi[i] + sm.cand_y[i] * in.scale;
            sm.cand_phi[i] = phi;
            sm.cand_y[i] = phi + sm.cand_g[i];
            if (i == n_cand - 1) sm.cand_y[n_cand] = -CUDART_INF;       // pad for the paired reads below
        }
        __syncthreads();

        // ---- 3b. merge with the running list: keep the K + 1 largest by (Y descending, id ascending) ----
        for (int e = tid; e < n_list + n_cand; e += kHeadThreads) {
            double y, phi;
            int id;
            int2 rows;
            if (e < n_list) { y = sm.list_y[cur][e]; phi = sm.list_phi[cur][e]; id = sm.list_id[cur][e]; rows = sm.list_rows[cur][e]; }
            else { y = sm.cand_y[e - n_list]; phi = sm.cand_phi[e - n_list]; id = sm.cand_id[e - n_list]; rows = sm.cand_rows[e - n_list]; }
            // rank = entries ahead of this one; scores are compared two at a time, ids are looked at
            // only when some other entry has exactly the same score
            int rank = 0, same = 0;
            const double2 *ly = reinterpret_cast<const double2 *>(sm.list_y[cur]);
            const double2 *cy = reinterpret_cast<const double2 *>(sm.cand_y);
#pragma unroll 2
            for (int a = 0; a < (n_list + 1) >> 1; ++a) {
                const double2 w = ly[a];
                rank += (w.x > y) + (w.y > y);
                same += (w.x == y) + (w.y == y);
            }
#pragma unroll 2
            for (int a = 0; a < (n_cand + 1) >> 1; ++a) {
                const double2 w = cy[a];
                rank += (w.x > y) + (w.y > y);
                same += (w.x == y) + (w.y == y);
            }
            if (same > 1) {
                for (int a = 0; a < n_list; ++a) rank += (sm.list_y[cur][a] == y && sm.list_id[cur][a] < id);
                for (int a = 0; a < n_cand; ++a) rank += (sm.cand_y[a] == y && sm.cand_id[a] < id);
            }
            if (rank <= K) {
                sm.list_y[cur ^ 1][rank] = y;
                sm.list_phi[cur ^ 1][rank] = phi;
                sm.list_id[cur ^ 1][rank] = id;
                sm.list_rows[cur ^ 1][rank] = rows;
            }
        }
        n_list = min(K + 1, n_list + n_cand);
        cur ^= 1;
        if (tid == 0) sm.list_y[cur][n_list] = -CUDART_INF;
        __syncthreads();
    }

    // ---- 4. corrections ----
    // Fewer than K + 1 ranked teams can only mean scores that do not compare (non-finite inputs):
    // the sample is completed with the first teams so that every index handed on is valid, and
    // the status word says so.
    const bool short_list = n_list < K + 1;
    const double tau = short_list ? __longlong_as_double(0x7FF8000000000000ll) : sm.list_y[cur][K];
    if (short_list && tid == 0 && in.status) atomicOr(in.status, 2);
    for (int a = tid; a < K; a += kHeadThreads) {
        int id;
        float logc;
        int2 rows;
        if (a < n_list && !short_list) {
            const double c = -expm1(-exp(sm.list_phi[cur][a] - tau));     // 1 - exp(-exp(phi - tau))
            logc = (float)log(c);
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

}  // namespace

cudaError_t launch_headplan(const PlanInputs &in, cudaStream_t s)
{
    // 256 threads per head while every head's block is resident at once (4 per SM by registers),
    // else 128 threads so that twice as many fit
    const int n_heads = in.bv.n_seqs * in.bv.n_q;
    const bool wide = n_heads <= 4 * attend_grid_size();
    if (in.bv.elem) {
        if (wide) headplan_kernel<256, true><<<n_heads, 256, 0, s>>>(in);
        else      headplan_kernel<128, true><<<n_heads, 128, 0, s>>>(in);
    } else {
        if (wide) headplan_kernel<256, false><<<n_heads, 256, 0, s>>>(in);
        else      headplan_kernel<128, false><<<n_heads, 128, 0, s>>>(in);
    }
    return cudaGetLastError();
}

}  // namespace santapp
