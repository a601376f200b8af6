// santapp_kmeans_fit: the fit of Algorithm 3 (global minibatch k-means parents), one independent
// problem per (sequence, KV head). Preparation path, run once after prefill.
//
// The paper names the routine and its settings and leaves the rest to its library; the reading
// taken here is written out in include/santapp.h. Every random choice is a Philox word with
// counter (slot, tag, stream, step), and every comparison is made on fp64 values obtained by the
// same operations in the same order wherever the order matters (sums over dimensions, over the
// sample, over a minibatch; separately rounded multiply and add), so a fit is a pure function
// of its arguments. Sums whose order matters run on one thread; the distance evaluations around
// them are spread over the grid.
#include <limits.h>
#include <math.h>

#include <algorithm>

#include "common.cuh"

namespace santapp {

namespace {

constexpr int kThreads = 256;
constexpr int kTile = 16;                 // centres staged per shared-memory tile
constexpr int kPollEvery = 16;            // steps between two looks at the fits' stop flags
constexpr uint32_t kTagSample = 1u, kTagStart = 2u, kTagBatch = 3u, kTagMove = 4u;

struct Pair {
    int b, j, N, k, n_init, L, t_max;
    uint32_t stream;
    int64_t row0, c0;
    size_t plane;                         // first row of the pair in a [n_kv][rows_total] array
    size_t cplane;                        // first centre of the pair in a [n_kv][centres_total] array
    int id;                               // j-major pair index into the per-pair scratch arrays
};

__device__ __forceinline__ Pair pair_of(const KmeansParams &p, int b, int j)
{
    Pair q;
    q.b = b;
    q.j = j;
    q.row0 = p.seq_row_off[b];
    q.N = (int)(p.seq_row_off[b + 1] - q.row0);
    q.c0 = p.seq_centre_off[b];
    q.k = (int)(p.seq_centre_off[b + 1] - q.c0);
    q.n_init = p.seq_n_init[b];
    q.L = p.seq_trials[b];
    q.t_max = p.seq_t_max[b];
    q.stream = p.stream_base + (uint32_t)(b * p.n_kv + j);
    q.plane = (size_t)j * p.rows_total + (size_t)q.row0;
    q.cplane = (size_t)j * p.centres_total + (size_t)q.c0;
    q.id = j * p.n_seqs + b;
    return q;
}

__device__ __forceinline__ uint32_t km_word(const KmeansParams &p, uint32_t slot, uint32_t tag, uint32_t stream, uint32_t step)
{
    return philox4x32_10(make_uint4(slot, tag, stream, step), p.seed_lo, p.seed_hi).x;
}
__device__ __forceinline__ int km_index(uint32_t word, int n) { return (int)(((unsigned long long)word * (unsigned long long)n) >> 32); }

template <bool kHalf>
__device__ __forceinline__ double sqdist_rows(const uint4 *a, const uint4 *b)
{
    double s = 0.0;
#pragma unroll 4
    for (int q = 0; q < 16; ++q) {
        const uint4 x4 = a[q], y4 = b[q];
        const uint32_t x[4] = {x4.x, x4.y, x4.z, x4.w}, y[4] = {y4.x, y4.y, y4.z, y4.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const double e0 = __dsub_rn((double)elem_lo<kHalf>(x[t]), (double)elem_lo<kHalf>(y[t]));
            const double e1 = __dsub_rn((double)elem_hi<kHalf>(x[t]), (double)elem_hi<kHalf>(y[t]));
            s = __dadd_rn(s, __dmul_rn(e0, e0));
            s = __dadd_rn(s, __dmul_rn(e1, e1));
        }
    }
    return s;
}

// ---- 1. initialisation sample: head of a Fisher-Yates shuffle ----
__global__ void __launch_bounds__(kThreads)
km_perm_identity_kernel(KmeansParams p)
{
    const Pair q = pair_of(p, blockIdx.y, blockIdx.z);
    const int i = blockIdx.x * kThreads + threadIdx.x;
    if (i < q.N) p.perm[q.plane + i] = i;
}

// One block per pair. The swaps run in order on one lane; when the sequence's index list fits in
// shared memory (smem_rows entries) it lives there for the shuffle -- a swap then costs two
// shared-memory round trips instead of two to L2 -- and only the head, the sample, is written out.
constexpr int kSampleSmemRows = 50 * 1024;
__global__ void __launch_bounds__(kThreads)
km_sample_kernel(KmeansParams p, int smem_rows)
{
    extern __shared__ int32_t perm_s[];
    const Pair q = pair_of(p, blockIdx.x, blockIdx.y);
    const int tid = threadIdx.x, lane = tid & 31;
    int32_t *perm_g = p.perm + q.plane;                       // (holds the identity when it is used for the shuffle)
    const bool in_smem = q.N <= smem_rows;
    if (in_smem)
        for (int i = tid; i < q.N; i += kThreads) perm_s[i] = i;
    __syncthreads();
    if (tid < 32) {
        int32_t *perm = in_smem ? perm_s : perm_g;
        // the words of 32 positions at a time, the swaps in order on one lane
        for (int i0 = 0; i0 < q.n_init; i0 += 32) {
            const int i = i0 + lane;
            const uint32_t w = i < q.n_init ? km_word(p, (uint32_t)i, kTagSample, q.stream, 0u) : 0u;
            for (int l = 0; l < 32 && i0 + l < q.n_init; ++l) {
                const uint32_t wl = __shfl_sync(0xFFFFFFFFu, w, l);
                if (lane == 0) {
                    const int at = i0 + l;
                    const int r = at + km_index(wl, q.N - at);
                    const int32_t t = perm[at];
                    perm[at] = perm[r];
                    perm[r] = t;
                }
            }
        }
    }
    __syncthreads();
    if (in_smem)
        for (int i = tid; i < q.n_init; i += kThreads) perm_g[i] = perm_s[i];
    if (tid == 0) p.pick[(size_t)q.id * p.trials_max] = km_index(km_word(p, 0u, kTagStart, q.stream, 0u), q.n_init);
}

// ---- 2. greedy k-means++ on the sample ----
constexpr int kSumBlock = 128;           // sums over the initialisation sample are taken in blocks of this many points
constexpr int kMaxSumBlocks = 224;       // an initialisation sample holds at most 28544 points (223 blocks)
constexpr int kDistPts = 1;              // points per thread
constexpr int kDistThreads = kSumBlock / kDistPts;   // a block covers one block of the sums
static_assert(kDistThreads % 64 == 0, "64 threads widen one candidate row");
constexpr int kDistTrials = 6;           // candidate points per block

// Distances of every sample point to the candidate points pick[0..n_cand): cand[l][i]; and, for c > 0,
// the sums of min(closest_i, cand[l][i]) over each block of kSumBlock consecutive sample points, added
// in order by one thread per candidate (the potential of a trial is the sum of its block sums in order).
template <bool kHalf>
__global__ void __launch_bounds__(kDistThreads)
km_candidate_dist_kernel(KmeansParams p, int c)
{
    __shared__ __align__(16) double y_s[kDistTrials][kHeadDim];
    __shared__ double term_s[kDistTrials][kSumBlock];
    const Pair q = pair_of(p, blockIdx.z / p.n_kv, blockIdx.z % p.n_kv);
    if (c >= q.k || blockIdx.x * kSumBlock >= q.n_init) return;
    const int L = c == 0 ? 1 : q.L;
    const int n_chunks = (L + kDistTrials - 1) / kDistTrials, per = (L + n_chunks - 1) / n_chunks;
    const int l0 = blockIdx.y * per, cn = min(per, L - l0);
    if (cn <= 0) return;
    const int tid = threadIdx.x;
    const int32_t *perm = p.perm + q.plane;
    const uint16_t *keys = p.k_prompt + q.plane * kHeadDim;
    __shared__ int row_s[kDistTrials];
    if (tid < cn) row_s[tid] = perm[p.pick[(size_t)q.id * p.trials_max + l0 + tid]];
    int i[kDistPts];
    const uint4 *row[kDistPts];
#pragma unroll
    for (int j = 0; j < kDistPts; ++j) {
        i[j] = blockIdx.x * kSumBlock + j * kDistThreads + tid;
        row[j] = reinterpret_cast<const uint4 *>(keys + (size_t)perm[min(i[j], q.n_init - 1)] * kHeadDim);
    }
    __syncthreads();
    {
        // the candidates' rows as doubles: a thread widens one packed word (two values) of every
        // kGroups-th row
        constexpr int kGroups = kDistThreads / 64, kMine = (kDistTrials + kGroups - 1) / kGroups;
        const int wi = tid & 63, v0 = tid >> 6;
        uint32_t yw[kMine];
#pragma unroll
        for (int m = 0; m < kMine; ++m) {
            const int v = v0 + m * kGroups;
            yw[m] = v < cn ? reinterpret_cast<const uint32_t *>(keys + (size_t)row_s[v] * kHeadDim)[wi] : 0u;
        }
#pragma unroll
        for (int m = 0; m < kMine; ++m) {
            const int v = v0 + m * kGroups;
            if (v < cn) {
                y_s[v][2 * wi] = (double)elem_lo<kHalf>(yw[m]);
                y_s[v][2 * wi + 1] = (double)elem_hi<kHalf>(yw[m]);
            }
        }
    }
    __syncthreads();
    double d[kDistPts][kDistTrials];
#pragma unroll
    for (int j = 0; j < kDistPts; ++j)
#pragma unroll
        for (int v = 0; v < kDistTrials; ++v) d[j][v] = 0.0;
    switch (cn) {
    case 1: dist_points<kHalf, kDistPts, 1, kDistTrials>(row, y_s, d); break;
    case 2: dist_points<kHalf, kDistPts, 2, kDistTrials>(row, y_s, d); break;
    case 3: dist_points<kHalf, kDistPts, 3, kDistTrials>(row, y_s, d); break;
    case 4: dist_points<kHalf, kDistPts, 4, kDistTrials>(row, y_s, d); break;
    case 5: dist_points<kHalf, kDistPts, 5, kDistTrials>(row, y_s, d); break;
    default: dist_points<kHalf, kDistPts, 6, kDistTrials>(row, y_s, d); break;
    }
#pragma unroll
    for (int j = 0; j < kDistPts; ++j) {
#pragma unroll
        for (int v = 0; v < kDistTrials; ++v) {
            if (v >= cn) continue;
            double term = -1.0;                             // marks a point past the end of the sample
            if (i[j] < q.n_init) {
                p.cand[((size_t)q.id * p.trials_max + l0 + v) * p.n_init_max + i[j]] = d[j][v];
                if (c > 0) {
                    const double o = p.closest[(size_t)q.id * p.n_init_max + i[j]];
                    term = d[j][v] < o ? d[j][v] : o;
                }
            }
            term_s[v][j * kDistThreads + tid] = term;
        }
    }
    if (c == 0) return;
    __syncthreads();
    if (tid < cn) {
        double w = 0.0;
#pragma unroll 8
        for (int u = 0; u < kSumBlock; ++u) {
            const double v = term_s[tid][u];
            if (v >= 0.0) w = __dadd_rn(w, v);
        }
        const int n_part = (p.n_init_max + kSumBlock - 1) / kSumBlock;
        p.part[((size_t)q.id * p.trials_max + l0 + tid) * n_part + blockIdx.x] = w;
    }
}

constexpr int kAcceptThreads = 1024;

// One block per pair: potentials of the trials (sums in blocks of kSumBlock sample points), the best
// trial becomes centre c, the nearest-centre distances are lowered, and the trial points of centre
// c + 1 are drawn. Every serial sum runs over shared memory with its loads ahead of its additions.
template <bool kHalf>
__global__ void __launch_bounds__(kAcceptThreads)
km_accept_kernel(KmeansParams p, int c)
{
    extern __shared__ double cum_s[];                       // [n_init + blocks] running sums, then [blocks] block offsets
    __shared__ int best_s;
    __shared__ double pot_s[32];
    const Pair q = pair_of(p, blockIdx.x, blockIdx.y);
    if (c >= q.k) return;
    const int tid = threadIdx.x;
    const int n_trials = c == 0 ? 1 : q.L;
    const int n_blocks = (q.n_init + kSumBlock - 1) / kSumBlock, n_part = (p.n_init_max + kSumBlock - 1) / kSumBlock;
    double *closest = p.closest + (size_t)q.id * p.n_init_max;
    const double *cand = p.cand + (size_t)q.id * p.trials_max * p.n_init_max;
    double *off_s = cum_s + p.n_init_max + kMaxSumBlocks;
    if (c > 0) {
        // the potential of a trial: its block sums (left by the distance kernel) added in order
        for (int e = tid; e < n_trials * n_blocks; e += kAcceptThreads) {
            const int l = e / n_blocks;
            cum_s[e] = p.part[((size_t)q.id * p.trials_max + l) * n_part + (e - l * n_blocks)];
        }
        __syncthreads();
        if (tid < n_trials) {
            double pot = 0.0;
#pragma unroll 8
            for (int blk = 0; blk < n_blocks; ++blk) pot = __dadd_rn(pot, cum_s[tid * n_blocks + blk]);
            pot_s[tid] = pot;
        }
    }
    __syncthreads();
    if (tid == 0) {
        int best = 0;
        for (int l = 1; l < n_trials; ++l)
            if (pot_s[l] < pot_s[best]) best = l;
        best_s = best;
    }
    __syncthreads();
    const int best = best_s;
    const double *win = cand + (size_t)best * p.n_init_max;
    if (tid < kHeadDim) {
        const int32_t *perm = p.perm + q.plane;
        const int at = p.pick[(size_t)q.id * p.trials_max + best];
        const uint16_t v = p.k_prompt[(q.plane + (size_t)perm[at]) * kHeadDim + tid];
        p.centres64[(q.cplane + (size_t)c) * kHeadDim + tid] = elem_to_double<kHalf>(v);
    }
    // The nearest-centre distances are lowered and kept in shared memory for the draw of the next
    // centre's trial points (inverse CDF over the sample in order). cum_s holds one pad word per
    // block of the sums (point i at i + i / kSumBlock), so that threads that walk different blocks do
    // not meet in one bank.
    for (int i0 = 0; i0 < q.n_init; i0 += 8 * kAcceptThreads) {
        double d[8], o[8];
#pragma unroll
        for (int v = 0; v < 8; ++v) {
            const int i = i0 + v * kAcceptThreads + tid;
            if (i < q.n_init) {
                d[v] = win[i];
                o[v] = c == 0 ? 0.0 : closest[i];
            }
        }
#pragma unroll
        for (int v = 0; v < 8; ++v) {
            const int i = i0 + v * kAcceptThreads + tid;
            if (i < q.n_init) {
                const double t = (c == 0 || d[v] < o[v]) ? d[v] : o[v];
                closest[i] = t;
                cum_s[i + i / kSumBlock] = t;
            }
        }
    }
    if (c + 1 >= q.k) return;                               // the pair's last centre draws nothing
    __syncthreads();
    // running sums inside each block (a thread per block), the block offsets in order, offset + running sum
    if (tid < n_blocks) {
        const int lo = tid * kSumBlock, cnt = min(kSumBlock, q.n_init - lo);
        double *blk_s = cum_s + lo + tid;
        double w = 0.0;
        for (int u = 0; u < cnt; u += 8) {
            double t[8];
#pragma unroll
            for (int v = 0; v < 8; ++v) t[v] = u + v < cnt ? blk_s[u + v] : 0.0;
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                if (u + v < cnt) {
                    w = __dadd_rn(w, t[v]);
                    blk_s[u + v] = w;
                }
            }
        }
        off_s[tid] = w;
    }
    __syncthreads();
    if (tid == 0) {                                         // sums of the earlier blocks, in order
        double off = 0.0;
#pragma unroll 8
        for (int blk = 0; blk < n_blocks; ++blk) {
            const double t = off_s[blk];
            off_s[blk] = off;
            off = __dadd_rn(off, t);
        }
    }
    __syncthreads();
    for (int i = tid; i < q.n_init; i += kAcceptThreads) cum_s[i + i / kSumBlock] = __dadd_rn(off_s[i / kSumBlock], cum_s[i + i / kSumBlock]);
    __syncthreads();
    if (tid < q.L) {
        const double total = cum_s[q.n_init - 1 + (q.n_init - 1) / kSumBlock];
        const uint32_t w = km_word(p, (uint32_t)tid, kTagStart, q.stream, (uint32_t)(c + 1));
        const double target = __dmul_rn(((double)w + 0.5) * (1.0 / 4294967296.0), total);
        int lo = 0, hi = q.n_init;                          // first i in [lo, hi) with cum_s[i] > target
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (cum_s[mid + mid / kSumBlock] > target) hi = mid; else lo = mid + 1;
        }
        p.pick[(size_t)q.id * p.trials_max + tid] = lo < q.n_init ? lo : q.n_init - 1;
    }
}

// ---- 3. minibatch steps ----
__device__ __forceinline__ bool pair_active(const KmeansParams &p, const Pair &q, int t)
{
    return t < q.t_max && !p.state[q.id].stopped;
}

// Draw the minibatch and assign each point to its nearest centre (ties to the smaller index). A thread
// holds two points and takes eight centres at a time (dist_points); every sum still adds its 128
// terms in order.
constexpr int kAssignPts = 2;             // points per thread
constexpr int kAssignBlock = 128 * kAssignPts;
constexpr int kAssignGroup = 8;           // centres per pass
static_assert(kTile % kAssignGroup == 0, "a tile of centres is a whole number of passes");
template <bool kHalf>
__global__ void __launch_bounds__(128)
km_batch_assign_kernel(KmeansParams p, int t)
{
    __shared__ __align__(16) double c[kTile][kHeadDim];
    const Pair q = pair_of(p, blockIdx.y / p.n_kv, blockIdx.y % p.n_kv);
    if (!pair_active(p, q, t)) return;
    const int tid = threadIdx.x;
    int s[kAssignPts], idx[kAssignPts];
    const uint4 *row[kAssignPts];
    double best[kAssignPts];
    int arg[kAssignPts];
#pragma unroll
    for (int j = 0; j < kAssignPts; ++j) {
        s[j] = blockIdx.x * kAssignBlock + j * 128 + tid;
        idx[j] = km_index(km_word(p, (uint32_t)(s[j] < p.batch ? s[j] : 0), kTagBatch, q.stream, (uint32_t)t), q.N);
        row[j] = reinterpret_cast<const uint4 *>(p.k_prompt + (q.plane + (size_t)idx[j]) * kHeadDim);
        best[j] = INFINITY;
        arg[j] = 0;
    }
    const double *cen = p.centres64 + q.cplane * kHeadDim;
    // this block searches one slice of the centres (a multiple of kTile each); the slices' results are
    // compared in slice order afterwards, so ties still go to the smaller centre index
    const int slice = blockIdx.z;
    const int per = ((q.k + p.assign_split - 1) / p.assign_split + kTile - 1) / kTile * kTile;
    const int k_lo = min(slice * per, q.k), k_hi = min(k_lo + per, q.k);
    for (int base = k_lo; base < k_hi; base += kTile) {
        const int nt = min(kTile, k_hi - base);
        __syncthreads();
        for (int e = tid; e < nt * kHeadDim; e += 128) c[e >> 7][e & 127] = cen[(size_t)base * kHeadDim + e];
        __syncthreads();
        for (int u = 0; u < nt; u += kAssignGroup) {
            // (rows of the tile past nt hold older values; their sums are not looked at)
            double d[kAssignPts][kAssignGroup];
#pragma unroll
            for (int j = 0; j < kAssignPts; ++j)
#pragma unroll
                for (int v = 0; v < kAssignGroup; ++v) d[j][v] = 0.0;
            dist_points<kHalf, kAssignPts, kAssignGroup, kAssignGroup>(row, c + u, d);
#pragma unroll
            for (int j = 0; j < kAssignPts; ++j)
#pragma unroll
                for (int v = 0; v < kAssignGroup; ++v)
                    if (u + v < nt && d[j][v] < best[j]) { best[j] = d[j][v]; arg[j] = base + u + v; }
        }
    }
#pragma unroll
    for (int j = 0; j < kAssignPts; ++j) {
        if (s[j] >= p.batch) continue;
        const size_t at = (size_t)q.id * p.batch + s[j];
        if (slice == 0) p.idx[at] = idx[j];
        if (p.assign_split == 1) {
            p.label[at] = arg[j];
            p.dist[at] = best[j];
        } else {
            const size_t pa = ((size_t)q.id * p.assign_split + slice) * p.batch + s[j];
            p.label_part[pa] = arg[j];
            p.dist_part[pa] = best[j];
        }
    }
}

// The nearest centre of each minibatch point over all slices (strictly smaller distance wins, slices in
// order of the centre index).
__global__ void __launch_bounds__(128)
km_assign_reduce_kernel(KmeansParams p, int t)
{
    const Pair q = pair_of(p, blockIdx.y / p.n_kv, blockIdx.y % p.n_kv);
    if (!pair_active(p, q, t)) return;
    const int s = blockIdx.x * 128 + threadIdx.x;
    if (s >= p.batch) return;
    double best = INFINITY;
    int arg = 0;
    for (int slice = 0; slice < p.assign_split; ++slice) {
        const size_t pa = ((size_t)q.id * p.assign_split + slice) * p.batch + s;
        const double d = p.dist_part[pa];
        if (d < best) { best = d; arg = p.label_part[pa]; }
    }
    const size_t at = (size_t)q.id * p.batch + s;
    p.label[at] = arg;
    p.dist[at] = best;
}

// The minibatch's slots ordered by (label, slot), one block per pair: a bitonic sort of the keys
// label << 12 | slot in shared memory (batch <= 4096; the keys are distinct, so the order is the
// minibatch order inside every label).
constexpr int kSortThreads = 1024, kSortKeys = 4096;
__global__ void __launch_bounds__(kSortThreads)
km_sort_batch_kernel(KmeansParams p, int t)
{
    __shared__ uint32_t key_s[kSortKeys];
    const Pair q = pair_of(p, blockIdx.x / p.n_kv, blockIdx.x % p.n_kv);
    if (!pair_active(p, q, t)) return;
    const int tid = threadIdx.x;
    for (int s = tid; s < kSortKeys; s += kSortThreads)
        key_s[s] = s < p.batch ? ((uint32_t)p.label[(size_t)q.id * p.batch + s] << 12) | (uint32_t)s : 0xFFFFFFFFu;
    __syncthreads();
    for (int size = 2; size <= kSortKeys; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int e = tid; e < kSortKeys / 2; e += kSortThreads) {
                const int lo = 2 * e - (e & (stride - 1)), hi = lo + stride;       // partners of this compare-exchange
                const bool up = (lo & size) == 0;
                const uint32_t a = key_s[lo], b = key_s[hi];
                if ((a > b) == up) { key_s[lo] = b; key_s[hi] = a; }
            }
            __syncthreads();
        }
    }
    for (int s = tid; s < kSortKeys; s += kSortThreads) p.sorted[(size_t)q.id * kSortKeys + s] = key_s[s];
}

// Cumulative-count update: thread (centre, dimension) adds the centre's new points in minibatch
// order (it finds them in the sorted slots); c <- (c * count + sum) / (count + n).
template <bool kHalf>
__global__ void __launch_bounds__(kThreads)
km_batch_update_kernel(KmeansParams p, int t)
{
    const Pair q = pair_of(p, blockIdx.y / p.n_kv, blockIdx.y % p.n_kv);
    if (!pair_active(p, q, t)) return;
    const int u = blockIdx.x * (kThreads / kHeadDim) + threadIdx.x / kHeadDim, d = threadIdx.x % kHeadDim;
    const bool live = u < q.k;
    double sum = 0.0, count = 0.0;
    int n = 0;
    if (live) {
        const uint32_t *sorted = p.sorted + (size_t)q.id * kSortKeys;
        int lo = 0, hi = kSortKeys;                         // first position with label >= u
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if ((sorted[mid] >> 12) >= (uint32_t)u) hi = mid; else lo = mid + 1;
        }
        count = p.count[q.cplane + u];
        const uint16_t *col = p.k_prompt + q.plane * kHeadDim + d;
        const int32_t *idx = p.idx + (size_t)q.id * p.batch;
        for (int at = lo; at < kSortKeys && (sorted[at] >> 12) == (uint32_t)u; ++at, ++n)
            sum = __dadd_rn(sum, elem_to_double<kHalf>(col[(size_t)idx[sorted[at] & 4095u] * kHeadDim]));
    }
    __syncthreads();                                        // every thread has read its centre's count
    if (live && n > 0) {
        const double grown = __dadd_rn(count, (double)n);
        double *cd = p.centres64 + (q.cplane + (size_t)u) * kHeadDim + d;
        *cd = __ddiv_rn(__dadd_rn(__dmul_rn(*cd, count), sum), grown);
        if (d == 0) p.count[q.cplane + u] = grown;
    }
}

// One block per pair: reassignment of starved centres, averaged inertia, stopping rule. The serial
// parts (the inertia is the sum of the minibatch distances in order) run on one thread over shared
// memory that all threads filled.
template <bool kHalf>
__global__ void __launch_bounds__(kThreads)
km_control_kernel(KmeansParams p, int t)
{
    extern __shared__ double ctl_dist[];                    // dist[batch], then int32 slots[batch], move_centre[batch / 2]
    __shared__ int n_move_s;
    __shared__ double cmin_s[kThreads / 32], cmax_s[kThreads / 32];
    const Pair q = pair_of(p, blockIdx.x, blockIdx.y);
    if (!pair_active(p, q, t)) return;
    const int tid = threadIdx.x;
    int32_t *slots = reinterpret_cast<int32_t *>(ctl_dist + p.batch), *move_centre = slots + p.batch;
    double *count = p.count + q.cplane;
    const int32_t *idx = p.idx + (size_t)q.id * p.batch;
    {
        const double *dist = p.dist + (size_t)q.id * p.batch;
        for (int s = tid; s < p.batch; s += kThreads) ctl_dist[s] = dist[s];
        double cmin = INFINITY, cmax = 0.0;                 // smallest and largest count: any order gives the same
        for (int u = tid; u < q.k; u += kThreads) {
            const double v = count[u];
            if (v < cmin) cmin = v;
            if (v > cmax) cmax = v;
        }
        for (int o = 16; o > 0; o >>= 1) {
            const double a = __shfl_xor_sync(0xffffffffu, cmin, o), b = __shfl_xor_sync(0xffffffffu, cmax, o);
            if (a < cmin) cmin = a;
            if (b > cmax) cmax = b;
        }
        if ((tid & 31) == 0) { cmin_s[tid >> 5] = cmin; cmax_s[tid >> 5] = cmax; }
    }
    __syncthreads();
    if (tid == 0) {
        int n_move = 0;
        double cmin = INFINITY, cmax = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) {
            if (cmin_s[w] < cmin) cmin = cmin_s[w];
            if (cmax_s[w] > cmax) cmax = cmax_s[w];
        }
        const long long period = 10 + (long long)floor(cmin);
        if (p.ratio > 0.0 && ((long long)t + 1) % period == 0) {
            const double thr = __dmul_rn(p.ratio, cmax);
            const int cap = p.batch / 2;
            double keep_min = INFINITY;
            for (int u = 0; u < q.k; ++u) {
                const double v = count[u];
                if (v < thr && n_move < cap) move_centre[n_move++] = u;
                else if (v < keep_min) keep_min = v;
            }
            if (n_move > 0) {
                for (int s = 0; s < p.batch; ++s) slots[s] = s;
                for (int i = 0; i < n_move; ++i) {
                    const int r = i + km_index(km_word(p, (uint32_t)i, kTagMove, q.stream, (uint32_t)t), p.batch - i);
                    const int tmp = slots[i];
                    slots[i] = slots[r];
                    slots[r] = tmp;
                }
                for (int i = 0; i < n_move; ++i) count[move_centre[i]] = keep_min;
            }
        }
        n_move_s = n_move;
    }
    __syncthreads();
    const int n_move = n_move_s;
    for (int e = tid; e < n_move * kHeadDim; e += kThreads) {   // the moved centres jump onto minibatch points
        const int i = e >> 7, d = e & (kHeadDim - 1);
        const uint16_t *src = p.k_prompt + (q.plane + (size_t)idx[slots[i]]) * kHeadDim;
        p.centres64[(q.cplane + (size_t)move_centre[i]) * kHeadDim + d] = elem_to_double<kHalf>(src[d]);
    }
    if (tid == 0) {
        double inertia = 0.0;
#pragma unroll 8
        for (int s = 0; s < p.batch; ++s) inertia = __dadd_rn(inertia, ctl_dist[s]);
        KmeansState &st = p.state[q.id];
        double alpha = __ddiv_rn(__dmul_rn(2.0, (double)p.batch), __dadd_rn((double)q.N, 1.0));
        if (alpha > 1.0) alpha = 1.0;
        const double per_point = __ddiv_rn(inertia, (double)p.batch);
        const double ewa = t == 0 ? per_point
                                  : __dadd_rn(__dmul_rn(st.ewa, __dsub_rn(1.0, alpha)), __dmul_rn(per_point, alpha));
        st.ewa = ewa;
        st.steps += 1;
        if (t == 0 || ewa < st.ewa_min) { st.ewa_min = ewa; st.bad = 0; }
        else if (++st.bad >= p.patience) st.stopped = 1;
    }
}

// How many fits still have steps to run after step t (one block; the host reads it now and then
// and stops enqueuing steps once it is zero).
__global__ void __launch_bounds__(kThreads)
km_count_active_kernel(KmeansParams p, int t)
{
    __shared__ int n_s;
    if (threadIdx.x == 0) n_s = 0;
    __syncthreads();
    const int pairs = p.n_seqs * p.n_kv;
    int n = 0;
    for (int i = threadIdx.x; i < pairs; i += kThreads) {
        const int b = i % p.n_seqs;                         // state is indexed j * n_seqs + b
        n += (t + 1 < p.seq_t_max[b] && !p.state[i].stopped) ? 1 : 0;
    }
    if (n) atomicAdd(&n_s, n);
    __syncthreads();
    if (threadIdx.x == 0) *p.active = n_s;
}

__global__ void __launch_bounds__(kThreads)
km_finish_kernel(KmeansParams p)
{
    const Pair q = pair_of(p, blockIdx.y, blockIdx.z);
    const int e = blockIdx.x * kThreads + threadIdx.x;
    if (e < q.k * kHeadDim) p.centres_out[q.cplane * kHeadDim + e] = __double2float_rn(p.centres64[q.cplane * kHeadDim + e]);
    if (e == 0 && p.steps_out) p.steps_out[q.id] = p.state[q.id].steps;
}

template <bool kHalf>
cudaError_t run_fit(const KmeansParams &p, cudaStream_t s)
{
    const int B = p.n_seqs, H = p.n_kv, pairs = B * H;
    cudaError_t err;
#define KM_CHECK() if ((err = cudaGetLastError()) != cudaSuccess) return err
    const int sample_smem_rows = std::min(p.max_rows_per_seq, kSampleSmemRows);
    if (p.max_rows_per_seq > sample_smem_rows) {              // some sequence shuffles its index list in global memory
        km_perm_identity_kernel<<<dim3((p.max_rows_per_seq + kThreads - 1) / kThreads, B, H), kThreads, 0, s>>>(p);
        KM_CHECK();
    }
    if ((err = cudaFuncSetAttribute(km_sample_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)sizeof(int32_t) * kSampleSmemRows)) != cudaSuccess) return err;
    km_sample_kernel<<<dim3(B, H), kThreads, sizeof(int32_t) * (size_t)sample_smem_rows, s>>>(p, sample_smem_rows);
    KM_CHECK();
    const dim3 dist_grid((p.n_init_max + kSumBlock - 1) / kSumBlock, (p.trials_max + kDistTrials - 1) / kDistTrials, pairs);
    const size_t draw_smem = sizeof(double) * ((size_t)p.n_init_max + 2 * kMaxSumBlocks);
    if ((err = cudaFuncSetAttribute(km_accept_kernel<kHalf>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)draw_smem)) != cudaSuccess)
        return err;
    for (int c = 0; c < p.k_max; ++c) {
        km_candidate_dist_kernel<kHalf><<<dist_grid, kDistThreads, 0, s>>>(p, c);
        KM_CHECK();
        km_accept_kernel<kHalf><<<dim3(B, H), kAcceptThreads, draw_smem, s>>>(p, c);     // ... and the trial points of centre c + 1
        KM_CHECK();
    }
    if ((err = cudaMemsetAsync(p.count, 0, sizeof(double) * (size_t)H * p.centres_total, s)) != cudaSuccess) return err;
    if ((err = cudaMemsetAsync(p.state, 0, sizeof(KmeansState) * (size_t)pairs, s)) != cudaSuccess) return err;
    const size_t control_smem = sizeof(double) * (size_t)p.batch + sizeof(int32_t) * ((size_t)p.batch + (size_t)p.batch / 2 + 1);
    if ((err = cudaFuncSetAttribute(km_control_kernel<kHalf>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)control_smem)) != cudaSuccess)
        return err;
    for (int t = 0; t < p.t_max_max; ++t) {
        km_batch_assign_kernel<kHalf><<<dim3((p.batch + kAssignBlock - 1) / kAssignBlock, pairs, p.assign_split), 128, 0, s>>>(p, t);
        KM_CHECK();
        if (p.assign_split > 1) {
            km_assign_reduce_kernel<<<dim3((p.batch + 127) / 128, pairs), 128, 0, s>>>(p, t);
            KM_CHECK();
        }
        km_sort_batch_kernel<<<dim3(pairs), kSortThreads, 0, s>>>(p, t);
        KM_CHECK();
        km_batch_update_kernel<kHalf><<<dim3((p.k_max + 1) / 2, pairs), kThreads, 0, s>>>(p, t);
        KM_CHECK();
        km_control_kernel<kHalf><<<dim3(B, H), kThreads, control_smem, s>>>(p, t);
        KM_CHECK();
        if (!p.no_host_poll && (t + 1) % kPollEvery == 0 && t + 1 < p.t_max_max) {
            // most fits stop long before the step limit: ask the device how many are still running
            // (the copy into pageable memory returns when it has completed)
            int active = 1;
            km_count_active_kernel<<<1, kThreads, 0, s>>>(p, t);
            KM_CHECK();
            if ((err = cudaMemcpyAsync(&active, p.active, sizeof(int), cudaMemcpyDeviceToHost, s)) != cudaSuccess) return err;
            if ((err = cudaStreamSynchronize(s)) != cudaSuccess) return err;
            if (active == 0) break;
        }
    }
    km_finish_kernel<<<dim3((p.k_max * kHeadDim + kThreads - 1) / kThreads, B, H), kThreads, 0, s>>>(p);
    KM_CHECK();
#undef KM_CHECK
    return cudaSuccess;
}

}  // namespace

namespace {
__global__ void __launch_bounds__(kKmTableChunk + 32)
km_tables_kernel(const __grid_constant__ KmTableChunk c, int64_t *row_off, int64_t *centre_off, int32_t *n_init,
                 int32_t *trials, int32_t *t_max)
{
    const int i = threadIdx.x;
    if (i <= c.n) {
        row_off[c.first + i] = c.row_off[i];
        centre_off[c.first + i] = c.centre_off[i];
    }
    if (i < c.n) {
        n_init[c.first + i] = c.n_init[i];
        trials[c.first + i] = c.trials[i];
        t_max[c.first + i] = c.t_max[i];
    }
}
}  // namespace

cudaError_t launch_kmeans_tables(const KmTableChunk &c, int64_t *row_off, int64_t *centre_off, int32_t *n_init,
                                 int32_t *trials, int32_t *t_max, cudaStream_t s)
{
    km_tables_kernel<<<1, kKmTableChunk + 32, 0, s>>>(c, row_off, centre_off, n_init, trials, t_max);
    return cudaGetLastError();
}

cudaError_t launch_kmeans_fit(const KmeansParams &p, cudaStream_t s)
{
    return p.elem ? run_fit<true>(p, s) : run_fit<false>(p, s);
}

}  // namespace santapp
