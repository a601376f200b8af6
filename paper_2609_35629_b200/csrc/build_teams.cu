// santapp_build_teams: contiguous parents (Algorithm 4) and actual-key teams (Algorithm 2),
// written as a team-contiguous copy of K/V with CSR offsets. Preparation path, run once after
// prefill; distances are evaluated in fp64 in a fixed order (token index, then dimension) with
// separate multiply and add, so that exact ties fall the way the paper's tie rules say.
#include <limits.h>

#include "build_util.cuh"
#include "common.cuh"

namespace santapp {

namespace {

constexpr int kBuildThreads = 256;
constexpr int kRowWords = 65;            // 64 data words + 1 pad word: conflict-free column walks

// Squared distance between row `i` (shared memory, bf16 words) and a reference vector in fp64,
// summed over dimensions in increasing order, multiply and add rounded separately.
template <bool kHalf>
__device__ __forceinline__ double sqdist_row_vec(const uint32_t *row, const double *ref)
{
    double s = 0.0;
#pragma unroll 8
    for (int w = 0; w < 64; ++w) {
        const uint32_t word = row[w];
        const double e0 = __dsub_rn((double)elem_lo<kHalf>(word), ref[2 * w]);
        const double e1 = __dsub_rn((double)elem_hi<kHalf>(word), ref[2 * w + 1]);
        s = __dadd_rn(s, __dmul_rn(e0, e0));
        s = __dadd_rn(s, __dmul_rn(e1, e1));
    }
    return s;
}

template <bool kHalf>
__device__ __forceinline__ double sqdist_row_row(const uint32_t *row, const uint32_t *ref)
{
    double s = 0.0;
#pragma unroll 8
    for (int w = 0; w < 64; ++w) {
        const uint32_t a = row[w], b = ref[w];
        const double e0 = __dsub_rn((double)elem_lo<kHalf>(a), (double)elem_lo<kHalf>(b));
        const double e1 = __dsub_rn((double)elem_hi<kHalf>(a), (double)elem_hi<kHalf>(b));
        s = __dadd_rn(s, __dmul_rn(e0, e0));
        s = __dadd_rn(s, __dmul_rn(e1, e1));
    }
    return s;
}

// One block per (parent, sequence, KV head): representatives, owners, team sizes.
template <bool kHalf>
__global__ void __launch_bounds__(kBuildThreads)
build_parent_kernel(BuildParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int parent = blockIdx.x, b = blockIdx.y, j = blockIdx.z;
    const int64_t row0 = p.bv.seq_row_off[b];
    const int N = (int)(p.bv.seq_row_off[b + 1] - row0);
    const int P = p.parent_size;
    const int first = parent * P;
    if (first >= N) return;
    const int nC = min(P, N - first);
    const int r = min(p.reps, nC);
    const int tid = threadIdx.x;

    double *mu = reinterpret_cast<double *>(smem_raw);                    // [128]
    double *mind = mu + kHeadDim;                                         // [P]
    ValIdx *scratch = reinterpret_cast<ValIdx *>(mind + P);               // [33]
    uint32_t *rows = reinterpret_cast<uint32_t *>(scratch + 33);          // [P][kRowWords]
    int *owner = reinterpret_cast<int *>(rows + (size_t)P * kRowWords);   // [P]
    int *count = owner + P;                                               // [P] (r used)
    int *rep_of = count + P;                                              // [P] (r used): row inside parent
    unsigned char *is_rep = reinterpret_cast<unsigned char *>(rep_of + P);  // [P]

    const uint32_t *src = reinterpret_cast<const uint32_t *>(p.k_prompt)
                          + ((size_t)j * p.bv.rows_total + row0 + first) * 64;
    for (int e = tid; e < nC * 64; e += kBuildThreads) rows[(e >> 6) * kRowWords + (e & 63)] = src[e];
    for (int i = tid; i < nC; i += kBuildThreads) { is_rep[i] = 0; count[i] = 0; }
    __syncthreads();

    // parent mean: rows added in token order, then one division
    if (tid < kHeadDim) {
        double s = 0.0;
        const int w = tid >> 1;
        const bool hi = tid & 1;
        for (int i = 0; i < nC; ++i) {
            const uint32_t word = rows[i * kRowWords + w];
            s = __dadd_rn(s, (double)(hi ? elem_hi<kHalf>(word) : elem_lo<kHalf>(word)));
        }
        mu[tid] = __ddiv_rn(s, (double)nC);
    }
    __syncthreads();

    // first representative: the actual key nearest the mean
    {
        ValIdx best = {INFINITY, INT_MAX};
        for (int i = tid; i < nC; i += kBuildThreads) {
            ValIdx c = {sqdist_row_vec<kHalf>(rows + i * kRowWords, mu), i};
            best = pick<true>(best, c);
        }
        best = block_arg<true>(best, scratch);
        if (tid == 0) { rep_of[0] = best.i; is_rep[best.i] = 1; }
    }
    __syncthreads();

    // farthest-first representatives; the running (nearest distance, owner) pair is the
    // nearest-representative assignment with ties going to the earlier-selected one
    for (int i = tid; i < nC; i += kBuildThreads) { mind[i] = INFINITY; owner[i] = 0; }
    for (int u = 0; u < r; ++u) {
        const uint32_t *ref = rows + rep_of[u] * kRowWords;
        ValIdx far = {-2.0, INT_MAX};
        for (int i = tid; i < nC; i += kBuildThreads) {
            const double dist = sqdist_row_row<kHalf>(rows + i * kRowWords, ref);
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
    // representative self-ownership
    for (int u = tid; u < r; u += kBuildThreads) owner[rep_of[u]] = u;
    __syncthreads();

    for (int i = tid; i < nC; i += kBuildThreads) atomicAdd(&count[owner[i]], 1);
    __syncthreads();

    // outputs: owner per row, team sizes (scanned later), representative keys
    uint16_t *owner_out = p.owner + (size_t)j * p.bv.rows_total + row0 + first;
    for (int i = tid; i < nC; i += kBuildThreads) owner_out[i] = (uint16_t)owner[i];

    const int64_t team0 = p.bv.seq_team_off[b];
    const int team_local0 = parent * p.teams_per_full_parent;
    int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    if (parent == 0 && tid == 0) csr[0] = 0;
    for (int u = tid; u < r; u += kBuildThreads) csr[1 + team_local0 + u] = count[u];

    uint32_t *rep_dst = reinterpret_cast<uint32_t *>(p.rep_keys)
                        + ((size_t)j * p.bv.teams_total + team0 + team_local0) * 64;
    for (int e = tid; e < r * 64; e += kBuildThreads)
        rep_dst[e] = rows[rep_of[e >> 6] * kRowWords + (e & 63)];
}

// One block per (sequence, KV head): team sizes -> CSR row offsets (inclusive scan in place).
__global__ void __launch_bounds__(kBuildThreads)
scan_team_sizes_kernel(BuildParams p)
{
    __shared__ int scratch[33];
    const int b = blockIdx.x, j = blockIdx.y;
    const int64_t team0 = p.bv.seq_team_off[b];
    const int M = (int)(p.bv.seq_team_off[b + 1] - team0);
    int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b + 1;
    if (threadIdx.x == 0 && p.team_count) p.team_count[(size_t)j * p.bv.n_seqs + b] = M;   // every slot is a team
    int carry = 0;
    for (int base = 0; base < M; base += kBuildThreads) {
        const int g = base + threadIdx.x;
        const int v = g < M ? csr[g] : 0;
        int total;
        const int excl = block_exclusive_scan(v, scratch, total);
        if (g < M) csr[g] = carry + excl + v;
        carry += total;
    }
}

// One block per (parent, sequence, KV head): stable partition of the parent's rows by team and
// copy of K/V rows into the packed layout.
__global__ void __launch_bounds__(kBuildThreads)
pack_parent_kernel(BuildParams p)
{
    __shared__ uint16_t owner[kMaxParent];
    __shared__ int dest[kMaxParent];
    const int parent = blockIdx.x, b = blockIdx.y, j = blockIdx.z;
    const int64_t row0 = p.bv.seq_row_off[b];
    const int N = (int)(p.bv.seq_row_off[b + 1] - row0);
    const int P = p.parent_size;
    const int first = parent * P;
    if (first >= N) return;
    const int nC = min(P, N - first);
    const int tid = threadIdx.x;

    const uint16_t *owner_in = p.owner + (size_t)j * p.bv.rows_total + row0 + first;
    for (int i = tid; i < nC; i += kBuildThreads) owner[i] = owner_in[i];
    __syncthreads();

    const int64_t team0 = p.bv.seq_team_off[b];
    const int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    const int team_local0 = parent * p.teams_per_full_parent;
    for (int i = tid; i < nC; i += kBuildThreads) {
        const int u = owner[i];
        int rank = 0;
        for (int a = 0; a < i; ++a) rank += (owner[a] == u);
        dest[i] = csr[team_local0 + u] + rank;              // members in increasing token index
    }
    __syncthreads();

    const size_t plane = (size_t)j * p.bv.rows_total + row0;
    const uint2 *ksrc = reinterpret_cast<const uint2 *>(p.k_prompt) + (plane + first) * 32;
    const uint2 *vsrc = reinterpret_cast<const uint2 *>(p.v_prompt) + (plane + first) * 32;
    uint2 *kdst = reinterpret_cast<uint2 *>(p.k_packed) + plane * 32;
    uint2 *vdst = reinterpret_cast<uint2 *>(p.v_packed) + plane * 32;
    const int lane = tid & 31, warp = tid >> 5;
    for (int i = warp; i < nC; i += kBuildThreads / 32) {
        const size_t d = (size_t)dest[i] * 32 + lane;
        kdst[d] = ksrc[(size_t)i * 32 + lane];
        vdst[d] = vsrc[(size_t)i * 32 + lane];
    }
    int32_t *tok = p.row_token + plane;
    for (int i = tid; i < nC; i += kBuildThreads) tok[dest[i]] = first + i;
}

size_t build_parent_smem(int P)
{
    return sizeof(double) * (kHeadDim + P) + sizeof(ValIdx) * 33 + sizeof(uint32_t) * (size_t)P * kRowWords
           + sizeof(int) * 3 * (size_t)P + (size_t)P + 16;
}

// Centroid-guided baseline of the paper's routing diagnostic, on the contiguous parents of
// Algorithm 4: one group per parent, routed by the arithmetic mean of its keys. A block per
// (parent, sequence, KV head), a thread per dimension: the mean is the fp64 sum in token order
// divided by the count, stored like every routing key as a 16-bit element (fp64 -> fp32 to nearest,
// then fp32 -> bf16 or fp16 to nearest even). Rows keep their token order, so the packed copies are copies.
template <bool kHalf>
__global__ void __launch_bounds__(kHeadDim)
group_mean_kernel(BuildParams p)
{
    const int parent = blockIdx.x, b = blockIdx.y, j = blockIdx.z, d = threadIdx.x;
    const int64_t row0 = p.bv.seq_row_off[b];
    const int N = (int)(p.bv.seq_row_off[b + 1] - row0);
    const int n_parents = (N + p.parent_size - 1) / p.parent_size;
    if (parent >= n_parents) return;
    const int lo = parent * p.parent_size, hi = min(lo + p.parent_size, N);
    const size_t plane = (size_t)j * p.bv.rows_total + (size_t)row0;
    const uint16_t *k = p.k_prompt + plane * kHeadDim;
    double sum = 0.0;
    for (int i = lo; i < hi; ++i) sum = __dadd_rn(sum, elem_to_double<kHalf>(k[(size_t)i * kHeadDim + d]));
    const int64_t team0 = p.bv.seq_team_off[b];                     // one team per parent
    p.rep_keys[((size_t)j * p.bv.teams_total + (size_t)team0 + parent) * kHeadDim + d] =
        double_to_elem<kHalf>(__ddiv_rn(sum, (double)(hi - lo)));
    int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    if (d == 0) {
        csr[parent] = lo;
        if (parent == n_parents - 1) csr[n_parents] = N;
        if (parent == 0 && p.team_count) p.team_count[(size_t)j * p.bv.n_seqs + b] = n_parents;
    }
    for (int i = lo + d; i < hi; i += kHeadDim) p.row_token[plane + i] = i;
    const uint4 *ks = reinterpret_cast<const uint4 *>(p.k_prompt + (plane + lo) * kHeadDim);
    const uint4 *vs = reinterpret_cast<const uint4 *>(p.v_prompt + (plane + lo) * kHeadDim);
    uint4 *kd = reinterpret_cast<uint4 *>(p.k_packed + (plane + lo) * kHeadDim);
    uint4 *vd = reinterpret_cast<uint4 *>(p.v_packed + (plane + lo) * kHeadDim);
    for (int idx = d; idx < (hi - lo) * (kHeadDim / 8); idx += kHeadDim) {
        kd[idx] = ks[idx];
        vd[idx] = vs[idx];
    }
}

}  // namespace

cudaError_t launch_build_groups_mean(const BuildParams &p, cudaStream_t s)
{
    dim3 grid(p.max_parents_per_seq, p.bv.n_seqs, p.bv.n_kv);
    if (p.bv.elem) group_mean_kernel<true><<<grid, kHeadDim, 0, s>>>(p);
    else           group_mean_kernel<false><<<grid, kHeadDim, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_build_teams(const BuildParams &p, cudaStream_t s)
{
    const size_t smem = build_parent_smem(p.parent_size);
    cudaError_t err = cudaFuncSetAttribute(p.bv.elem ? build_parent_kernel<true> : build_parent_kernel<false>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    dim3 grid(p.max_parents_per_seq, p.bv.n_seqs, p.bv.n_kv);
    if (p.bv.elem) build_parent_kernel<true><<<grid, kBuildThreads, smem, s>>>(p);
    else           build_parent_kernel<false><<<grid, kBuildThreads, smem, s>>>(p);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    scan_team_sizes_kernel<<<dim3(p.bv.n_seqs, p.bv.n_kv), kBuildThreads, 0, s>>>(p);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    pack_parent_kernel<<<grid, kBuildThreads, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace santapp
