// Team records from an arbitrary parent partition (the partition Algorithm 3 returns: parents of
// any size, in centre order, empty ones omitted), and the nearest-centre assignment that closes
// Algorithm 3. Preparation path, run once after prefill. As in the contiguous builder, distances
// are fp64, summed over dimensions in increasing order with separately rounded multiply and add,
// so exact ties fall the way the paper's tie rules say.
//
// Steps: count the tokens of each label; scan the counts into member-list offsets and number the
// teams (a parent of c tokens yields min(R, c)); list each parent's tokens in increasing index
// (stable scatter); Algorithm 2 per non-empty parent; scan team sizes into CSR offsets; stable
// scatter of the tokens by team; copy K/V rows into the team-contiguous layout.
#include <limits.h>

#include <algorithm>

#include "build_util.cuh"
#include "common.cuh"

namespace santapp {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ int clamp_label(int v, int n) { return min(max(v, 0), n - 1); }

// ---- Algorithm 3, assignment step: b_i = argmin_u |k_i - mu_u|^2, ties to the smaller u ----
constexpr int kAssignThreads = 128;
constexpr int kAssignPts = 2;             // tokens per thread
constexpr int kAssignGroup = 8;           // centres per pass
constexpr int kCentreTile = 16;
static_assert(kCentreTile % kAssignGroup == 0, "a tile of centres is a whole number of passes");

// A thread holds two tokens and takes eight centres at a time (dist_points: a centre value read from
// shared memory serves both tokens, a token value is widened once for the eight centres).
template <bool kHalf>
__global__ void __launch_bounds__(kAssignThreads)
assign_parents_kernel(AssignParams p)
{
    __shared__ __align__(16) double c[kCentreTile][kHeadDim];
    const int b = blockIdx.y, j = blockIdx.z, tid = threadIdx.x;
    const int64_t row0 = p.seq_row_off[b];
    const int N = (int)(p.seq_row_off[b + 1] - row0);
    if ((int)(blockIdx.x * kAssignThreads * kAssignPts) >= N) return;
    const int64_t c0off = p.seq_centre_off[b];
    const int n_centres = (int)(p.seq_centre_off[b + 1] - c0off);
    int i[kAssignPts], arg[kAssignPts];
    const uint4 *row[kAssignPts];
    double best[kAssignPts];
#pragma unroll
    for (int u = 0; u < kAssignPts; ++u) {
        i[u] = (blockIdx.x * kAssignPts + u) * kAssignThreads + tid;
        row[u] = reinterpret_cast<const uint4 *>(p.k_prompt + ((size_t)j * p.rows_total + row0 + min(i[u], N - 1)) * kHeadDim);
        best[u] = INFINITY;
        arg[u] = 0;
    }
    const float *cen = p.centres + ((size_t)j * p.centres_total + c0off) * kHeadDim;
    for (int base = 0; base < n_centres; base += kCentreTile) {
        const int nt = min(kCentreTile, n_centres - base);
        __syncthreads();
        for (int e = tid; e < nt * kHeadDim; e += kAssignThreads)
            c[e >> 7][e & 127] = (double)cen[(size_t)base * kHeadDim + e];
        __syncthreads();
        for (int t = 0; t < nt; t += kAssignGroup) {
            // (rows of the tile past nt hold older values; their sums are not looked at)
            double s[kAssignPts][kAssignGroup];
#pragma unroll
            for (int u = 0; u < kAssignPts; ++u)
#pragma unroll
                for (int v = 0; v < kAssignGroup; ++v) s[u][v] = 0.0;
            dist_points<kHalf, kAssignPts, kAssignGroup, kAssignGroup>(row, c + t, s);
#pragma unroll
            for (int u = 0; u < kAssignPts; ++u)
#pragma unroll
                for (int v = 0; v < kAssignGroup; ++v)
                    if (t + v < nt && s[u][v] < best[u]) { best[u] = s[u][v]; arg[u] = base + t + v; }
        }
    }
#pragma unroll
    for (int u = 0; u < kAssignPts; ++u)
        if (i[u] < N) p.parent_of[(size_t)j * p.rows_total + row0 + i[u]] = arg[u];
}

// ---- token counts per label ----
__global__ void __launch_bounds__(kThreads)
count_labels_kernel(ParentBuildParams p)
{
    const int b = blockIdx.y, j = blockIdx.z;
    const int64_t row0 = p.bv.seq_row_off[b];
    const int N = (int)(p.bv.seq_row_off[b + 1] - row0);
    const int i = blockIdx.x * kThreads + threadIdx.x;
    if (i >= N) return;
    const int64_t l0 = p.seq_label_off[b];
    const int n_labels = (int)(p.seq_label_off[b + 1] - l0);
    const int u = clamp_label(p.parent_of[(size_t)j * p.bv.rows_total + row0 + i], n_labels);
    atomicAdd(p.parent_cursor + (size_t)j * p.labels_total + l0 + u, 1);
}

// One block per (sequence, KV head): counts -> member-list offsets, team numbering, team count.
__global__ void __launch_bounds__(kThreads)
scan_parents_kernel(ParentBuildParams p)
{
    __shared__ int scratch[33];
    const int b = blockIdx.x, j = blockIdx.y;
    const int64_t l0 = p.seq_label_off[b];
    const int n_labels = (int)(p.seq_label_off[b + 1] - l0);
    int32_t *cursor = p.parent_cursor + (size_t)j * p.labels_total + l0;
    int32_t *tbase = p.parent_team_base + (size_t)j * p.labels_total + l0;
    int32_t *pstart = p.parent_start + (size_t)j * (p.labels_total + p.bv.n_seqs) + l0 + b;
    int rows_carry = 0, teams_carry = 0;
    for (int base = 0; base < n_labels; base += kThreads) {
        const int u = base + threadIdx.x;
        const int cnt = u < n_labels ? cursor[u] : 0;
        const int r = min(cnt, p.reps);
        int rows_total, teams_total;
        const int rows_excl = block_exclusive_scan(cnt, scratch, rows_total);
        const int teams_excl = block_exclusive_scan(r, scratch, teams_total);
        if (u < n_labels) {
            pstart[u] = rows_carry + rows_excl;
            cursor[u] = rows_carry + rows_excl;
            tbase[u] = teams_carry + teams_excl;
        }
        rows_carry += rows_total;
        teams_carry += teams_total;
    }
    if (threadIdx.x == 0) {
        pstart[n_labels] = rows_carry;
        p.team_count[(size_t)j * p.bv.n_seqs + b] = teams_carry;
    }
}

// One block per (sequence, KV head): position of every token in the list ordered by (label, token
// index). One warp takes the tokens 32 at a time in increasing index; lanes with the same label
// form a group whose lowest lane reserves the group's slots at the label's cursor, and each lane
// takes the slot of its rank inside the group. The full-warp shuffle that hands the reserved base
// round also makes every reservation of one step complete before the next step begins. The
// cursors are copied into shared memory by the whole block when they fit (smem_labels of them: a
// step then costs a shared-memory atomic instead of a round trip to L2; they are not needed
// afterwards), and a step's labels are requested one step ahead.
//   kInverse: out[position] = token (member lists); otherwise out[token] = position.
constexpr int kScatterSmemLabels = 50 * 1024;               // cursors that fit in shared memory (200 KB)
template <bool kInverse>
__global__ void __launch_bounds__(kThreads)
stable_scatter_kernel(const int32_t *labels, int32_t *cursors, int32_t *out, const int64_t *seq_row_off,
                      const int64_t *seq_label_off, int64_t rows_total, int64_t labels_total, int smem_labels)
{
    extern __shared__ int32_t cur_s[];
    const int b = blockIdx.x, j = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
    const int64_t row0 = seq_row_off[b];
    const int N = (int)(seq_row_off[b + 1] - row0);
    const int64_t l0 = seq_label_off[b];
    const int n_labels = (int)(seq_label_off[b + 1] - l0);
    const int32_t *lab = labels + (size_t)j * rows_total + row0;
    int32_t *cur = cursors + (size_t)j * labels_total + l0;
    int32_t *dst = out + (size_t)j * rows_total + row0;
    const bool in_smem = n_labels <= smem_labels;
    if (in_smem)
        for (int u = tid; u < n_labels; u += kThreads) cur_s[u] = cur[u];
    __syncthreads();
    if (tid >= 32) return;
    int next = lane < N ? lab[lane] : 0;
    for (int i0 = 0; i0 < N; i0 += 32) {
        const int i = i0 + lane;
        const bool valid = i < N;
        const int mine = next;
        if (i + 32 < N) next = lab[i + 32];
        const int u = valid ? clamp_label(mine, n_labels) : -1 - lane;         // idle lanes stay alone
        const unsigned group = __match_any_sync(0xFFFFFFFFu, u);
        const int leader = __ffs(group) - 1;
        const int rank = __popc(group & ((1u << lane) - 1u));
        int base = 0;
        if (valid && lane == leader) base = in_smem ? atomicAdd(cur_s + u, __popc(group)) : atomicAdd(cur + u, __popc(group));
        base = __shfl_sync(0xFFFFFFFFu, base, leader);
        if (valid) {
            if (kInverse) dst[base + rank] = i;
            else dst[i] = base + rank;
        }
    }
}

template <bool kHalf>
__device__ __forceinline__ double sqdist_grow_vec(const uint4 *row, const double *ref)
{
    double s = 0.0;
#pragma unroll 4
    for (int q = 0; q < 16; ++q) {
        const uint4 w4 = row[q];
        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const double e0 = __dsub_rn((double)elem_lo<kHalf>(w[t]), ref[8 * q + 2 * t]);
            const double e1 = __dsub_rn((double)elem_hi<kHalf>(w[t]), ref[8 * q + 2 * t + 1]);
            s = __dadd_rn(s, __dmul_rn(e0, e0));
            s = __dadd_rn(s, __dmul_rn(e1, e1));
        }
    }
    return s;
}

template <bool kHalf>
__device__ __forceinline__ double sqdist_grow_row(const uint4 *row, const uint32_t *ref)
{
    double s = 0.0;
#pragma unroll 4
    for (int q = 0; q < 16; ++q) {
        const uint4 w4 = row[q];
        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const uint32_t r = ref[4 * q + t];
            const double e0 = __dsub_rn((double)elem_lo<kHalf>(w[t]), (double)elem_lo<kHalf>(r));
            const double e1 = __dsub_rn((double)elem_hi<kHalf>(w[t]), (double)elem_hi<kHalf>(r));
            s = __dadd_rn(s, __dmul_rn(e0, e0));
            s = __dadd_rn(s, __dmul_rn(e1, e1));
        }
    }
    return s;
}

// Algorithm 2 for one parent of any size. One block per (label, sequence, KV head); the parent's
// tokens are read through its member list, and the per-member state lives in global memory.
template <bool kHalf>
__global__ void __launch_bounds__(kThreads)
build_parent_general_kernel(ParentBuildParams p)
{
    __shared__ double mu[kHeadDim];
    __shared__ uint32_t ref[64];
    __shared__ ValIdx scratch[33];
    __shared__ int count[kMaxParent];
    __shared__ int rep_pos[kMaxParent];
    const int u_parent = blockIdx.x, b = blockIdx.y, j = blockIdx.z, tid = threadIdx.x;
    const int64_t l0 = p.seq_label_off[b];
    const int n_labels = (int)(p.seq_label_off[b + 1] - l0);
    if (u_parent >= n_labels) return;
    const int32_t *pstart = p.parent_start + (size_t)j * (p.labels_total + p.bv.n_seqs) + l0 + b;
    const int s0 = pstart[u_parent];
    const int nC = pstart[u_parent + 1] - s0;
    if (nC == 0) return;                                   // empty parents are omitted
    const int r = min(p.reps, nC);
    const int64_t row0 = p.bv.seq_row_off[b];
    const size_t plane = (size_t)j * p.bv.rows_total + row0;
    const int32_t *mem = p.members + plane + s0;
    double *mind = p.mind + plane + s0;
    int32_t *owner = p.owner + plane + s0;
    unsigned char *is_rep = p.is_rep + plane + s0;
    const uint4 *kbase = reinterpret_cast<const uint4 *>(p.k_prompt + plane * kHeadDim);   // 16 per row

    for (int i = tid; i < nC; i += kThreads) { is_rep[i] = 0; mind[i] = INFINITY; owner[i] = 0; }
    for (int u = tid; u < r; u += kThreads) count[u] = 0;

    // parent mean: rows added in token order, then one division
    if (tid < kHeadDim) {
        const uint16_t *col = p.k_prompt + plane * kHeadDim + tid;
        double s = 0.0;
        for (int i = 0; i < nC; ++i) s = __dadd_rn(s, elem_to_double<kHalf>(col[(size_t)mem[i] * kHeadDim]));
        mu[tid] = __ddiv_rn(s, (double)nC);
    }
    __syncthreads();

    if (p.mean_keys) {
        // centroid-guided baseline: the parent is one group, routed by its mean stored as a 16-bit
        // element (fp64 -> fp32 to nearest, fp32 -> bf16 or fp16 to nearest even)
        const int tb = p.parent_team_base[(size_t)j * p.labels_total + l0 + u_parent];
        const int64_t t0 = p.bv.seq_team_off[b];
        int32_t *tof = p.team_of + plane;
        for (int i = tid; i < nC; i += kThreads) tof[mem[i]] = tb;
        if (tid == 0) p.team_row_start[(size_t)j * (p.bv.teams_total + p.bv.n_seqs) + t0 + b + 1 + tb] = nC;
        if (tid < kHeadDim)
            p.rep_keys[((size_t)j * p.bv.teams_total + t0 + tb) * kHeadDim + tid] = double_to_elem<kHalf>(mu[tid]);
        return;
    }

    // first representative: the actual key nearest the mean
    {
        ValIdx best = {INFINITY, INT_MAX};
        for (int i = tid; i < nC; i += kThreads) {
            ValIdx c = {sqdist_grow_vec<kHalf>(kbase + (size_t)mem[i] * 16, mu), i};
            best = pick<true>(best, c);
        }
        best = block_arg<true>(best, scratch);
        if (tid == 0) { rep_pos[0] = best.i; is_rep[best.i] = 1; }
    }
    __syncthreads();

    // farthest-first representatives; the running (nearest distance, owner) pair is the
    // nearest-representative assignment with ties going to the earlier-selected one
    for (int u = 0; u < r; ++u) {
        if (tid < 64) ref[tid] = reinterpret_cast<const uint32_t *>(kbase + (size_t)mem[rep_pos[u]] * 16)[tid];
        __syncthreads();
        ValIdx far = {-2.0, INT_MAX};
        for (int i = tid; i < nC; i += kThreads) {
            const double dist = sqdist_grow_row<kHalf>(kbase + (size_t)mem[i] * 16, ref);
            double m = mind[i];
            if (dist < m) { m = dist; mind[i] = dist; owner[i] = u; }
            ValIdx c = {is_rep[i] ? -1.0 : m, i};
            far = pick<false>(far, c);
        }
        if (u + 1 < r) {
            far = block_arg<false>(far, scratch);
            if (tid == 0) { rep_pos[u + 1] = far.i; is_rep[far.i] = 1; }
        }
        __syncthreads();
    }
    // representative self-ownership
    for (int u = tid; u < r; u += kThreads) owner[rep_pos[u]] = u;
    __syncthreads();
    for (int i = tid; i < nC; i += kThreads) atomicAdd(&count[owner[i]], 1);
    __syncthreads();

    // outputs: team of every token, team sizes (scanned later), representative keys
    const int tbase = p.parent_team_base[(size_t)j * p.labels_total + l0 + u_parent];
    int32_t *team_of = p.team_of + plane;
    for (int i = tid; i < nC; i += kThreads) team_of[mem[i]] = tbase + owner[i];
    const int64_t team0 = p.bv.seq_team_off[b];
    int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    for (int u = tid; u < r; u += kThreads) csr[1 + tbase + u] = count[u];
    uint32_t *rep_dst = reinterpret_cast<uint32_t *>(p.rep_keys) + ((size_t)j * p.bv.teams_total + team0 + tbase) * 64;
    for (int e = tid; e < r * 64; e += kThreads)
        rep_dst[e] = reinterpret_cast<const uint32_t *>(kbase + (size_t)mem[rep_pos[e >> 6]] * 16)[e & 63];
}

// One block per (sequence, KV head): team sizes -> CSR row offsets; the slots behind the pair's
// last team are empty teams (offset = prompt length); the cursors of the scatter by team.
__global__ void __launch_bounds__(kThreads)
scan_teams_kernel(ParentBuildParams p)
{
    __shared__ int scratch[33];
    const int b = blockIdx.x, j = blockIdx.y;
    const int64_t team0 = p.bv.seq_team_off[b];
    const int slots = (int)(p.bv.seq_team_off[b + 1] - team0);
    const int M = p.team_count[(size_t)j * p.bv.n_seqs + b];
    const int N = (int)(p.bv.seq_row_off[b + 1] - p.bv.seq_row_off[b]);
    int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    int32_t *cursor = p.team_cursor + (size_t)j * p.bv.teams_total + team0;
    int carry = 0;
    for (int base = 0; base < slots; base += kThreads) {
        const int g = base + threadIdx.x;
        const int v = g < M ? csr[1 + g] : 0;
        int total;
        const int excl = block_exclusive_scan(v, scratch, total);
        if (g < slots) {
            csr[1 + g] = g < M ? carry + excl + v : N;
            cursor[g] = g < M ? carry + excl : N;
        }
        carry += total;
    }
    if (threadIdx.x == 0) csr[0] = 0;
}

// One warp per row: copy the K/V rows to their packed position.
__global__ void __launch_bounds__(kThreads)
pack_rows_kernel(ParentBuildParams p)
{
    const int b = blockIdx.y, j = blockIdx.z;
    const int64_t row0 = p.bv.seq_row_off[b];
    const int N = (int)(p.bv.seq_row_off[b + 1] - row0);
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (i >= N) return;
    const size_t plane = (size_t)j * p.bv.rows_total + row0;
    const int d = p.dest[plane + i];
    const uint2 *ksrc = reinterpret_cast<const uint2 *>(p.k_prompt) + (plane + i) * 32;
    const uint2 *vsrc = reinterpret_cast<const uint2 *>(p.v_prompt) + (plane + i) * 32;
    uint2 *kdst = reinterpret_cast<uint2 *>(p.k_packed) + (plane + d) * 32;
    uint2 *vdst = reinterpret_cast<uint2 *>(p.v_packed) + (plane + d) * 32;
    kdst[lane] = ksrc[lane];
    vdst[lane] = vsrc[lane];
    if (lane == 0) p.row_token[plane + d] = i;
}

}  // namespace

cudaError_t launch_assign_parents(const AssignParams &p, cudaStream_t s)
{
    dim3 grid((p.max_rows_per_seq + kAssignThreads * kAssignPts - 1) / (kAssignThreads * kAssignPts), p.n_seqs, p.n_kv);
    if (p.elem) assign_parents_kernel<true><<<grid, kAssignThreads, 0, s>>>(p);
    else        assign_parents_kernel<false><<<grid, kAssignThreads, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_build_teams_parents(const ParentBuildParams &p, cudaStream_t s)
{
    const int B = p.bv.n_seqs, H = p.bv.n_kv;
    cudaError_t err = cudaMemsetAsync(p.parent_cursor, 0, sizeof(int32_t) * (size_t)H * p.labels_total, s);
    if (err != cudaSuccess) return err;
    // representative keys of the empty slots are zero
    err = cudaMemsetAsync(p.rep_keys, 0, sizeof(uint16_t) * (size_t)H * p.bv.teams_total * kHeadDim, s);
    if (err != cudaSuccess) return err;
    count_labels_kernel<<<dim3((p.max_rows_per_seq + kThreads - 1) / kThreads, B, H), kThreads, 0, s>>>(p);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    scan_parents_kernel<<<dim3(B, H), kThreads, 0, s>>>(p);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    // cursors in shared memory when a sequence's labels (teams: at most reps per label) fit
    const int lab_smem = std::min(p.max_labels_per_seq, kScatterSmemLabels);
    const long long max_teams = (long long)p.max_labels_per_seq * p.reps;
    const int team_smem = (int)std::min<long long>(max_teams, kScatterSmemLabels);
    if ((err = cudaFuncSetAttribute(stable_scatter_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)sizeof(int32_t) * kScatterSmemLabels)) != cudaSuccess) return err;
    if ((err = cudaFuncSetAttribute(stable_scatter_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)sizeof(int32_t) * kScatterSmemLabels)) != cudaSuccess) return err;
    stable_scatter_kernel<true><<<dim3(B, H), kThreads, sizeof(int32_t) * (size_t)lab_smem, s>>>(
        p.parent_of, p.parent_cursor, p.members, p.bv.seq_row_off, p.seq_label_off, p.bv.rows_total, p.labels_total, lab_smem);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    if (p.bv.elem) build_parent_general_kernel<true><<<dim3(p.max_labels_per_seq, B, H), kThreads, 0, s>>>(p);
    else           build_parent_general_kernel<false><<<dim3(p.max_labels_per_seq, B, H), kThreads, 0, s>>>(p);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    scan_teams_kernel<<<dim3(B, H), kThreads, 0, s>>>(p);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    stable_scatter_kernel<false><<<dim3(B, H), kThreads, sizeof(int32_t) * (size_t)team_smem, s>>>(
        p.team_of, p.team_cursor, p.dest, p.bv.seq_row_off, p.bv.seq_team_off, p.bv.rows_total, p.bv.teams_total, team_smem);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    pack_rows_kernel<<<dim3((p.max_rows_per_seq + kThreads / 32 - 1) / (kThreads / 32), B, H), kThreads, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace santapp
