// Read plan of one (sequence, KV head) pair, as a block-wide device function: the GQA union of the
// heads' samples (Algorithm 1; the samples and their corrections come from headplan.cuh) in team
// order with head masks, per-head log2(e) * log c_g, segment row prefix, and the exact suffix as a
// last segment.
#pragma once

#include <math_constants.h>

#include "common.cuh"

namespace santapp {

constexpr int kEntCap = 1024;           // G * K entries of a plan
constexpr int kSegMax = 1025;           // segments of a plan (entries + suffix)
constexpr int kBitmapWords = kMaxTeamsPerSeq / 32;

struct alignas(16) PlanScratch {
    uint32_t bitmap[kBitmapWords];
    int wprefix[kBitmapWords];
    int seg_rows[kSegMax + 3];
    int scan[40];
    int misc[8];
};

// Block: plan of `pair` into shared-memory tables (seg_prefix[nseg+1], seg_row, seg_mask) and the
// pair's log c table in global memory (g_logc [kSegMax][8]). All threads call; blockDim.x ==
// kPlanThreads (a multiple of 32). Returns the number of segments in nseg_out and of rows in
// rows_out. write_debug: also fill the caller's diagnostics (one block per pair should).
// max_words: bitmap words that cover the longest sequence's teams (a host scalar, so that the
// tables can be cleared while the first loads are still in flight).
template <int kPlanThreads>
__device__ __forceinline__ void build_pair_plan(const PlanInputs &in, int pair, int max_words, PlanScratch &sc, int *seg_prefix,
                                                int *seg_row, uint32_t *seg_mask, float *g_logc, int &nseg_out, int &rows_out,
                                                bool write_debug)
{
    constexpr int kEntPerThread = (kEntCap + kPlanThreads - 1) / kPlanThreads;   // entries a thread keeps in registers
    const int G = in.bv.group;
    const int tid = threadIdx.x;
    const int b = pair / in.bv.n_kv, j = pair - b * in.bv.n_kv;
    const int K = in.n_sample;
    const int E = G * K;
    const size_t head0 = (size_t)b * in.bv.n_q + (size_t)j * G;       // first query head of the pair
    // The heads' samples, requested before anything else so that they travel together with the
    // sequence offsets: each thread keeps its entries in registers. (When every team is read,
    // K >= M, nothing was sampled and the values are not used.)
    int ent_team[kEntPerThread];
    float ent_logc[kEntPerThread];
    int2 ent_rows[kEntPerThread];
#pragma unroll
    for (int u = 0; u < kEntPerThread; ++u) {
        const int e = tid + u * kPlanThreads;
        ent_team[u] = 0;
        ent_logc[u] = 0.f;
        ent_rows[u] = make_int2(0, 0);
        if (e < E) {                                                  // entry e: head e / K, rank e % K
            const size_t at = head0 * K + e;
            ent_team[u] = __ldcg(in.sel_team + at);
            ent_logc[u] = __ldcg(in.sel_logc + at);
            ent_rows[u] = __ldcg(in.sel_rows + at);
        }
    }
    const int M = pair_team_count(in.bv, b, j);
    const int64_t row0 = in.bv.seq_row_off[b];
    const int N = (int)(in.bv.seq_row_off[b + 1] - row0);
    int t_suffix = 0;
    if (in.suffix_len != nullptr && in.suffix_cap > 0) t_suffix = max(0, min(in.suffix_len[b], in.suffix_cap));
    const uint32_t all_heads = (1u << G) - 1u;
    const float kLog2e = 1.4426950408889634f;

    // clear the tables while those loads are in flight
    for (int i = tid; i < max_words; i += kPlanThreads) sc.bitmap[i] = 0u;
    for (int i = tid; i <= min(E, kSegMax - 1); i += kPlanThreads) seg_mask[i] = 0u;
    __syncthreads();
    trace_mark(in.trace, 2, 2);

    const int Ke = min(K, M);
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
        for (int e = tid; write_debug && e < G * K; e += kPlanThreads) {
            const int h = e / K, a = e - h * K;
            if (in.dbg_sel_idx) in.dbg_sel_idx[(head0 + h) * K + a] = a < M ? a : -1;
            if (in.dbg_sel_logc) in.dbg_sel_logc[(head0 + h) * K + a] = 0.f;
        }
        if (write_debug && tid < G && in.dbg_tau) in.dbg_tau[head0 + tid] = __longlong_as_double(0x7FF8000000000000ll);
        __syncthreads();
        nseg_out = sc.misc[0];
        rows_out = sc.misc[1];
        return;
    }

    // ---- here K < M, so every head has exactly K sampled teams ----
    const int n_words = (M + 31) / 32;
    int ent_key[kEntPerThread];                                       // team * 8 + head, -1: none
#pragma unroll
    for (int u = 0; u < kEntPerThread; ++u) {
        const int e = tid + u * kPlanThreads;
        // a team id outside the pair's range cannot come from the sampler; refusing it here keeps
        // the tables in bounds whatever the workspace holds
        const bool ok = e < E && ent_team[u] >= 0 && ent_team[u] < M;
        ent_key[u] = ok ? ent_team[u] * kMaxGroup + e / K : -1;
        if (ok) atomicOr(&sc.bitmap[ent_team[u] >> 5], 1u << (ent_team[u] & 31));
    }
    __syncthreads();
    // Segment index of a team = selected teams before it: prefix over the bitmap's words.
    int ent_seg[kEntPerThread];
    int nseg_prompt;
    if (n_words <= 64) {
        // every warp sums the (at most 64) words for itself, two per lane: no table, no barrier
        const int lane = tid & 31;
        const uint32_t w0 = 2 * lane < n_words ? sc.bitmap[2 * lane] : 0u;
        const uint32_t w1 = 2 * lane + 1 < n_words ? sc.bitmap[2 * lane + 1] : 0u;
        const int c0 = __popc(w0), c1 = __popc(w1);
        int incl = c0 + c1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        nseg_prompt = __shfl_sync(0xFFFFFFFFu, incl, 31);
        const int excl = incl - c0 - c1;
#pragma unroll
        for (int u = 0; u < kEntPerThread; ++u) {
            const int team = ent_key[u] >= 0 ? ent_key[u] >> 3 : 0;
            const int word = team >> 5, src = word >> 1;
            // every lane takes part in every exchange; the choice between a lane's two words comes after
            const int s_excl = __shfl_sync(0xFFFFFFFFu, excl, src), s_c0 = __shfl_sync(0xFFFFFFFFu, c0, src);
            const uint32_t s_w0 = __shfl_sync(0xFFFFFFFFu, w0, src), s_w1 = __shfl_sync(0xFFFFFFFFu, w1, src);
            const uint32_t bits = (word & 1) ? s_w1 : s_w0;
            ent_seg[u] = s_excl + ((word & 1) ? s_c0 : 0) + __popc(bits & ((1u << (team & 31)) - 1u));
        }
    } else {
        // thread t owns the contiguous words [t * wpt, (t + 1) * wpt)
        const int wpt = (n_words + kPlanThreads - 1) / kPlanThreads;
        const int lo = min(tid * wpt, n_words), hi = min(lo + wpt, n_words);
        int sum = 0;
        for (int w = lo; w < hi; ++w) sum += __popc(sc.bitmap[w]);
        int total;
        int run = block_exclusive_scan(sum, sc.scan, total);
        for (int w = lo; w < hi; ++w) { sc.wprefix[w] = run; run += __popc(sc.bitmap[w]); }
        __syncthreads();
        nseg_prompt = total;
#pragma unroll
        for (int u = 0; u < kEntPerThread; ++u) {
            const int team = ent_key[u] >= 0 ? ent_key[u] >> 3 : 0;
            ent_seg[u] = sc.wprefix[team >> 5] + __popc(sc.bitmap[team >> 5] & ((1u << (team & 31)) - 1u));
        }
    }
#pragma unroll
    for (int u = 0; u < kEntPerThread; ++u) {
        if (ent_key[u] >= 0) {
            const int h = ent_key[u] & 7, seg = ent_seg[u];
            atomicOr(&seg_mask[seg], 1u << h);
            g_logc[(size_t)seg * kMaxGroup + h] = kLog2e * ent_logc[u];
            seg_row[seg] = (int32_t)(row0 + ent_rows[u].x);           // same value from every selecting head
            sc.seg_rows[seg] = ent_rows[u].y;
        }
    }
    if (t_suffix > 0 && tid < kMaxGroup) g_logc[(size_t)nseg_prompt * kMaxGroup + tid] = 0.f;
    __syncthreads();
    // row prefix of the segments, then the suffix segment
    {
        const int spt = (nseg_prompt + kPlanThreads - 1) / kPlanThreads;
        const int lo = min(tid * spt, nseg_prompt), hi = min(lo + spt, nseg_prompt);
        int sum = 0;
        for (int sg = lo; sg < hi; ++sg) sum += sc.seg_rows[sg];
        int total;
        int run = block_exclusive_scan(sum, sc.scan, total);
        for (int sg = lo; sg < hi; ++sg) { seg_prefix[sg] = run; run += sc.seg_rows[sg]; }
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
    }
    __threadfence_block();                                            // the log c table is read back through asynchronous copies
    __syncthreads();
    nseg_out = sc.misc[0];
    rows_out = sc.misc[1];
}

}  // namespace santapp
