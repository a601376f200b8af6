// Sampling for SANTA++ decode attention (Algorithm 1, the Gumbel-top-K step and the correction):
//   select_plan_kernel   per query head: the K largest perturbed scores Y (ties to the smaller
//                        team id), tau = the (K+1)-st largest, log c_g (Eq. method-inclusion).
//                        The last head of a (sequence, KV head) pair to finish builds the pair's
//                        read plan: the union of the heads' selections in team order with head
//                        masks and per-head corrections (GQA rule), plus the exact suffix.
//
// Selection is exact. The scores are fp64; a histogram over the top of the value range finds a
// bucket boundary below which nothing can be among the K+1 largest, the few candidates above it
// are ranked exactly by (score, team id), and a radix selection over the raw bit patterns takes
// over when the histogram cannot separate the scores (heavy ties, extreme outliers).
#include "common.cuh"
#include "plan.cuh"

namespace santapp {

namespace {

constexpr int kSelectThreads = 256;
constexpr int kBins = 4096;
constexpr int kBinsPerThread = kBins / kSelectThreads;
constexpr int kCandMax = 1024;             // candidates ranked exactly; also G * K entries of a plan
constexpr int kLevels = 3;
constexpr double kBinSpan = 64.0;          // score range covered by one histogram level

struct SelectShared {
    union {
        struct {
            unsigned long long cand_key[kCandMax];
            int cand_id[kCandMax];
            int cand_rank[kCandMax];
            int hist[kBins];
        } s;
        struct {
            int ent_key[kCandMax];         // team * 8 + head
            float ent_logc[kCandMax];
            int srt_key[kCandMax];
            float srt_logc[kCandMax];
            int seg_rows[kCandMax];
        } p;
    };
    int scan[33];
    double red[2 * (kSelectThreads / 32)];
    double lvl_lo[kLevels], lvl_inv[kLevels];
    double tau;
    unsigned long long prefix;
    int need;
    int is_last;
    int n_cand;
    int misc[4];
};

__device__ __forceinline__ int bin_of(double y, double lo, double inv)
{
    if (!(y >= lo)) return 0;
    const double t = (y - lo) * inv;
    return t >= (double)(kBins - 1) ? kBins - 1 : (int)t;
}

// Block-wide minimum and maximum of one double per thread (all threads get both).
__device__ void block_min_max(double &mn, double &mx, double *red)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mn = fmin(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, o));
        mx = fmax(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    }
    __syncthreads();
    if (lane == 0) { red[2 * warp] = mn; red[2 * warp + 1] = mx; }
    __syncthreads();
    mn = red[0];
    mx = red[1];
#pragma unroll
    for (int w = 1; w < kSelectThreads / 32; ++w) { mn = fmin(mn, red[2 * w]); mx = fmax(mx, red[2 * w + 1]); }
}

// Histogram selection. On success the candidates (every score that can be among the `need`
// largest, at least `need` of them) are in sh.s.cand_key / cand_id, sh.n_cand holds their count
// and the function returns true. All threads call.
__device__ bool select_by_histogram(const double *ys, int M, int need_total, SelectShared &sh)
{
    const int tid = threadIdx.x;
    int need = need_total;
    int taken = 0;                 // scores already known to be above the current range
    int final_level = -1, b_star = 0;
    for (int lvl = 0; lvl < kLevels; ++lvl) {
        // scores still undecided: bin 0 at every earlier level
        double mn = INFINITY, mx = -INFINITY;
        for (int g = tid; g < M; g += kSelectThreads) {
            const double y = ys[g];
            bool rem = true;
            for (int l = 0; l < lvl; ++l) rem = rem && bin_of(y, sh.lvl_lo[l], sh.lvl_inv[l]) == 0;
            if (rem) { mn = fmin(mn, y); mx = fmax(mx, y); }
        }
        block_min_max(mn, mx, sh.red);
        if (!(mx > mn)) return false;                               // all equal (or none): ties decide
        const double lo = fmax(mn, mx - kBinSpan);
        const double inv = (double)kBins / (mx - lo);
        for (int i = tid; i < kBins; i += kSelectThreads) sh.s.hist[i] = 0;
        if (tid == 0) { sh.lvl_lo[lvl] = lo; sh.lvl_inv[lvl] = inv; }
        __syncthreads();
        for (int g = tid; g < M; g += kSelectThreads) {
            const double y = ys[g];
            bool rem = true;
            for (int l = 0; l < lvl; ++l) rem = rem && bin_of(y, sh.lvl_lo[l], sh.lvl_inv[l]) == 0;
            if (rem) atomicAdd(&sh.s.hist[bin_of(y, lo, inv)], 1);
        }
        __syncthreads();
        // thread t owns bins kBins-1-16t ... kBins-16-16t (descending); find where the count
        // from the top reaches `need`
        int local[kBinsPerThread], sum = 0;
#pragma unroll
        for (int i = 0; i < kBinsPerThread; ++i) {
            local[i] = sh.s.hist[kBins - 1 - (tid * kBinsPerThread + i)];
            sum += local[i];
        }
        int total;
        const int before = block_exclusive_scan(sum, sh.scan, total);
        if (before < need && before + sum >= need) {
            int acc = before;
#pragma unroll
            for (int i = 0; i < kBinsPerThread; ++i) {
                if (acc < need && acc + local[i] >= need) {
                    sh.misc[0] = kBins - 1 - (tid * kBinsPerThread + i);    // boundary bin
                    sh.misc[1] = acc;                                       // scores in bins above it
                    sh.misc[2] = local[i];
                }
                acc += local[i];
            }
        }
        __syncthreads();
        const int bb = sh.misc[0], above = sh.misc[1], pop = sh.misc[2];
        __syncthreads();
        if (bb > 0 || lo <= mn) {
            if (taken + above + pop > kCandMax) return false;
            final_level = lvl;
            b_star = bb;
            break;
        }
        // the boundary lies below this level's range: every score in bins >= 1 is selected
        const int up = total - sh.s.hist[0];
        taken += up;
        need -= up;
        if (taken > kCandMax) return false;
    }
    if (final_level < 0) return false;
    if (tid == 0) sh.n_cand = 0;
    __syncthreads();
    for (int g = tid; g < M; g += kSelectThreads) {
        const double y = ys[g];
        bool cand = false, rem = true;
        for (int l = 0; l < final_level; ++l) {
            if (rem && bin_of(y, sh.lvl_lo[l], sh.lvl_inv[l]) != 0) { cand = true; rem = false; }
        }
        if (rem && bin_of(y, sh.lvl_lo[final_level], sh.lvl_inv[final_level]) >= b_star) cand = true;
        if (cand) {
            const int slot = atomicAdd(&sh.n_cand, 1);
            sh.s.cand_key[slot] = sortable_key(y);
            sh.s.cand_id[slot] = g;
        }
    }
    __syncthreads();
    return true;
}

// Radix selection over the bit patterns: exactly the Ke largest (ties to the smaller id) go to
// the candidate arrays, sh.tau gets the (Ke+1)-st largest. All threads call.
__device__ void select_by_radix(const double *ys, int M, int Ke, SelectShared &sh)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) { sh.prefix = 0ull; sh.need = Ke + 1; }
    __syncthreads();
    for (int pass = 7; pass >= 0; --pass) {
        const int shift = pass * 8;
        sh.s.hist[tid] = 0;                                        // kSelectThreads == 256 bins
        __syncthreads();
        const unsigned long long prefix = sh.prefix;
        const int need = sh.need;
        for (int g = tid; g < M; g += kSelectThreads) {
            const unsigned long long k = sortable_key(ys[g]);
            const bool match = (pass == 7) || ((k >> (shift + 8)) == (prefix >> (shift + 8)));
            if (match) atomicAdd(&sh.s.hist[(int)((k >> shift) & 255ull)], 1);
        }
        __syncthreads();
        if (warp == 0) {
            int local[8], sum = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { local[i] = sh.s.hist[255 - (lane * 8 + i)]; sum += local[i]; }
            int incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += t;
            }
            const int before = incl - sum;
            if (before < need && incl >= need) {
                int acc = before;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (acc < need && acc + local[i] >= need) {
                        sh.prefix = prefix | ((unsigned long long)(255 - (lane * 8 + i)) << shift);
                        sh.need = need - acc;
                    }
                    acc += local[i];
                }
            }
        }
        __syncthreads();
    }
    const unsigned long long thr = sh.prefix;                      // key of the (Ke+1)-st largest
    const int eq_take = sh.need - 1;                               // equal keys that still belong to the top Ke
    const int per = (M + kSelectThreads - 1) / kSelectThreads;
    const int lo = min(tid * per, M), hi = min(lo + per, M);
    int n_eq = 0;
    for (int g = lo; g < hi; ++g) n_eq += sortable_key(ys[g]) == thr;
    int total_eq, total_take;
    const int off_eq = block_exclusive_scan(n_eq, sh.scan, total_eq);
    int n_take = 0;
    {
        int eq_seen = off_eq;
        for (int g = lo; g < hi; ++g) {
            const unsigned long long k = sortable_key(ys[g]);
            if (k > thr) ++n_take;
            else if (k == thr) { if (eq_seen < eq_take) ++n_take; ++eq_seen; }
        }
    }
    int off = block_exclusive_scan(n_take, sh.scan, total_take);
    {
        int eq_seen = off_eq;
        for (int g = lo; g < hi; ++g) {
            const unsigned long long k = sortable_key(ys[g]);
            bool take = k > thr;
            if (k == thr) { take = eq_seen < eq_take; ++eq_seen; }
            if (take) { sh.s.cand_key[off] = k; sh.s.cand_id[off] = g; ++off; }
        }
    }
    if (tid == 0) { sh.n_cand = Ke; sh.tau = key_to_double(thr); }
    __syncthreads();
}

template <int G>
__global__ void __launch_bounds__(kSelectThreads)
select_plan_kernel(SelectParams p)
{
    extern __shared__ __align__(16) double ys[];                   // [M] perturbed scores
    __shared__ SelectShared sh;

    const int tid = threadIdx.x;
    const int hg = blockIdx.x, pair = blockIdx.y;
    const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;
    const int head = j * G + hg;
    const int64_t team0 = p.bv.seq_team_off[b];
    const int M = (int)(p.bv.seq_team_off[b + 1] - team0);
    const int K = p.n_sample;
    const int Ke = min(K, M);
    const size_t sel_base = ((size_t)b * p.bv.n_q + head) * K;

    if (Ke == M) {
        // every team selected with correction one
        for (int a = tid; a < K; a += kSelectThreads) {
            const int id = a < M ? a : -1;
            p.sel_team[sel_base + a] = id;
            p.sel_logc[sel_base + a] = 0.f;
            if (p.dbg_sel_idx) p.dbg_sel_idx[sel_base + a] = id;
            if (p.dbg_sel_logc) p.dbg_sel_logc[sel_base + a] = 0.f;
        }
        if (tid == 0) {
            const double nan = __longlong_as_double(0x7FF8000000000000ll);
            p.tau[(size_t)b * p.bv.n_q + head] = nan;
            if (p.dbg_tau) p.dbg_tau[(size_t)b * p.bv.n_q + head] = nan;
        }
    } else {
        const double *y = p.y + (size_t)head * p.bv.teams_total + team0;
        for (int g = tid; g < M; g += kSelectThreads) ys[g] = __ldcg(y + g);
        __syncthreads();
        const bool by_hist = select_by_histogram(ys, M, Ke + 1, sh);
        if (!by_hist) select_by_radix(ys, M, Ke, sh);
        // exact ranks among the candidates: descending score, ties to the smaller team id
        const int n_cand = sh.n_cand;
        for (int t = tid; t < n_cand; t += kSelectThreads) {
            const unsigned long long k = sh.s.cand_key[t];
            const int id = sh.s.cand_id[t];
            int rank = 0;
            for (int a = 0; a < n_cand; ++a) {
                const unsigned long long ka = sh.s.cand_key[a];
                rank += (ka > k) || (ka == k && sh.s.cand_id[a] < id);
            }
            sh.s.cand_rank[t] = rank;
            if (by_hist && rank == Ke) sh.tau = key_to_double(k);  // the (K+1)-st largest
        }
        __syncthreads();
        const double tau = sh.tau;
        const uint32_t step = p.step + (p.step_dev ? *p.step_dev : 0u);
        for (int t = tid; t < n_cand; t += kSelectThreads) {
            const int rank = sh.s.cand_rank[t];
            if (rank >= Ke) continue;
            const int id = sh.s.cand_id[t];
            // phi = Y - G with the same draw the scorer used
            const uint4 words = philox4x32_10(
                make_uint4((uint32_t)id >> 2, step, (uint32_t)head, p.stream_base + (uint32_t)b),
                p.seed_lo, p.seed_hi);
            const double phi = key_to_double(sh.s.cand_key[t]) - gumbel_from_word(pick_word(words, id & 3));
            const double c = -expm1(-exp(phi - tau));              // 1 - exp(-exp(phi - tau))
            const float logc = (float)log(c);
            p.sel_team[sel_base + rank] = id;
            p.sel_logc[sel_base + rank] = logc;
            if (p.dbg_sel_idx) p.dbg_sel_idx[sel_base + rank] = id;
            if (p.dbg_sel_logc) p.dbg_sel_logc[sel_base + rank] = logc;
        }
        if (tid == 0) {
            p.tau[(size_t)b * p.bv.n_q + head] = tau;
            if (p.dbg_tau) p.dbg_tau[(size_t)b * p.bv.n_q + head] = tau;
        }
    }

    // ---- the last head of the pair builds the read plan ----
    __threadfence();
    __syncthreads();
    if (tid == 0) sh.is_last = (atomicAdd(p.ctl.select_ticket + pair, 1) == G - 1);
    __syncthreads();
    if (!sh.is_last) return;
    __threadfence();
    if (tid == 0) p.ctl.select_ticket[pair] = 0;                   // all G heads of the pair have arrived

    const int cap = p.plan.seg_cap;
    int32_t *seg_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
    int32_t *seg_row = p.plan.seg_row + (size_t)pair * cap;
    uint32_t *seg_mask = p.plan.seg_mask + (size_t)pair * cap;
    float *seg_logc = p.plan.seg_logc + (size_t)pair * cap * kMaxGroup;
    const int64_t row0 = p.bv.seq_row_off[b];
    const int N = (int)(p.bv.seq_row_off[b + 1] - row0);
    const float kLog2e = 1.4426950408889634f;

    if (Ke == M) {
        if (tid == 0) {
            seg_row[0] = (int32_t)row0;
            seg_mask[0] = (1u << G) - 1u;
            for (int h = 0; h < kMaxGroup; ++h) seg_logc[h] = 0.f;
            seg_prefix[0] = 0;
            finish_plan(p, pair, b, 1, N);
        }
        publish_pair_prefix(p, &sh.is_last, sh.scan);
        return;
    }

    // the G * Ke (team, head, log c) entries, sorted by team: equal teams become one segment
    const int E = G * Ke;
    const size_t pair_sel = ((size_t)b * p.bv.n_q + (size_t)j * G) * K;
    for (int e = tid; e < E; e += kSelectThreads) {
        const int h = e / Ke, a = e - h * Ke;
        sh.p.ent_key[e] = __ldcg(p.sel_team + pair_sel + (size_t)h * K + a) * kMaxGroup + h;
        sh.p.ent_logc[e] = __ldcg(p.sel_logc + pair_sel + (size_t)h * K + a);
    }
    __syncthreads();
    for (int e = tid; e < E; e += kSelectThreads) {
        const int k = sh.p.ent_key[e];
        int rank = 0;
        for (int a = 0; a < E; ++a) rank += sh.p.ent_key[a] < k;   // keys are distinct
        sh.p.srt_key[rank] = k;
        sh.p.srt_logc[rank] = sh.p.ent_logc[e];
    }
    __syncthreads();
    // each thread owns a contiguous run of sorted entries; an entry opens a segment when its
    // team differs from the previous entry's
    const int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    const int per = (E + kSelectThreads - 1) / kSelectThreads;
    const int lo = min(tid * per, E), hi = min(lo + per, E);
    int n_open = 0;
    for (int e = lo; e < hi; ++e)
        n_open += (e == 0) || ((sh.p.srt_key[e] >> 3) != (sh.p.srt_key[e - 1] >> 3));
    int nseg;
    int seg = block_exclusive_scan(n_open, sh.scan, nseg);
    for (int e = lo; e < hi; ++e) {
        const int team = sh.p.srt_key[e] >> 3;
        if (e != 0 && team == (sh.p.srt_key[e - 1] >> 3)) continue;
        uint32_t mask = 0u;
        float lc[kMaxGroup];
#pragma unroll
        for (int h = 0; h < kMaxGroup; ++h) lc[h] = 0.f;
        for (int a = e; a < E && (sh.p.srt_key[a] >> 3) == team; ++a) {
            const int h = sh.p.srt_key[a] & 7;
            mask |= 1u << h;
#pragma unroll
            for (int hh = 0; hh < kMaxGroup; ++hh)
                if (hh == h) lc[hh] = kLog2e * sh.p.srt_logc[a];
        }
        const int r_lo = csr[team];
        seg_row[seg] = (int32_t)(row0 + r_lo);
        seg_mask[seg] = mask;
        float4 *dst = reinterpret_cast<float4 *>(seg_logc + (size_t)seg * kMaxGroup);
        dst[0] = make_float4(lc[0], lc[1], lc[2], lc[3]);
        dst[1] = make_float4(lc[4], lc[5], lc[6], lc[7]);
        sh.p.seg_rows[seg] = csr[team + 1] - r_lo;
        ++seg;
    }
    __syncthreads();
    // segment sizes -> exclusive prefix
    {
        const int per_s = (nseg + kSelectThreads - 1) / kSelectThreads;
        const int s_lo = min(tid * per_s, nseg), s_hi = min(s_lo + per_s, nseg);
        int sum = 0;
        for (int s = s_lo; s < s_hi; ++s) sum += sh.p.seg_rows[s];
        int total;
        int run = block_exclusive_scan(sum, sh.scan, total);
        for (int s = s_lo; s < s_hi; ++s) { seg_prefix[s] = run; run += sh.p.seg_rows[s]; }
        if (tid == 0) sh.misc[1] = total;
    }
    __syncthreads();
    if (tid == 0) finish_plan(p, pair, b, nseg, sh.misc[1]);
    publish_pair_prefix(p, &sh.is_last, sh.scan);
}

template <int G>
cudaError_t launch_select_plan_g(const SelectParams &p, int max_teams, cudaStream_t s)
{
    const size_t smem = sizeof(double) * (size_t)max_teams + 64;
    static thread_local size_t smem_set = 0;             // raise the limit once per thread and size
    if (smem > smem_set) {
        cudaError_t err = cudaFuncSetAttribute(select_plan_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               (int)smem);
        if (err != cudaSuccess) return err;
        smem_set = smem;
    }
    select_plan_kernel<G><<<dim3(G, p.n_pairs), kSelectThreads, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_select_plan(const SelectParams &p, int max_teams_per_seq, cudaStream_t s)
{
    if (p.n_sample < max_teams_per_seq && p.bv.group * p.n_sample > kCandMax) return cudaErrorInvalidValue;
    switch (p.bv.group) {
        case 1: return launch_select_plan_g<1>(p, max_teams_per_seq, s);
        case 2: return launch_select_plan_g<2>(p, max_teams_per_seq, s);
        case 3: return launch_select_plan_g<3>(p, max_teams_per_seq, s);
        case 4: return launch_select_plan_g<4>(p, max_teams_per_seq, s);
        case 5: return launch_select_plan_g<5>(p, max_teams_per_seq, s);
        case 6: return launch_select_plan_g<6>(p, max_teams_per_seq, s);
        case 7: return launch_select_plan_g<7>(p, max_teams_per_seq, s);
        case 8: return launch_select_plan_g<8>(p, max_teams_per_seq, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace santapp
