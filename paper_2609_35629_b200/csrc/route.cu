// Routing and sampling for SANTA++ decode attention (Algorithm 1, the steps before the reads):
//   route_score_kernel   representative scores for the query heads of a KV head, routing logit
//                        phi_g = log n_g + q.l_g * scale (Eq. method-routing), Gumbel draw from
//                        the keyed Philox stream, perturbed score Y_g = phi_g + G_g. fp64.
//   select_plan_kernel   per query head: the K largest Y (exact radix selection, ties to the
//                        smaller team id), tau = the (K+1)-st largest, log c_g
//                        (Eq. method-inclusion); the last head of a (sequence, KV head) pair to
//                        finish builds the pair's read plan: the union of the heads' selections
//                        with head masks and per-head corrections (GQA rule), plus the suffix.
//   dense_plan_kernel    the trivial plan that reads every prompt row and the suffix.
#include "common.cuh"

namespace santapp {

namespace {

constexpr int kRouteThreads = 256;
constexpr int kRouteTeamsPerCta = 64;      // 8 warps x 2 quads x 4 teams
constexpr int kSelectThreads = 256;

// ---------------------------------------------------------------------------------------------
// route_score_kernel
// ---------------------------------------------------------------------------------------------

// Sum 32 per-lane values over the warp so that lane L ends up with the total of value L.
__device__ __forceinline__ double reduce_scatter32(double (&v)[32], int lane)
{
#pragma unroll
    for (int half = 16; half >= 1; half >>= 1) {
        const bool upper = (lane & half) != 0;
#pragma unroll
        for (int i = 0; i < half; ++i) {
            const double send = upper ? v[i] : v[i + half];
            const double keep = upper ? v[i + half] : v[i];
            v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, half);
        }
    }
    return v[0];
}

template <int G>
__global__ void __launch_bounds__(kRouteThreads)
route_score_kernel(RouteParams p)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pair = blockIdx.y;
    const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;

    // The first block clears the tickets the later kernels of this call count on.
    if (blockIdx.x == 0 && blockIdx.y == 0) {
        for (int i = tid; i < p.n_pairs; i += kRouteThreads) {
            p.ctl.select_ticket[i] = 0;
            p.ctl.attend_ticket[i] = 0;
        }
        if (tid == 0) {
            *p.ctl.plan_ticket = 0;
            if (p.status) *p.status = 0;
        }
    }

    const int64_t team0 = p.bv.seq_team_off[b];
    const int M = (int)(p.bv.seq_team_off[b + 1] - team0);
    if (p.n_sample >= M) return;                       // every team is read; nothing is drawn
    const int tile0 = blockIdx.x * kRouteTeamsPerCta;
    if (tile0 >= M) return;

    // q for the G heads of this KV head: lane holds elements [4 lane, 4 lane + 4) as fp64
    double qd[G][4];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        const uint2 w = *reinterpret_cast<const uint2 *>(
            p.q + ((size_t)b * p.bv.n_q + (size_t)j * G + h) * kHeadDim + lane * 4);
        qd[h][0] = (double)bf16_lo(w.x); qd[h][1] = (double)bf16_hi(w.x);
        qd[h][2] = (double)bf16_lo(w.y); qd[h][3] = (double)bf16_hi(w.y);
    }

    const uint16_t *rep = p.rep_keys + ((size_t)j * p.bv.teams_total + team0) * kHeadDim;
    const int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    const uint32_t step = p.step + (p.step_dev ? *p.step_dev : 0u);

#pragma unroll 1
    for (int it = 0; it < 2; ++it) {
        const int g0 = tile0 + (warp * 2 + it) * 4;
        if (g0 >= M) break;
        uint2 kw[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            kw[t] = make_uint2(0u, 0u);
            if (g0 + t < M)
                kw[t] = __ldg(reinterpret_cast<const uint2 *>(rep + (size_t)(g0 + t) * kHeadDim + lane * 4));
        }
        double v[32];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const double k0 = (double)bf16_lo(kw[t].x), k1 = (double)bf16_hi(kw[t].x);
            const double k2 = (double)bf16_lo(kw[t].y), k3 = (double)bf16_hi(kw[t].y);
#pragma unroll
            for (int h = 0; h < 8; ++h) {
                if (h < G) {
                    double a = k0 * qd[h][0];
                    a = fma(k1, qd[h][1], a);
                    a = fma(k2, qd[h][2], a);
                    a = fma(k3, qd[h][3], a);
                    v[t * 8 + h] = a;
                } else {
                    v[t * 8 + h] = 0.0;
                }
            }
        }
        const double dot = reduce_scatter32(v, lane);
        const int t = lane >> 3, h = lane & 7, g = g0 + t;
        if (h < G && g < M) {
            const int n_g = csr[g + 1] - csr[g];
            const double phi = log((double)n_g) + dot * p.scale;
            const uint32_t head = (uint32_t)(j * G + h);
            const uint4 words = philox4x32_10(
                make_uint4((uint32_t)g >> 2, step, head, p.stream_base + (uint32_t)b), p.seed_lo, p.seed_hi);
            const double y = phi + gumbel_from_word(pick_word(words, g & 3));
            p.y[(size_t)head * p.bv.teams_total + team0 + g] = y;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// select_plan_kernel
// ---------------------------------------------------------------------------------------------

struct SelectShared {
    int hist[256];
    int scan[33];
    unsigned long long prefix;
    int need;
    int is_last;
    int misc[4];
};

// Writes the plan's suffix segment (if any) and the pair totals. One thread.
__device__ void finish_plan(const SelectParams &p, int pair, int b, int nseg, int prompt_rows)
{
    const int cap = p.plan.seg_cap;
    int32_t *seg_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
    int t = 0;
    if (p.suffix_len != nullptr && p.suffix_cap > 0) t = max(0, min(p.suffix_len[b], p.suffix_cap));
    int total = prompt_rows;
    if (t > 0) {
        p.plan.seg_row[(size_t)pair * cap + nseg] = pair * p.suffix_cap;     // pair = b * n_kv + j
        p.plan.seg_mask[(size_t)pair * cap + nseg] = ((1u << p.bv.group) - 1u) | kSrcSuffix;
        for (int h = 0; h < p.bv.group; ++h)
            p.plan.seg_logc[((size_t)pair * cap + nseg) * p.bv.group + h] = 0.f;
        seg_prefix[nseg] = total;
        total += t;
        ++nseg;
    }
    seg_prefix[nseg] = total;
    p.plan.pair_nseg[pair] = nseg;
    p.plan.pair_rows[pair] = total;
    p.plan.pair_union_rows[pair] = prompt_rows;
    if (p.dbg_union_rows) p.dbg_union_rows[pair] = prompt_rows;
}

// The last pair to finish turns pair_rows into the global exclusive prefix. All threads call.
__device__ void publish_pair_prefix(const SelectParams &p, int *flag_smem, int *scan_smem /* [33] */)
{
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *flag_smem = (atomicAdd(p.ctl.plan_ticket, 1) == p.n_pairs - 1);
    __syncthreads();
    if (!*flag_smem) return;
    __threadfence();
    if (threadIdx.x == 0) *p.ctl.plan_ticket = 0;                  // every pair has arrived
    int64_t carry = 0;
    for (int base = 0; base < p.n_pairs; base += (int)blockDim.x) {
        const int i = base + (int)threadIdx.x;
        const int v = i < p.n_pairs ? __ldcg(p.plan.pair_rows + i) : 0;
        int total;
        const int excl = block_exclusive_scan(v, scan_smem, total);
        if (i < p.n_pairs) p.plan.pair_row_prefix[i] = carry + excl;
        carry += total;
    }
    if (threadIdx.x == 0) p.plan.pair_row_prefix[p.n_pairs] = carry;
}

template <int G>
__global__ void __launch_bounds__(kSelectThreads)
select_plan_kernel(SelectParams p)
{
    extern __shared__ __align__(16) unsigned long long keys[];     // [M] sortable keys; reused by the plan
    __shared__ SelectShared sh;
    __shared__ unsigned long long cand_key[kSelectThreads];
    __shared__ int cand_id[kSelectThreads];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
        for (int g = tid; g < M; g += kSelectThreads) keys[g] = sortable_key(__ldcg(y + g));
        if (tid == 0) { sh.prefix = 0ull; sh.need = Ke + 1; }
        __syncthreads();

        // radix selection of the (Ke+1)-st largest key, 8 bits per pass from the top
        for (int pass = 7; pass >= 0; --pass) {
            const int shift = pass * 8;
            sh.hist[tid] = 0;                                      // kSelectThreads == 256 bins
            __syncthreads();
            const unsigned long long prefix = sh.prefix;
            const int need = sh.need;
            for (int g = tid; g < M; g += kSelectThreads) {
                const unsigned long long k = keys[g];
                const bool match = (pass == 7) || ((k >> (shift + 8)) == (prefix >> (shift + 8)));
                if (match) atomicAdd(&sh.hist[(int)((k >> shift) & 255ull)], 1);
            }
            __syncthreads();
            if (warp == 0) {
                // lane l owns bins 255 - 8 l ... 248 - 8 l (descending)
                int local[8], sum = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) { local[i] = sh.hist[255 - (lane * 8 + i)]; sum += local[i]; }
                int incl = sum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += t;
                }
                const int before = incl - sum;                     // keys in higher bins than this lane's
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
        const unsigned long long thr = sh.prefix;                  // key of the (Ke+1)-st largest
        // keys above the threshold are selected; among keys equal to it (more than one only on
        // an exact tie) the first sh.need - 1 in team order are, too
        const int eq_take = sh.need - 1;
        const int per = (M + kSelectThreads - 1) / kSelectThreads;
        const int lo = min(tid * per, M), hi = min(lo + per, M);
        int n_eq = 0;
        for (int g = lo; g < hi; ++g) n_eq += keys[g] == thr;
        int total_eq, total_gt;
        const int off_eq = block_exclusive_scan(n_eq, sh.scan, total_eq);
        int n_take = 0;
        {
            int eq_seen = off_eq;
            for (int g = lo; g < hi; ++g) {
                const unsigned long long k = keys[g];
                if (k > thr) ++n_take;
                else if (k == thr) { if (eq_seen < eq_take) ++n_take; ++eq_seen; }
            }
        }
        int off = block_exclusive_scan(n_take, sh.scan, total_gt);
        {
            int eq_seen = off_eq;
            for (int g = lo; g < hi; ++g) {
                const unsigned long long k = keys[g];
                bool take = k > thr;
                if (k == thr) { take = eq_seen < eq_take; ++eq_seen; }
                if (take) { cand_key[off] = k; cand_id[off] = g; ++off; }
            }
        }
        __syncthreads();
        // order the Ke selected teams by descending score (ties: smaller id first), compute log c_g
        const double tau = key_to_double(thr);
        if (tid < Ke) {
            const unsigned long long k = cand_key[tid];
            const int id = cand_id[tid];
            int rank = 0;
            for (int a = 0; a < Ke; ++a) {
                const unsigned long long ka = cand_key[a];
                rank += (ka > k) || (ka == k && cand_id[a] < id);
            }
            // phi = Y - G with the same draw the scorer used
            const uint32_t step = p.step + (p.step_dev ? *p.step_dev : 0u);
            const uint4 words = philox4x32_10(
                make_uint4((uint32_t)id >> 2, step, (uint32_t)head, p.stream_base + (uint32_t)b),
                p.seed_lo, p.seed_hi);
            const double phi = key_to_double(k) - gumbel_from_word(pick_word(words, id & 3));
            const double x = phi - tau;
            const double c = -expm1(-exp(x));                      // 1 - exp(-exp(phi - tau))
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
        for (int a = Ke + tid; a < K; a += kSelectThreads) {      // not reached: Ke == K here
            p.sel_team[sel_base + a] = -1;
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
    float *seg_logc = p.plan.seg_logc + (size_t)pair * cap * G;
    const int64_t row0 = p.bv.seq_row_off[b];
    const int N = (int)(p.bv.seq_row_off[b + 1] - row0);
    const float kLog2e = 1.4426950408889634f;

    if (Ke == M) {
        if (tid == 0) {
            seg_row[0] = (int32_t)row0;
            seg_mask[0] = (1u << G) - 1u;
            for (int h = 0; h < G; ++h) seg_logc[h] = 0.f;
            seg_prefix[0] = 0;
            finish_plan(p, pair, b, 1, N);
        }
        publish_pair_prefix(p, &sh.is_last, sh.scan);
        return;
    }

    // head masks per team: one byte per team, four teams per 32-bit word
    uint32_t *tmask = reinterpret_cast<uint32_t *>(keys);                    // [(M + 3) / 4]
    int32_t *seg_of = reinterpret_cast<int32_t *>(keys) + ((M + 3) / 4);     // [M]
    for (int i = tid; i < (M + 3) / 4; i += kSelectThreads) tmask[i] = 0u;
    __syncthreads();
    const size_t pair_sel = ((size_t)b * p.bv.n_q + (size_t)j * G) * K;
    for (int e = tid; e < G * Ke; e += kSelectThreads) {
        const int h = e / Ke, a = e - h * Ke;
        const int g = __ldcg(p.sel_team + pair_sel + (size_t)h * K + a);
        atomicOr(&tmask[g >> 2], 1u << ((g & 3) * 8 + h));
    }
    __syncthreads();
    const int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    {
        const int per = (M + kSelectThreads - 1) / kSelectThreads;
        const int lo = min(tid * per, M), hi = min(lo + per, M);
        int n = 0;
        for (int g = lo; g < hi; ++g) n += ((tmask[g >> 2] >> ((g & 3) * 8)) & 0xFFu) != 0u;
        int nseg;
        int off = block_exclusive_scan(n, sh.scan, nseg);
        for (int g = lo; g < hi; ++g) {
            const uint32_t m = (tmask[g >> 2] >> ((g & 3) * 8)) & 0xFFu;
            if (m) {
                const int r0 = csr[g];
                seg_row[off] = (int32_t)(row0 + r0);
                seg_mask[off] = m;
                seg_prefix[off + 1] = csr[g + 1] - r0;             // sizes now, prefix below
                seg_of[g] = off;
                ++off;
            }
        }
        if (tid == 0) sh.misc[0] = nseg;
    }
    __syncthreads();
    const int nseg = sh.misc[0];
    for (int e = tid; e < nseg * G; e += kSelectThreads) seg_logc[e] = 0.f;
    __syncthreads();
    for (int e = tid; e < G * Ke; e += kSelectThreads) {
        const int h = e / Ke, a = e - h * Ke;
        const int g = __ldcg(p.sel_team + pair_sel + (size_t)h * K + a);
        seg_logc[(size_t)seg_of[g] * G + h] = kLog2e * __ldcg(p.sel_logc + pair_sel + (size_t)h * K + a);
    }
    // sizes -> exclusive prefix (chunked block scan with carry)
    {
        int carry = 0;
        for (int base = 0; base < nseg; base += kSelectThreads) {
            const int s = base + tid;
            const int v = s < nseg ? seg_prefix[s + 1] : 0;
            int total;
            const int excl = block_exclusive_scan(v, sh.scan, total);
            __syncthreads();
            if (s < nseg) seg_prefix[s + 1] = carry + excl + v;
            carry += total;
        }
        if (tid == 0) { seg_prefix[0] = 0; sh.misc[1] = carry; }
    }
    __syncthreads();
    if (tid == 0) finish_plan(p, pair, b, nseg, sh.misc[1]);
    publish_pair_prefix(p, &sh.is_last, sh.scan);
}

// ---------------------------------------------------------------------------------------------
// dense_plan_kernel: one thread per pair
// ---------------------------------------------------------------------------------------------
__global__ void dense_plan_kernel(SelectParams p)
{
    __shared__ int flag;
    __shared__ int scan[33];
    // single block; tickets are cleared here for the attend kernel
    for (int pair = threadIdx.x; pair < p.n_pairs; pair += blockDim.x) {
        const int b = pair / p.bv.n_kv;
        p.ctl.attend_ticket[pair] = 0;
        const int cap = p.plan.seg_cap;
        const int64_t row0 = p.bv.seq_row_off[b];
        const int N = (int)(p.bv.seq_row_off[b + 1] - row0);
        p.plan.seg_row[(size_t)pair * cap] = (int32_t)row0;
        p.plan.seg_mask[(size_t)pair * cap] = (1u << p.bv.group) - 1u;
        for (int h = 0; h < p.bv.group; ++h) p.plan.seg_logc[(size_t)pair * cap * p.bv.group + h] = 0.f;
        p.plan.seg_prefix[(size_t)pair * (cap + 1)] = 0;
        finish_plan(p, pair, b, 1, N);
    }
    if (threadIdx.x == 0) *p.ctl.plan_ticket = p.n_pairs - 1;    // this block is the last arrival
    __syncthreads();
    publish_pair_prefix(p, &flag, scan);
}

template <int G>
cudaError_t launch_route_score_g(const RouteParams &p, int max_teams, cudaStream_t s)
{
    dim3 grid((max_teams + kRouteTeamsPerCta - 1) / kRouteTeamsPerCta, p.n_pairs);
    route_score_kernel<G><<<grid, kRouteThreads, 0, s>>>(p);
    return cudaGetLastError();
}

template <int G>
cudaError_t launch_select_plan_g(const SelectParams &p, int max_teams, cudaStream_t s)
{
    const size_t smem = sizeof(unsigned long long) * (size_t)max_teams + 64;
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

#define SANTAPP_DISPATCH_G(G, CALL)                         \
    switch (G) {                                            \
        case 1: return CALL<1>;                             \
        case 2: return CALL<2>;                             \
        case 3: return CALL<3>;                             \
        case 4: return CALL<4>;                             \
        case 5: return CALL<5>;                             \
        case 6: return CALL<6>;                             \
        case 7: return CALL<7>;                             \
        case 8: return CALL<8>;                             \
        default: return nullptr;                            \
    }

cudaError_t launch_route_score(const RouteParams &p, int max_teams_per_seq, cudaStream_t s)
{
    auto pick = [](int g) -> cudaError_t (*)(const RouteParams &, int, cudaStream_t) {
        SANTAPP_DISPATCH_G(g, launch_route_score_g)
    };
    auto fn = pick(p.bv.group);
    return fn ? fn(p, max_teams_per_seq, s) : cudaErrorInvalidValue;
}

cudaError_t launch_select_plan(const SelectParams &p, int max_teams_per_seq, cudaStream_t s)
{
    auto pick = [](int g) -> cudaError_t (*)(const SelectParams &, int, cudaStream_t) {
        SANTAPP_DISPATCH_G(g, launch_select_plan_g)
    };
    auto fn = pick(p.bv.group);
    return fn ? fn(p, max_teams_per_seq, s) : cudaErrorInvalidValue;
}

cudaError_t launch_dense_plan(const SelectParams &p, cudaStream_t s)
{
    dense_plan_kernel<<<1, 256, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace santapp
