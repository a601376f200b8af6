// Exact attention over a read plan (Algorithm 1, the reads and the estimator):
// every member row of every selected team enters head h's sums with weight e^{s_i} / c_g
// (applied as s_i - log c_g, so the same correction enters the mass and the value sum), every
// suffix row with weight e^{s_i}; Eq. (method-estimate).
//
// The rows of all (sequence, KV head) pairs form one global row space that is cut into equal
// contiguous ranges, one per CTA (split-K by rows, not by teams), one CTA per SM. Inside a CTA
// one producer thread streams the range through a ring of shared-memory stages with bulk
// asynchronous copies (whole runs of team-contiguous rows per copy, K and V), eight consumer
// warps evaluate the rows (half a warp per row) with an online softmax, and the CTA leaves one
// partial per pair it touched. The last CTA to finish a pair merges that pair's partials by
// log-sum-exp (the split-softmax reduction).
//
// Every wait on a barrier is bounded: on expiry the kernel raises a status bit and leaves.
#include <math_constants.h>

#include "common.cuh"

namespace santapp {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = 32 * kConsumerWarps;
constexpr int kAttendThreads = kConsumerThreads + 32;       // + one producer warp
constexpr int kHalfWarps = kConsumerThreads / 16;           // rows evaluated side by side
constexpr int kStageRows = 32;
constexpr int kRowsPerHalfWarp = kStageRows / kHalfWarps;   // 2
constexpr int kStages = 8;
constexpr int kRowBytes = kHeadDim * 2;                     // one bf16 row
constexpr int kStageBytes = kStageRows * kRowBytes * 2;     // K block then V block
constexpr int kSegMax = 1025;                               // plan segments of one pair (G * K + suffix)
constexpr int kPairMax = 1024;                              // pairs whose offsets are staged
constexpr int kMaxAttendGrid = 512;
constexpr uint32_t kSpinLimit = 1u << 22;

// ---- mbarrier / bulk copy primitives (shared::cta addresses as 32-bit) ----
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait. Returns false when the limit ran out or another thread already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier. Both addresses
// and the size are multiples of 16 (rows are 256 bytes).
__device__ __forceinline__ void bulk_copy_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// ---- shared memory carve-up (dynamic) ----
template <int G>
struct Smem {
    static constexpr size_t ring = 0;                                           // kStages * kStageBytes
    static constexpr size_t bars = ring + (size_t)kStages * kStageBytes;        // full[kStages], empty[kStages]
    static constexpr size_t q = bars + 2 * kStages * 8;                          // float [G][128]
    static constexpr size_t seg_prefix = q + (size_t)G * kHeadDim * 4;          // int [kSegMax + 1] (+pad)
    static constexpr size_t seg_row = seg_prefix + (kSegMax + 3) * 4;           // int [kSegMax]
    static constexpr size_t seg_mask = seg_row + (kSegMax + 3) * 4;             // uint [kSegMax]
    static constexpr size_t seg_logc = seg_mask + (kSegMax + 3) * 4;            // float [kSegMax][G]
    static constexpr size_t pair_prefix = (seg_logc + (size_t)kSegMax * G * 4 + 15) / 16 * 16;  // int64 [kPairMax+1]
    static constexpr size_t pair_nseg = pair_prefix + (kPairMax + 1) * 8;       // int [kPairMax]
    static constexpr size_t misc = pair_nseg + kPairMax * 4;                    // flags
    static constexpr size_t total = misc + 64;
    // aliases of the ring, used only after a span's stages are consumed
    static constexpr size_t red_acc = ring;                                     // float [warps][G][128]
    static constexpr size_t red_m = red_acc + (size_t)kConsumerWarps * G * kHeadDim * 4;   // float [warps][G]
    static constexpr size_t red_l = red_m + (size_t)kConsumerWarps * G * 4;
    static constexpr size_t wbuf = red_l + (size_t)kConsumerWarps * G * 4;      // float [G][kMaxAttendGrid]
    static_assert(wbuf + (size_t)G * kMaxAttendGrid * 4 <= bars, "merge scratch must fit in the ring");
};

template <int G, bool kAll>
__global__ void __launch_bounds__(kAttendThreads, 1)
attend_kernel(AttendParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    using S = Smem<G>;
    unsigned char *ring = smem + S::ring;
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + S::bars);
    uint64_t *empty_bar = full_bar + kStages;
    float(*q_s)[kHeadDim] = reinterpret_cast<float(*)[kHeadDim]>(smem + S::q);
    int *seg_prefix = reinterpret_cast<int *>(smem + S::seg_prefix);
    int *seg_row = reinterpret_cast<int *>(smem + S::seg_row);
    uint32_t *seg_mask = reinterpret_cast<uint32_t *>(smem + S::seg_mask);
    float(*seg_logc)[G] = reinterpret_cast<float(*)[G]>(smem + S::seg_logc);
    int64_t *pair_prefix = reinterpret_cast<int64_t *>(smem + S::pair_prefix);
    int *pair_nseg = reinterpret_cast<int *>(smem + S::pair_nseg);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + S::misc);
    int *last_flag = reinterpret_cast<int *>(smem + S::misc) + 1;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hw = tid >> 4, l16 = tid & 15;
    const bool is_producer = warp == kConsumerWarps;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar + s, 1);
            mbar_init(empty_bar + s, kConsumerWarps);
        }
        fence_barrier_init();
        *abort_flag = 0;
    }
    for (int i = tid; i <= p.n_pairs; i += kAttendThreads) pair_prefix[i] = p.plan.pair_row_prefix[i];
    for (int i = tid; i < p.n_pairs; i += kAttendThreads) pair_nseg[i] = p.plan.pair_nseg[i];
    __syncthreads();

    const int64_t total = pair_prefix[p.n_pairs];
    int64_t rows_per_cta = (total + gridDim.x - 1) / gridDim.x;
    if (rows_per_cta < p.min_rows_per_cta) rows_per_cta = p.min_rows_per_cta;
    int64_t r0 = (int64_t)blockIdx.x * rows_per_cta;
    if (r0 >= total) return;
    const int64_t r1 = min(r0 + rows_per_cta, total);

    int pair;
    {
        int lo = 0, hi = p.n_pairs;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (pair_prefix[mid] <= r0) lo = mid; else hi = mid;
        }
        pair = lo;
    }

    uint32_t g_stage = 0;          // stages issued so far by this CTA (same count in every thread)

    while (r0 < r1) {
        const int64_t pb = pair_prefix[pair], pe = pair_prefix[pair + 1];
        const int a = (int)(r0 - pb);
        const int bnd = (int)(min(r1, pe) - pb);
        const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;
        const int cap = p.plan.seg_cap;
        const int nseg = pair_nseg[pair];

        __syncthreads();                                   // the previous span is done with the tables
        {
            const int32_t *g_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
            const int32_t *g_row = p.plan.seg_row + (size_t)pair * cap;
            const uint32_t *g_mask = p.plan.seg_mask + (size_t)pair * cap;
            const float *g_logc = p.plan.seg_logc + (size_t)pair * cap * G;
            for (int i = tid; i < nseg; i += kAttendThreads) {
                seg_prefix[i] = g_prefix[i];
                seg_row[i] = g_row[i];
                seg_mask[i] = g_mask[i];
            }
            if (tid == 0) seg_prefix[nseg] = g_prefix[nseg];
            if (!kAll)
                for (int e = tid; e < nseg * G; e += kAttendThreads) (&seg_logc[0][0])[e] = g_logc[e];
            for (int e = tid; e < G * kHeadDim; e += kAttendThreads) {
                const int h = e >> 7, d = e & 127;
                q_s[h][d] = bf16_to_float(p.q[((size_t)b * p.bv.n_q + (size_t)j * G + h) * kHeadDim + d])
                            * p.qk_scale_log2;
            }
        }
        __syncthreads();

        const int n_st = (bnd - a + kStageRows - 1) / kStageRows;
        const unsigned char *k_plane = reinterpret_cast<const unsigned char *>(p.k_packed)
                                       + (size_t)j * p.bv.rows_total * kRowBytes;
        const unsigned char *v_plane = reinterpret_cast<const unsigned char *>(p.v_packed)
                                       + (size_t)j * p.bv.rows_total * kRowBytes;

        float m[G], l[G], acc[G][8];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            m[h] = -CUDART_INF_F;
            l[h] = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[h][i] = 0.f;
        }

        int st_issued = 0;                                 // producer thread: stages issued in this span
        if (is_producer) {
            if (lane == 0) {
                // the ring may have been used as scratch by the previous span's merge
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                int cur = 0;
                {   // first segment of the span
                    int lo = 0, hi = nseg;
                    while (hi - lo > 1) {
                        const int mid = (lo + hi) >> 1;
                        if (seg_prefix[mid] <= a) lo = mid; else hi = mid;
                    }
                    cur = lo;
                }
                for (int st = 0; st < n_st; ++st) {
                    const uint32_t gs = g_stage + st;
                    const int slot = gs % kStages;
                    if (gs >= kStages && !mbar_wait(empty_bar + slot, ((gs / kStages) - 1) & 1, abort_flag)) break;
                    const int base = a + st * kStageRows, end = min(base + kStageRows, bnd);
                    unsigned char *kst = ring + (size_t)slot * kStageBytes;
                    unsigned char *vst = kst + kStageRows * kRowBytes;
                    mbar_arrive_expect_tx(full_bar + slot, (uint32_t)(end - base) * 2 * kRowBytes);
                    int pos = base;
                    while (pos < end) {
                        while (pos >= seg_prefix[cur + 1]) ++cur;
                        const int run_end = min(end, seg_prefix[cur + 1]);
                        const uint32_t bytes = (uint32_t)(run_end - pos) * kRowBytes;
                        const size_t row = (size_t)seg_row[cur] + (size_t)(pos - seg_prefix[cur]);
                        const bool suf = (seg_mask[cur] & kSrcSuffix) != 0u;
                        const unsigned char *ks = (suf ? reinterpret_cast<const unsigned char *>(p.k_suffix) : k_plane)
                                                  + row * kRowBytes;
                        const unsigned char *vs = (suf ? reinterpret_cast<const unsigned char *>(p.v_suffix) : v_plane)
                                                  + row * kRowBytes;
                        bulk_copy_g2s(kst + (size_t)(pos - base) * kRowBytes, ks, bytes, full_bar + slot);
                        bulk_copy_g2s(vst + (size_t)(pos - base) * kRowBytes, vs, bytes, full_bar + slot);
                        pos = run_end;
                    }
                    st_issued = st + 1;
                }
            }
        } else {
            int cur = 0;
            {
                int lo = 0, hi = nseg;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (seg_prefix[mid] <= a) lo = mid; else hi = mid;
                }
                cur = lo;
            }
            for (int st = 0; st < n_st; ++st) {
                const uint32_t gs = g_stage + st;
                const int slot = gs % kStages;
                if (!mbar_wait(full_bar + slot, (gs / kStages) & 1, abort_flag)) break;
                const int base = a + st * kStageRows, end = min(base + kStageRows, bnd);
                const unsigned char *kst = ring + (size_t)slot * kStageBytes;
                const unsigned char *vst = kst + kStageRows * kRowBytes;

                uint4 kk[kRowsPerHalfWarp], vv[kRowsPerHalfWarp];
                int segi[kRowsPerHalfWarp];
                uint32_t msk[kRowsPerHalfWarp];
                uint32_t any = 0u;
#pragma unroll
                for (int u = 0; u < kRowsPerHalfWarp; ++u) {
                    const int pos = base + u * kHalfWarps + hw;
                    msk[u] = 0u;
                    segi[u] = 0;
                    kk[u] = make_uint4(0u, 0u, 0u, 0u);
                    vv[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (pos < end) {
                        while (pos >= seg_prefix[cur + 1]) ++cur;
                        kk[u] = *reinterpret_cast<const uint4 *>(kst + (size_t)(pos - base) * kRowBytes + l16 * 16);
                        vv[u] = *reinterpret_cast<const uint4 *>(vst + (size_t)(pos - base) * kRowBytes + l16 * 16);
                        msk[u] = seg_mask[cur] & 0xFFu;
                        segi[u] = cur;
                    }
                    any |= msk[u];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar + slot);          // the rows are in registers
                if (!kAll) any |= __shfl_xor_sync(0xFFFFFFFFu, any, 16);

#pragma unroll
                for (int h = 0; h < G; ++h) {
                    if (kAll || ((any >> h) & 1u)) {
                        const float4 qa = *reinterpret_cast<const float4 *>(&q_s[h][l16 * 8]);
                        const float4 qb = *reinterpret_cast<const float4 *>(&q_s[h][l16 * 8 + 4]);
                        float sc[kRowsPerHalfWarp];
                        float mx = -CUDART_INF_F;
#pragma unroll
                        for (int u = 0; u < kRowsPerHalfWarp; ++u) {
                            float d = bf16_lo(kk[u].x) * qa.x;
                            d = fmaf(bf16_hi(kk[u].x), qa.y, d);
                            d = fmaf(bf16_lo(kk[u].y), qa.z, d);
                            d = fmaf(bf16_hi(kk[u].y), qa.w, d);
                            d = fmaf(bf16_lo(kk[u].z), qb.x, d);
                            d = fmaf(bf16_hi(kk[u].z), qb.y, d);
                            d = fmaf(bf16_lo(kk[u].w), qb.z, d);
                            d = fmaf(bf16_hi(kk[u].w), qb.w, d);
                            d += __shfl_xor_sync(0xFFFFFFFFu, d, 8);
                            d += __shfl_xor_sync(0xFFFFFFFFu, d, 4);
                            d += __shfl_xor_sync(0xFFFFFFFFu, d, 2);
                            d += __shfl_xor_sync(0xFFFFFFFFu, d, 1);
                            const bool on = (msk[u] >> h) & 1u;
                            if (!kAll) d -= seg_logc[segi[u]][h];
                            sc[u] = on ? d : -CUDART_INF_F;
                            mx = fmaxf(mx, sc[u]);
                        }
                        if (mx > m[h]) {
                            const float f = exp2f(m[h] - mx);          // 0 on the first rows
                            l[h] *= f;
#pragma unroll
                            for (int i = 0; i < 8; ++i) acc[h][i] *= f;
                            m[h] = mx;
                        }
#pragma unroll
                        for (int u = 0; u < kRowsPerHalfWarp; ++u) {
                            const bool on = (msk[u] >> h) & 1u;
                            const float pw = on ? exp2f(sc[u] - m[h]) : 0.f;
                            l[h] += pw;
                            acc[h][0] = fmaf(pw, bf16_lo(vv[u].x), acc[h][0]);
                            acc[h][1] = fmaf(pw, bf16_hi(vv[u].x), acc[h][1]);
                            acc[h][2] = fmaf(pw, bf16_lo(vv[u].y), acc[h][2]);
                            acc[h][3] = fmaf(pw, bf16_hi(vv[u].y), acc[h][3]);
                            acc[h][4] = fmaf(pw, bf16_lo(vv[u].z), acc[h][4]);
                            acc[h][5] = fmaf(pw, bf16_hi(vv[u].z), acc[h][5]);
                            acc[h][6] = fmaf(pw, bf16_lo(vv[u].w), acc[h][6]);
                            acc[h][7] = fmaf(pw, bf16_hi(vv[u].w), acc[h][7]);
                        }
                    }
                }
            }
        }
        g_stage += (uint32_t)n_st;
        __syncthreads();                                   // every stage of the span is consumed
        if (*abort_flag) {
            // a bounded wait ran out: report, let copies already issued land, and leave
            if (tid == 0 && p.status) atomicOr(p.status, 2);
            if (is_producer && lane == 0) {
                const uint32_t issued = g_stage - (uint32_t)n_st + (uint32_t)st_issued;
                for (uint32_t gs = issued > (uint32_t)kStages ? issued - kStages : 0u; gs < issued; ++gs)
                    for (uint32_t it = 0; it < kSpinLimit; ++it)
                        if (mbar_try_wait(full_bar + gs % kStages, (gs / kStages) & 1)) break;
            }
            __syncthreads();
            return;
        }

        // ---- merge the consumer warps into one partial (the ring is free: reuse it) ----
        float(*red_acc)[G][kHeadDim] = reinterpret_cast<float(*)[G][kHeadDim]>(smem + S::red_acc);
        float(*red_m)[G] = reinterpret_cast<float(*)[G]>(smem + S::red_m);
        float(*red_l)[G] = reinterpret_cast<float(*)[G]>(smem + S::red_l);
        if (!is_producer) {
#pragma unroll
            for (int h = 0; h < G; ++h) {
                const float mo = __shfl_xor_sync(0xFFFFFFFFu, m[h], 16);
                const float mm = fmaxf(m[h], mo);
                const float f = m[h] > -CUDART_INF_F ? exp2f(m[h] - mm) : 0.f;
                float lh = l[h] * f;
                lh += __shfl_xor_sync(0xFFFFFFFFu, lh, 16);
                float av[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    av[i] = acc[h][i] * f;
                    av[i] += __shfl_xor_sync(0xFFFFFFFFu, av[i], 16);
                }
                if (lane < 16) {
                    *reinterpret_cast<float4 *>(&red_acc[warp][h][l16 * 8]) = make_float4(av[0], av[1], av[2], av[3]);
                    *reinterpret_cast<float4 *>(&red_acc[warp][h][l16 * 8 + 4]) = make_float4(av[4], av[5], av[6], av[7]);
                }
                if (lane == 0) { red_m[warp][h] = mm; red_l[warp][h] = lh; }
            }
        }
        __syncthreads();
        const int slot_id = blockIdx.x + pair;
        float *part = p.partials + (size_t)slot_id * G * kPartialStride;
        if (!is_producer) {
            for (int e = tid; e < G * kHeadDim; e += kConsumerThreads) {
                const int h = e >> 7, d = e & 127;
                float mh = -CUDART_INF_F;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) mh = fmaxf(mh, red_m[w][h]);
                float num = 0.f, den = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float mw = red_m[w][h];
                    const float f = mw > -CUDART_INF_F ? exp2f(mw - mh) : 0.f;
                    num = fmaf(f, red_acc[w][h][d], num);
                    den = fmaf(f, red_l[w][h], den);
                }
                part[h * kPartialStride + 4 + d] = num;
                if (d == 0) { part[h * kPartialStride] = mh; part[h * kPartialStride + 1] = den; }
            }
        }

        // ---- last CTA of the pair: log-sum-exp merge of the pair's partials ----
        const int c_lo = (int)(pb / rows_per_cta), c_hi = (int)((pe - 1) / rows_per_cta);
        const int n_ctas = c_hi - c_lo + 1;
        __threadfence();
        __syncthreads();
        if (tid == 0) *last_flag = (atomicAdd(p.ctl.attend_ticket + pair, 1) == n_ctas - 1);
        __syncthreads();
        if (*last_flag) {
            __threadfence();
            if (tid == 0) p.ctl.attend_ticket[pair] = 0;              // every CTA of the pair has arrived
            const float *first = p.partials + (size_t)(c_lo + pair) * G * kPartialStride;
            float(*wbuf)[kMaxAttendGrid] = reinterpret_cast<float(*)[kMaxAttendGrid]>(smem + S::wbuf);
            if (warp < G) {
                const int h = warp;
                float mh = -CUDART_INF_F;
                for (int c = lane; c < n_ctas; c += 32)
                    mh = fmaxf(mh, __ldcg(first + ((size_t)c * G + h) * kPartialStride));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mh = fmaxf(mh, __shfl_xor_sync(0xFFFFFFFFu, mh, o));
                float den = 0.f;
                for (int c = lane; c < n_ctas; c += 32) {
                    const float *pp = first + ((size_t)c * G + h) * kPartialStride;
                    const float mj = __ldcg(pp);
                    const float wgt = mj > -CUDART_INF_F ? exp2f(mj - mh) : 0.f;
                    wbuf[h][c] = wgt;
                    den = fmaf(wgt, __ldcg(pp + 1), den);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xFFFFFFFFu, den, o);
                __syncwarp();
                float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
                for (int c = 0; c < n_ctas; ++c) {
                    const float wgt = wbuf[h][c];
                    const float4 *pp = reinterpret_cast<const float4 *>(first + ((size_t)c * G + h) * kPartialStride + 4);
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (wgt != 0.f) v = __ldcg(pp + lane);
                    num.x = fmaf(wgt, v.x, num.x);
                    num.y = fmaf(wgt, v.y, num.y);
                    num.z = fmaf(wgt, v.z, num.z);
                    num.w = fmaf(wgt, v.w, num.w);
                }
                const float inv = 1.f / den;
                const float4 o = make_float4(num.x * inv, num.y * inv, num.z * inv, num.w * inv);
                *reinterpret_cast<float4 *>(p.out + ((size_t)b * p.bv.n_q + (size_t)j * G + h) * kHeadDim + lane * 4) = o;
                if (p.status && !(isfinite(o.x) && isfinite(o.y) && isfinite(o.z) && isfinite(o.w)))
                    atomicOr(p.status, 1);
            }
        }
        r0 = pb + bnd;
        ++pair;
    }
}

template <int G>
cudaError_t launch_attend_g(const AttendParams &p, bool all_heads, int grid, cudaStream_t s)
{
    const size_t smem = Smem<G>::total;
    static thread_local bool attr_set = false;
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(attend_kernel<G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               (int)smem);
        if (err != cudaSuccess) return err;
        err = cudaFuncSetAttribute(attend_kernel<G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    if (all_heads) attend_kernel<G, true><<<grid, kAttendThreads, smem, s>>>(p);
    else           attend_kernel<G, false><<<grid, kAttendThreads, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

int attend_grid_size()
{
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms > kMaxAttendGrid ? kMaxAttendGrid : sms;
}

int attend_max_segments() { return kSegMax; }
int attend_max_pairs() { return kPairMax; }

cudaError_t launch_attend(const AttendParams &p, bool all_heads, int grid, cudaStream_t s)
{
    switch (p.bv.group) {
        case 1: return launch_attend_g<1>(p, all_heads, grid, s);
        case 2: return launch_attend_g<2>(p, all_heads, grid, s);
        case 3: return launch_attend_g<3>(p, all_heads, grid, s);
        case 4: return launch_attend_g<4>(p, all_heads, grid, s);
        case 5: return launch_attend_g<5>(p, all_heads, grid, s);
        case 6: return launch_attend_g<6>(p, all_heads, grid, s);
        case 7: return launch_attend_g<7>(p, all_heads, grid, s);
        case 8: return launch_attend_g<8>(p, all_heads, grid, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace santapp
