// Exact attention over a read plan (Algorithm 1, the reads and the estimator):
// every member row of every selected team enters head h's sums with weight e^{s_i} / c_g
// (applied as s_i - log c_g, so the same correction enters the mass and the value sum), every
// suffix row with weight e^{s_i}; Eq. (method-estimate). The rows of all (sequence, KV head)
// pairs form one global row space that is cut into equal contiguous ranges, one per CTA
// (split-K by rows, not by teams); each CTA leaves one online-softmax partial per pair it
// touched and the last CTA to finish a pair merges that pair's partials by log-sum-exp.
#include <math_constants.h>

#include "common.cuh"

namespace santapp {

namespace {

constexpr int kAttendThreads = 256;
constexpr int kHalfWarps = kAttendThreads / 16;
constexpr int kSegStage = 128;         // plan segments staged in shared memory at a time
constexpr int kMaxAttendGrid = 512;    // partial slots of one pair that a merge can weigh

__device__ __forceinline__ uint4 ld_stream(const uint4 *ptr)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(ptr));
    return r;
}

template <int G>
struct AttendShared {
    float q[G][kHeadDim];              // pre-multiplied by scale * log2(e)
    int seg_prefix[kSegStage + 1];
    int seg_row[kSegStage];
    uint32_t seg_mask[kSegStage];
    float seg_logc[kSegStage][G];
    float red_m[kHalfWarps][G];
    float out_l[G];
    float out_acc[G][kHeadDim];
    float w[kMaxAttendGrid][G];
    int flag;
};

template <int G, bool kAll, int U>
__global__ void __launch_bounds__(kAttendThreads, kAll ? 1 : 2)
attend_kernel(AttendParams p)
{
    __shared__ AttendShared<G> sh;
    const int tid = threadIdx.x;
    const int hw = tid >> 4, l16 = tid & 15;

    const int64_t total = p.plan.pair_row_prefix[p.n_pairs];
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
            if (p.plan.pair_row_prefix[mid] <= r0) lo = mid; else hi = mid;
        }
        pair = lo;
    }

    while (r0 < r1) {
        const int64_t pb = p.plan.pair_row_prefix[pair], pe = p.plan.pair_row_prefix[pair + 1];
        int a = (int)(r0 - pb);
        const int bnd = (int)(min(r1, pe) - pb);
        const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;
        const int cap = p.plan.seg_cap;
        const int32_t *g_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
        const int32_t *g_row = p.plan.seg_row + (size_t)pair * cap;
        const uint32_t *g_mask = p.plan.seg_mask + (size_t)pair * cap;
        const float *g_logc = p.plan.seg_logc + (size_t)pair * cap * G;
        const int nseg = p.plan.pair_nseg[pair];

        __syncthreads();
        for (int e = tid; e < G * kHeadDim; e += kAttendThreads) {
            const int h = e >> 7, d = e & 127;
            sh.q[h][d] = bf16_to_float(p.q[((size_t)b * p.bv.n_q + (size_t)j * G + h) * kHeadDim + d])
                         * p.qk_scale_log2;
            sh.out_acc[h][d] = 0.f;
        }
        if (tid < G) sh.out_l[tid] = 0.f;

        float m[G], l[G], acc[G][8];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            m[h] = -CUDART_INF_F;
            l[h] = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[h][i] = 0.f;
        }

        int s;      // first segment of the span: g_prefix[s] <= a < g_prefix[s + 1]
        {
            int lo = 0, hi = nseg;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (g_prefix[mid] <= a) lo = mid; else hi = mid;
            }
            s = lo;
        }

        const uint16_t *k_plane = p.k_packed + (size_t)j * p.bv.rows_total * kHeadDim;
        const uint16_t *v_plane = p.v_packed + (size_t)j * p.bv.rows_total * kHeadDim;

        while (a < bnd) {
            __syncthreads();
            const int nload = min(kSegStage, nseg - s);
            for (int i = tid; i < nload; i += kAttendThreads) {
                sh.seg_prefix[i] = g_prefix[s + i];
                sh.seg_row[i] = g_row[s + i];
                sh.seg_mask[i] = g_mask[s + i];
            }
            if (tid == 0) sh.seg_prefix[nload] = g_prefix[s + nload];
            if (!kAll)
                for (int e = tid; e < nload * G; e += kAttendThreads)
                    sh.seg_logc[e / G][e % G] = g_logc[(size_t)s * G + e];
            __syncthreads();
            const int sub_end = min(bnd, sh.seg_prefix[nload]);

            int cur = 0;
            for (int base = a; base < sub_end; base += kHalfWarps * U) {
                uint4 kk[U], vv[U];
                int segi[U];
                uint32_t msk[U];
                uint32_t any = 0u;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int pos = base + u * kHalfWarps + hw;
                    msk[u] = 0u;
                    segi[u] = 0;
                    kk[u] = make_uint4(0u, 0u, 0u, 0u);
                    vv[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (pos < sub_end) {
                        while (pos >= sh.seg_prefix[cur + 1]) ++cur;
                        const uint32_t mk = sh.seg_mask[cur];
                        const size_t row = (size_t)sh.seg_row[cur] + (size_t)(pos - sh.seg_prefix[cur]);
                        const bool suf = (mk & kSrcSuffix) != 0u;
                        const uint16_t *kb = suf ? p.k_suffix : k_plane;
                        const uint16_t *vb = suf ? p.v_suffix : v_plane;
                        kk[u] = ld_stream(reinterpret_cast<const uint4 *>(kb + row * kHeadDim) + l16);
                        vv[u] = ld_stream(reinterpret_cast<const uint4 *>(vb + row * kHeadDim) + l16);
                        msk[u] = mk & 0xFFu;
                        segi[u] = cur;
                    }
                    any |= msk[u];
                }
                if (!kAll) any |= __shfl_xor_sync(0xFFFFFFFFu, any, 16);

#pragma unroll
                for (int h = 0; h < G; ++h) {
                    if (kAll || ((any >> h) & 1u)) {
                        const float4 qa = *reinterpret_cast<const float4 *>(&sh.q[h][l16 * 8]);
                        const float4 qb = *reinterpret_cast<const float4 *>(&sh.q[h][l16 * 8 + 4]);
                        float sc[U];
                        float mx = -CUDART_INF_F;
#pragma unroll
                        for (int u = 0; u < U; ++u) {
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
                            if (!kAll) d -= sh.seg_logc[segi[u]][h];
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
                        for (int u = 0; u < U; ++u) {
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
            a = sub_end;
            s += nload;
        }

        // ---- merge the 16 half-warps of the CTA into one partial ----
        if (l16 == 0) {
#pragma unroll
            for (int h = 0; h < G; ++h) sh.red_m[hw][h] = m[h];
        }
        __syncthreads();
        const int slot = blockIdx.x + pair;
        float *part = p.partials + (size_t)slot * G * kPartialStride;
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float mh = -CUDART_INF_F;
#pragma unroll
            for (int w = 0; w < kHalfWarps; ++w) mh = fmaxf(mh, sh.red_m[w][h]);
            if (m[h] > -CUDART_INF_F) {
                const float f = exp2f(m[h] - mh);
                if (l16 == 0) atomicAdd(&sh.out_l[h], l[h] * f);
#pragma unroll
                for (int i = 0; i < 8; ++i) atomicAdd(&sh.out_acc[h][l16 * 8 + i], acc[h][i] * f);
            }
            if (tid == 0) part[h * kPartialStride] = mh;
        }
        __syncthreads();
        for (int e = tid; e < G * kHeadDim; e += kAttendThreads) {
            const int h = e >> 7, d = e & 127;
            part[h * kPartialStride + 4 + d] = sh.out_acc[h][d];
        }
        if (tid < G) part[tid * kPartialStride + 1] = sh.out_l[tid];

        // ---- last CTA of the pair: log-sum-exp merge of the pair's partials ----
        const int c_lo = (int)(pb / rows_per_cta), c_hi = (int)((pe - 1) / rows_per_cta);
        const int n_ctas = c_hi - c_lo + 1;
        __threadfence();
        __syncthreads();
        if (tid == 0) sh.flag = (atomicAdd(p.ctl.attend_ticket + pair, 1) == n_ctas - 1);
        __syncthreads();
        if (sh.flag) {
            __threadfence();
            if (tid == 0) p.ctl.attend_ticket[pair] = 0;              // every CTA of the pair has arrived
            const float *first = p.partials + (size_t)(c_lo + pair) * G * kPartialStride;
            // common scale per head, then weights per (slot, head)
            if (tid < G) {
                float mh = -CUDART_INF_F;
                for (int c = 0; c < n_ctas; ++c)
                    mh = fmaxf(mh, __ldcg(first + ((size_t)c * G + tid) * kPartialStride));
                sh.out_l[tid] = mh;                                   // reuse as the common scale
            }
            __syncthreads();
            for (int e = tid; e < n_ctas * G; e += kAttendThreads) {
                const int c = e / G, h = e - c * G;
                const float mj = __ldcg(first + ((size_t)c * G + h) * kPartialStride);
                sh.w[c][h] = mj > -CUDART_INF_F ? exp2f(mj - sh.out_l[h]) : 0.f;
            }
            __syncthreads();
            for (int e = tid; e < G * kHeadDim; e += kAttendThreads) {
                const int h = e >> 7, d = e & 127;
                float num = 0.f, den = 0.f;
                for (int c = 0; c < n_ctas; ++c) {
                    const float wgt = sh.w[c][h];
                    if (wgt != 0.f) {
                        const float *pp = first + ((size_t)c * G + h) * kPartialStride;
                        num = fmaf(wgt, __ldcg(pp + 4 + d), num);
                        den = fmaf(wgt, __ldcg(pp + 1), den);
                    }
                }
                const float o = num / den;
                p.out[((size_t)b * p.bv.n_q + (size_t)j * G + h) * kHeadDim + d] = o;
                if (p.status && !isfinite(o)) atomicOr(p.status, 1);
            }
        }
        r0 = pb + bnd;
        ++pair;
    }
}

template <int G>
cudaError_t launch_attend_g(const AttendParams &p, bool all_heads, int grid, cudaStream_t s)
{
    if (all_heads) attend_kernel<G, true, 2><<<grid, kAttendThreads, 0, s>>>(p);
    else           attend_kernel<G, false, 4><<<grid, kAttendThreads, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

int attend_grid_size()
{
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int grid = 2 * sms;
    return grid > kMaxAttendGrid ? kMaxAttendGrid : grid;
}

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
