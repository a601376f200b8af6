// Routing for SANTA++ decode attention (Algorithm 1, the steps before the selection):
//   route_score_kernel   representative scores for the query heads of a KV head, routing logit
//                        phi_g = log n_g + q.l_g * scale (Eq. method-routing), Gumbel draw from
//                        the keyed Philox stream, perturbed score Y_g = phi_g + G_g. fp64.
//   dense_plan_kernel    the trivial plan that reads every prompt row and the suffix.
#include "common.cuh"
#include "plan.cuh"

namespace santapp {

namespace {

constexpr int kRouteThreads = 256;
constexpr int kRouteTeamsPerCta = 64;      // 8 warps x 2 quads x 4 teams

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
        for (int h = 0; h < kMaxGroup; ++h) p.plan.seg_logc[(size_t)pair * cap * kMaxGroup + h] = 0.f;
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

cudaError_t launch_dense_plan(const SelectParams &p, cudaStream_t s)
{
    dense_plan_kernel<<<1, 256, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace santapp
