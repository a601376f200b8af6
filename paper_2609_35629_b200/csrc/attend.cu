// Exact attention over a read plan (Algorithm 1, the reads and the estimator):
// every member row of every selected team enters head h's sums with weight e^{s_i} / c_g
// (applied as s_i - log c_g, so the same correction enters the mass and the value sum), every
// suffix row with weight e^{s_i}; Eq. (method-estimate).
//
// Work split. The rows of all (sequence, KV head) pairs form one global row space that is cut
// into equal contiguous ranges, one per CTA (split-K by rows, not by teams), one CTA per SM.
// Inside a CTA the range is dealt out in blocks of 16 rows to eight consumer warps; two
// producer warps stream each block's K and V rows into that warp's private two-slot ring in
// shared memory with 16-byte asynchronous copies (whole 256-byte rows per half warp, XOR
// swizzled so that ldmatrix is bank-conflict free) and signal an mbarrier.
//
// Arithmetic. The GQA group is a real MMA tile: the query heads of the KV head (at most 8)
// are the M rows of S^T = q K^T (mma.sync m16n8k16, bf16 inputs, fp32 accumulation), so one
// row of K serves every head at once; a team contributes to a head only where the head
// selected it (mask), with the head's own correction. The weights are split into two bf16
// terms (p = p_hi + p_lo) so that O^T += V^T P^T keeps fp32-level accuracy.
//
// Each CTA leaves one online-softmax partial per pair it touched; the last CTA to finish a
// pair merges that pair's partials by log-sum-exp (the split-softmax reduction).
// Every wait on a barrier is bounded: on expiry the kernel raises a status bit and leaves.
#include <math_constants.h>

#include "common.cuh"

namespace santapp {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kProducerWarps = 2;
constexpr int kConsumerThreads = 32 * kConsumerWarps;
constexpr int kAttendThreads = 32 * (kConsumerWarps + kProducerWarps);
constexpr int kBlockRows = 16;                              // rows per block (one warp, one MMA K step)
constexpr int kSlots = 2;                                   // ring slots per consumer warp
constexpr int kRowBytes = kHeadDim * 2;                     // one bf16 row
constexpr int kTileBytes = kBlockRows * kRowBytes;          // K tile or V tile of a block
constexpr int kSlotBytes = 2 * kTileBytes;                  // K tile then V tile
constexpr int kSegMax = 1025;                               // plan segments of one pair (G * K + suffix)
constexpr int kPairMax = 1024;                              // pairs whose offsets are staged
constexpr int kMaxAttendGrid = 512;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kNoSeg = 0xFFFF;

// ---- primitives ----
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
// The executing thread's earlier cp.async copies arrive on the barrier when they complete.
__device__ __forceinline__ void cp_async_arrive(uint64_t *bar)
{
    asm volatile("cp.async.mbarrier.arrive.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
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
// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros instead.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D += A (16x16, row) * B (16x8, col), bf16 inputs, fp32 accumulation.
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                 "{%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// (lo, hi) -> bf16x2 with lo in the low half, round to nearest even.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// ---- shared memory carve-up (dynamic) ----
template <int G>
struct Smem {
    static constexpr size_t ring = 0;                                           // [warps][kSlots][kSlotBytes]
    static constexpr size_t ring_bytes = (size_t)kConsumerWarps * kSlots * kSlotBytes;
    static constexpr size_t bars = ring + ring_bytes;                           // full[w][s], empty[w][s]
    static constexpr size_t row_seg = bars + 2 * kConsumerWarps * kSlots * 8;   // u16 [w][s][16]
    static constexpr size_t seg_prefix = row_seg + kConsumerWarps * kSlots * kBlockRows * 2;   // int [kSegMax+1]
    static constexpr size_t seg_row = seg_prefix + (kSegMax + 3) * 4;           // int [kSegMax]
    static constexpr size_t seg_mask = seg_row + (kSegMax + 3) * 4;             // uint [kSegMax]
    static constexpr size_t seg_logc = seg_mask + (kSegMax + 3) * 4;            // float [kSegMax][G]
    static constexpr size_t pair_prefix = (seg_logc + (size_t)kSegMax * G * 4 + 15) / 16 * 16;  // int64 [kPairMax+1]
    static constexpr size_t pair_nseg = pair_prefix + (kPairMax + 1) * 8;       // int [kPairMax]
    static constexpr size_t misc = pair_nseg + kPairMax * 4;                    // flags
    static constexpr size_t total = misc + 64;
    // aliases of the ring, used only after a span's blocks are consumed
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
    extern __shared__ __align__(1024) unsigned char smem[];
    using S = Smem<G>;
    unsigned char *ring = smem + S::ring;
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + S::bars);          // [w * kSlots + s]
    uint64_t *empty_bar = full_bar + kConsumerWarps * kSlots;
    uint16_t *row_seg = reinterpret_cast<uint16_t *>(smem + S::row_seg);        // [(w * kSlots + s) * 16 + r]
    int *seg_prefix = reinterpret_cast<int *>(smem + S::seg_prefix);
    int *seg_row = reinterpret_cast<int *>(smem + S::seg_row);
    uint32_t *seg_mask = reinterpret_cast<uint32_t *>(smem + S::seg_mask);
    float(*seg_logc)[G] = reinterpret_cast<float(*)[G]>(smem + S::seg_logc);
    int64_t *pair_prefix = reinterpret_cast<int64_t *>(smem + S::pair_prefix);
    int *pair_nseg = reinterpret_cast<int *>(smem + S::pair_nseg);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + S::misc);
    int *last_flag = reinterpret_cast<int *>(smem + S::misc) + 1;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool is_producer = warp >= kConsumerWarps;
    const int g = lane >> 2, c = lane & 3;                 // MMA fragment coordinates

    if (tid == 0) {
        for (int s = 0; s < kConsumerWarps * kSlots; ++s) {
            mbar_init(full_bar + s, 32);                   // one arrival per producer lane
            mbar_init(empty_bar + s, 1);                   // the consumer warp's lane 0
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

    uint32_t g_block = 0;          // blocks dealt out so far by this CTA (same count in every thread)

    while (r0 < r1) {
        const int64_t pb = pair_prefix[pair], pe = pair_prefix[pair + 1];
        const int a = (int)(r0 - pb);
        const int bnd = (int)(min(r1, pe) - pb);
        const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;
        const int cap = p.plan.seg_cap;
        const int nseg = pair_nseg[pair];

        __syncthreads();                                   // the previous span is done with the tables
        {
            // one round trip: every load is issued before the first store
            const int32_t *g_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
            const int32_t *g_row = p.plan.seg_row + (size_t)pair * cap;
            const uint32_t *g_mask = p.plan.seg_mask + (size_t)pair * cap;
            const float *g_logc = p.plan.seg_logc + (size_t)pair * cap * G;
            for (int i0 = 0; i0 <= nseg; i0 += kAttendThreads) {
                const int i = i0 + tid;
                int v_prefix = 0, v_row = 0;
                uint32_t v_mask = 0u;
                float v_logc[G];
                if (i <= nseg) v_prefix = g_prefix[i];
                if (i < nseg) {
                    v_row = g_row[i];
                    v_mask = g_mask[i];
                    if (!kAll) {
#pragma unroll
                        for (int h = 0; h < G; ++h) v_logc[h] = g_logc[(size_t)i * G + h];
                    }
                }
                if (i <= nseg) seg_prefix[i] = v_prefix;
                if (i < nseg) {
                    seg_row[i] = v_row;
                    seg_mask[i] = v_mask;
                    if (!kAll) {
#pragma unroll
                        for (int h = 0; h < G; ++h) seg_logc[i][h] = v_logc[h];
                    }
                }
            }
        }
        // A fragments of q for the 8 k-steps: head g (zero rows for g >= G and for M rows 8..15)
        uint32_t qa[8][2];
        if (!is_producer) {
            const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
                p.q + ((size_t)b * p.bv.n_q + (size_t)j * G + (g < G ? g : 0)) * kHeadDim);
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                qa[s][0] = g < G ? __ldg(qrow + 8 * s + c) : 0u;
                qa[s][1] = g < G ? __ldg(qrow + 8 * s + 4 + c) : 0u;
            }
        }
        __syncthreads();

        const int n_blk = (bnd - a + kBlockRows - 1) / kBlockRows;
        const unsigned char *k_plane = reinterpret_cast<const unsigned char *>(p.k_packed)
                                       + (size_t)j * p.bv.rows_total * kRowBytes;
        const unsigned char *v_plane = reinterpret_cast<const unsigned char *>(p.v_packed)
                                       + (size_t)j * p.bv.rows_total * kRowBytes;

        // online-softmax state of head g (replicated over the quad) and O^T fragments:
        // o[t][r]: d = 16 t + g + 8 (r >> 1), head = 2 c + (r & 1)
        float m_run = -CUDART_INF_F, l_run = 0.f;
        float o[8][4];
#pragma unroll
        for (int t = 0; t < 8; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }

        if (is_producer) {
            // ---------------- producer warps: blocks of alternating parity ----------------
            const int pw = warp - kConsumerWarps;
            int cur = 0;                                   // segment cursor of lane r (r < 16)
            for (int bi = 0; bi < n_blk; ++bi) {
                const uint32_t gb = g_block + bi;
                if ((int)(gb % kProducerWarps) != pw) continue;
                const int w = gb % kConsumerWarps;
                const uint32_t u = gb / kConsumerWarps;
                const int slot = u % kSlots;
                const int bs = w * kSlots + slot;
                if (u >= (uint32_t)kSlots &&
                    !__all_sync(0xFFFFFFFFu, mbar_wait(empty_bar + bs, ((u / kSlots) - 1) & 1, abort_flag)))
                    break;
                // lane r < 16 resolves row r of the block
                const int pos = a + bi * kBlockRows + (lane & 15);
                const bool valid = pos < bnd;
                int64_t grow = 0;
                int suf = 0;
                if (valid) {
                    if (pos >= seg_prefix[cur + 1]) {      // moved on: binary search from here
                        int lo = cur + 1, hi = nseg;
                        while (hi - lo > 1) {
                            const int mid = (lo + hi) >> 1;
                            if (seg_prefix[mid] <= pos) lo = mid; else hi = mid;
                        }
                        cur = lo;
                    }
                    grow = (int64_t)seg_row[cur] + (pos - seg_prefix[cur]);
                    suf = (seg_mask[cur] & kSrcSuffix) ? 1 : 0;
                }
                if (lane < 16) row_seg[bs * kBlockRows + lane] = (uint16_t)(valid ? cur : kNoSeg);
                const uint32_t slot_addr = smem_u32(ring + (size_t)bs * kSlotBytes);
                const int chunk = lane & 15;
#pragma unroll
                for (int piece = 0; piece < kBlockRows / 2; ++piece) {
                    const int row = 2 * piece + (lane >> 4);
                    const int64_t rr = __shfl_sync(0xFFFFFFFFu, grow, row);
                    const int rs = __shfl_sync(0xFFFFFFFFu, suf, row);
                    const int rv = __shfl_sync(0xFFFFFFFFu, (int)valid, row);
                    const unsigned char *ks = (rs ? reinterpret_cast<const unsigned char *>(p.k_suffix) : k_plane)
                                              + rr * kRowBytes + chunk * 16;
                    const unsigned char *vs = (rs ? reinterpret_cast<const unsigned char *>(p.v_suffix) : v_plane)
                                              + rr * kRowBytes + chunk * 16;
                    const uint32_t dst = slot_addr + row * kRowBytes + ((chunk ^ (row & 7)) << 4);
                    cp_async16(dst, ks, rv ? 16u : 0u);
                    cp_async16(dst + kTileBytes, vs, rv ? 16u : 0u);
                }
                cp_async_arrive(full_bar + bs);
                mbar_arrive(full_bar + bs);
            }
        } else {
            // ---------------- consumer warps ----------------
            const float qk = p.qk_scale_log2;
            int first = (int)((warp + kConsumerWarps - (g_block % kConsumerWarps)) % kConsumerWarps);
            for (int bi = first; bi < n_blk; bi += kConsumerWarps) {
                const uint32_t gb = g_block + bi;
                const uint32_t u = gb / kConsumerWarps;
                const int slot = u % kSlots;
                const int bs = warp * kSlots + slot;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait(full_bar + bs, (u / kSlots) & 1, abort_flag))) break;
                const uint32_t k_addr = smem_u32(ring + (size_t)bs * kSlotBytes);
                const uint32_t v_addr = k_addr + kTileBytes;

                // the four (row, head g) entries of this thread: rows 2c, 2c+1, 8+2c, 9+2c
                bool on[4];
                float lc[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = 2 * c + (i & 1) + 8 * (i >> 1);
                    lc[i] = 0.f;
                    if (kAll) {
                        on[i] = (g < G) && (a + bi * kBlockRows + r < bnd);
                    } else {
                        const int sg = row_seg[bs * kBlockRows + r];
                        on[i] = false;
                        if (sg != kNoSeg && g < G) {
                            on[i] = (seg_mask[sg] >> g) & 1u;
                            lc[i] = seg_logc[sg][g];
                        }
                    }
                }

                // S^T = q K^T for the two 8-row groups
                float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
                {
                    const int lrow = lane & 7, lmat = lane >> 3;
#pragma unroll
                    for (int sp = 0; sp < 4; ++sp) {
                        uint32_t kb0[4], kb1[4];
                        const int chunk = 4 * sp + lmat;
                        ldmatrix_x4(kb0, k_addr + lrow * kRowBytes + ((chunk ^ lrow) << 4));
                        ldmatrix_x4(kb1, k_addr + (8 + lrow) * kRowBytes + ((chunk ^ lrow) << 4));
                        mma_bf16(s0, qa[2 * sp][0], 0u, qa[2 * sp][1], 0u, kb0[0], kb0[1]);
                        mma_bf16(s1, qa[2 * sp][0], 0u, qa[2 * sp][1], 0u, kb1[0], kb1[1]);
                        mma_bf16(s0, qa[2 * sp + 1][0], 0u, qa[2 * sp + 1][1], 0u, kb0[2], kb0[3]);
                        mma_bf16(s1, qa[2 * sp + 1][0], 0u, qa[2 * sp + 1][1], 0u, kb1[2], kb1[3]);
                    }
                }
                float sc[4];
                sc[0] = on[0] ? fmaf(s0[0], qk, -lc[0]) : -CUDART_INF_F;
                sc[1] = on[1] ? fmaf(s0[1], qk, -lc[1]) : -CUDART_INF_F;
                sc[2] = on[2] ? fmaf(s1[0], qk, -lc[2]) : -CUDART_INF_F;
                sc[3] = on[3] ? fmaf(s1[1], qk, -lc[3]) : -CUDART_INF_F;
                float mloc = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
                mloc = fmaxf(mloc, __shfl_xor_sync(0xFFFFFFFFu, mloc, 1));
                mloc = fmaxf(mloc, __shfl_xor_sync(0xFFFFFFFFu, mloc, 2));
                const float m_new = fmaxf(m_run, mloc);
                const bool grew = m_new > m_run;
                if (__any_sync(0xFFFFFFFFu, grew)) {
                    const float f = grew ? exp2f(m_run - m_new) : 1.f;          // exp2f(-inf) = 0 on first rows
                    l_run *= f;
                    const float fe = __shfl_sync(0xFFFFFFFFu, f, 8 * c);        // head 2c lives in lanes 8c..8c+3
                    const float fo = __shfl_sync(0xFFFFFFFFu, f, 8 * c + 4);    // head 2c+1
#pragma unroll
                    for (int t = 0; t < 8; ++t) { o[t][0] *= fe; o[t][1] *= fo; o[t][2] *= fe; o[t][3] *= fo; }
                    m_run = m_new;
                }
                float pw[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) pw[i] = on[i] ? exp2f(sc[i] - m_run) : 0.f;
                l_run += (pw[0] + pw[1]) + (pw[2] + pw[3]);
                // P^T as B fragments, split in two bf16 terms
                const uint32_t ph0 = pack_bf16x2(pw[0], pw[1]), ph1 = pack_bf16x2(pw[2], pw[3]);
                const uint32_t pl0 = pack_bf16x2(pw[0] - bf16_lo(ph0), pw[1] - bf16_hi(ph0));
                const uint32_t pl1 = pack_bf16x2(pw[2] - bf16_lo(ph1), pw[3] - bf16_hi(ph1));

                // O^T += V^T P^T
                {
                    const int lrow = lane & 7, lmat = lane >> 3;
                    const int vrow = (lmat >> 1) * 8 + lrow;
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        uint32_t va[4];
                        const int chunk = 2 * t + (lmat & 1);
                        ldmatrix_x4_trans(va, v_addr + vrow * kRowBytes + ((chunk ^ lrow) << 4));
                        mma_bf16(o[t], va[0], va[1], va[2], va[3], ph0, ph1);
                        mma_bf16(o[t], va[0], va[1], va[2], va[3], pl0, pl1);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar + bs);
            }
        }
        g_block += (uint32_t)n_blk;
        __syncthreads();                                   // every block of the span is consumed
        if (*abort_flag) {
            // a bounded wait ran out: report, let copies already issued land, and leave
            if (tid == 0 && p.status) atomicOr(p.status, 2);
            if (is_producer) asm volatile("cp.async.wait_all;" ::: "memory");
            __syncthreads();
            return;
        }

        // ---- merge the consumer warps into one partial (the ring is free: reuse it) ----
        float(*red_acc)[G][kHeadDim] = reinterpret_cast<float(*)[G][kHeadDim]>(smem + S::red_acc);
        float(*red_m)[G] = reinterpret_cast<float(*)[G]>(smem + S::red_m);
        float(*red_l)[G] = reinterpret_cast<float(*)[G]>(smem + S::red_l);
        if (!is_producer) {
            l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 1);
            l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 2);
            if (c == 0 && g < G) { red_m[warp][g] = m_run; red_l[warp][g] = l_run; }
#pragma unroll
            for (int t = 0; t < 8; ++t) {
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int h = 2 * c + (r & 1), d = 16 * t + g + 8 * (r >> 1);
                    if (h < G) red_acc[warp][h][d] = o[t][r];
                }
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
                for (int cc = lane; cc < n_ctas; cc += 32)
                    mh = fmaxf(mh, __ldcg(first + ((size_t)cc * G + h) * kPartialStride));
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) mh = fmaxf(mh, __shfl_xor_sync(0xFFFFFFFFu, mh, off));
                float den = 0.f;
                for (int cc = lane; cc < n_ctas; cc += 32) {
                    const float *pp = first + ((size_t)cc * G + h) * kPartialStride;
                    const float mj = __ldcg(pp);
                    const float wgt = mj > -CUDART_INF_F ? exp2f(mj - mh) : 0.f;
                    wbuf[h][cc] = wgt;
                    den = fmaf(wgt, __ldcg(pp + 1), den);
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) den += __shfl_xor_sync(0xFFFFFFFFu, den, off);
                __syncwarp();
                float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
                for (int cc = 0; cc < n_ctas; ++cc) {
                    const float wgt = wbuf[h][cc];
                    const float4 *pp = reinterpret_cast<const float4 *>(first + ((size_t)cc * G + h) * kPartialStride + 4);
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (wgt != 0.f) v = __ldcg(pp + lane);
                    num.x = fmaf(wgt, v.x, num.x);
                    num.y = fmaf(wgt, v.y, num.y);
                    num.z = fmaf(wgt, v.z, num.z);
                    num.w = fmaf(wgt, v.w, num.w);
                }
                const float inv = 1.f / den;
                const float4 ov = make_float4(num.x * inv, num.y * inv, num.z * inv, num.w * inv);
                *reinterpret_cast<float4 *>(p.out + ((size_t)b * p.bv.n_q + (size_t)j * G + h) * kHeadDim + lane * 4) = ov;
                if (p.status && !(isfinite(ov.x) && isfinite(ov.y) && isfinite(ov.z) && isfinite(ov.w)))
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
