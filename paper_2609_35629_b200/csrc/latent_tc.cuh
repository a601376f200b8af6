// Attention over shared-latent rows on the 5th-generation tensor cores (tcgen05, accumulators in
// tensor memory). Included by latent.cu, which defines the parameter struct and the constants.
//
// One block per SM, thirteen warps with fixed roles:
//   warps 0-3   softmax: read S^T (rows x heads) from tensor memory, keep the running reference
//               maximum and the row sums, write P^T (two bf16 terms) to shared memory, rescale
//               O^T when the maximum has grown by more than 2^8, write the block's partial result
//   warp 4      one lane issues every tcgen05.mma: S^T = Rows Q^T (M = 64 rows, N = 16 heads,
//               36 steps of K = 16), then O^T += V^T P^T (M = 128 value columns x 4, N = 16 heads,
//               K = 64 rows, for both terms of P)
//   warps 5-8 / 9-12  copy the even / odd 64-row tiles from global to shared memory (cp.async,
//               16-byte pieces laid out as the MMA's canonical no-swizzle layout, see below)
// The roles meet on mbarriers; every wait is bounded, and a wait that expires raises bit 2 of the
// status word, after which all waits return at once (the control flow never depends on data, so the
// block still ends; its result is then meaningless).
//
// Shared-memory layout of a tile of rows (and of the queries): the tensor core's 128-byte swizzle.
// 64 consecutive values of 8 consecutive rows form one 1024-byte atom: row r of the atom holds its
// eight 16-byte pieces j at r * 128 + ((j ^ r) * 16). The atom of row group g (8 rows) and column
// block a (64 values) lies at (a * groups + g) * 1024. A global sector (32 bytes of a row) thus lands
// in one 32-byte piece of shared memory, and a row's 128 bytes in one line, which keeps the copies'
// shared-memory writes few. Read as a K-major operand (S^T: rows are M, the 576 values K) row groups
// are 1024 bytes apart (stride offset) and a step of K = 16 advances the start by 32 bytes inside an
// atom; read as an MN-major operand (O^T: the value columns are M, the rows K) the same bytes have
// blocks of 64 value columns 1024 * groups bytes apart (leading offset) and groups of 8 rows 1024
// bytes (stride offset). One copy of a row serves as key and as value, and nothing is transposed.
#pragma once

namespace {

constexpr int kTcThreads = 416;
constexpr int kTcRows = 64;                                          // rows per tile = M of the S^T MMA
constexpr int kTcColBytes = (kTcRows / 8) * 1024;                    // 8192: one block of 64 values of all 64 rows
constexpr int kTcStageBytes = (kRowDim / 64) * kTcColBytes;          // 73728
constexpr int kTcQColBytes = (kHeads / 8) * 1024;                    // 2048: the same for the 16 queries
constexpr int kTcOffQ = 2 * kTcStageBytes;                           // queries, same layout (16 heads = 2 groups)
constexpr int kTcOffP = kTcOffQ + (kRowDim / 64) * kTcQColBytes;                 // P^T: [tile parity][term][2048]
constexpr int kTcOffBias = kTcOffP + 2 * 2 * 2048;                   // [tile parity][64 rows][kBiasPitch] floats
constexpr int kTcOffPrefix = kTcOffBias + 2 * kTcRows * kBiasPitch * 4;
constexpr int kTcOffRed = kTcOffPrefix + (kMaxLatentSeqs + 4) * 4;   // [2][4 warps][16] column maxima, [4][16] sums
constexpr int kTcOffBar = kTcOffRed + (2 * 4 * 16 + 4 * 16) * 4;     // 10 mbarriers
constexpr int kTcOffMisc = kTcOffBar + 10 * 8;                       // tensor-memory base, abort flag, scan scratch
constexpr int kTcSmemBytes = kTcOffMisc + 8 + 48 * 4;
constexpr uint32_t kTcColumns = 256;                                 // tensor-memory columns: S^T at columns 0 and 64, O^T 4 x 16 from column 128
constexpr uint32_t kTcColO = 128;
constexpr int kTcWaitLimit = 1 << 22;

enum { kBarFull = 0, kBarPvDone = 2, kBarSReady = 4, kBarSFree = 6, kBarPReady = 8 };

__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr, uint32_t leading_bytes, uint32_t stride_bytes)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((leading_bytes >> 4) & 0x3FFFu) << 16)
           | ((uint64_t)((stride_bytes >> 4) & 0x3FFFu) << 32) | ((uint64_t)1 << 46);      // version 1, no swizzle
}
__device__ __forceinline__ uint64_t tc_desc_sw128(uint32_t saddr, uint32_t leading_bytes, uint32_t stride_bytes)
{
    return tc_desc(saddr, leading_bytes, stride_bytes) | ((uint64_t)2 << 61);                // 128-byte swizzle
}
__device__ __forceinline__ uint32_t tc_idesc(int M, int N, int a_mn_major, int b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16)
           | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);                       // fp32 accumulate, bf16 x bf16
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n" ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
                 : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                   "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&v)[16])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
                 "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
                 "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Wait until the phase of `bar` with index `use` (0, 1, 2, ... in the order the phases complete) is
// over. The waiter is never more than one phase behind, so the parity identifies the phase.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t use, volatile int *abort_flag, int32_t *status)
{
    if (*abort_flag) return;
    for (int i = 0; i < kTcWaitLimit; ++i) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}\n"
                     : "=r"(done)
                     : "r"(bar), "r"(use & 1u)
                     : "memory");
        if (done) return;
    }
    *abort_flag = 1;
    if (status != nullptr) atomicOr(status, 4);
}

// Diagnostic: the calling thread notes the device timer in mark `slot` of its block (kernel 3 of the trace).
__device__ __forceinline__ void tc_mark(unsigned long long *trace, bool on, int slot)
{
    if (trace != nullptr && on && blockIdx.x < (unsigned)kTraceBlocks) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        trace[((size_t)3 * kTraceBlocks + blockIdx.x) * kTraceSlots + slot] = t;
    }
}

// One look at the phase (true once it is over, or once the block has given up waiting).
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t use, volatile int *abort_flag)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(done)
                 : "r"(bar), "r"(use & 1u)
                 : "memory");
    return done != 0 || *abort_flag != 0;
}

template <bool kAll>
__global__ void __launch_bounds__(kTcThreads, 1)
latent_attend_tc_kernel(LatentAttendParams p, int32_t *status)
{
    extern __shared__ __align__(1024) unsigned char smem_tc[];
    unsigned char *smem = smem_tc;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t *prefix = reinterpret_cast<uint32_t *>(smem + kTcOffPrefix);
    float *red_max = reinterpret_cast<float *>(smem + kTcOffRed);            // [2][4][16]
    float *red_sum = red_max + 2 * 4 * 16;                                   // [4][16]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kTcOffMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kTcOffMisc + 4);
    int *scan = reinterpret_cast<int *>(smem + kTcOffMisc + 8);
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t bar0 = smem_base + kTcOffBar;
    const int n = p.lv.n_seqs, H = p.lv.n_heads;

    // ---- set-up: barriers, tensor memory, the sequences' row prefix ----
    if (tid == 0) {
        *abort_flag = 0;
        const uint32_t counts[10] = {128, 128, 1, 1, 1, 1, 128, 128, 128, 128};
        for (int i = 0; i < 10; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0 + 8 * i), "r"(counts[i]));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_base + kTcOffMisc), "r"(kTcColumns));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    {
        uint32_t carry = 0;
        for (int base = 0; base < n; base += kTcThreads) {
            const int i = base + tid;
            int v = 0;
            if (i < n) {
                if (kAll) {
                    v = (int)(p.lv.seq_row_off[i + 1] - p.lv.seq_row_off[i]);
                    if (p.suffix_len != nullptr && p.suffix_cap > 0) v += max(0, min(p.suffix_len[i], p.suffix_cap));
                } else {
                    v = __ldcg(p.pair_rows + i);
                }
            }
            int total;
            const int excl = block_exclusive_scan(v, scan, total);
            if (i < n) prefix[i] = carry + (uint32_t)excl;
            carry += (uint32_t)total;
        }
        if (tid == 0) prefix[n] = carry;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (blockIdx.x == 0)
        for (int i = tid; i <= n; i += kTcThreads) p.pair_prefix[i] = prefix[i];
    const uint32_t total = prefix[n];
    const uint32_t per = (total + gridDim.x - 1) / gridDim.x;
    const uint32_t lo = min(total, blockIdx.x * per), hi = min(total, lo + per);
    int pr = 0;
    {
        int a = 0, c = n;                                   // largest pr with prefix[pr] <= lo
        while (c - a > 1) {
            const int mid = (a + c) >> 1;
            if (prefix[mid] <= lo) a = mid; else c = mid;
        }
        pr = a;
    }
    const uint4 *rows_g = reinterpret_cast<const uint4 *>(p.rows_packed);
    const uint4 *suffix_g = reinterpret_cast<const uint4 *>(p.suffix_rows);
    const uint32_t idesc_s = tc_idesc(kTcRows, kHeads, 0, 0), idesc_o = tc_idesc(128, kHeads, 1, 1);
    uint32_t gt0 = 0;                                       // tiles this block has processed before the current share

    for (; lo < hi && pr < n && prefix[pr] < hi; ++pr) {
        if (prefix[pr + 1] <= lo) continue;
        const int b = pr;
        const int s_lo = (int)(max(lo, prefix[pr]) - prefix[pr]), s_hi = (int)(min(hi, prefix[pr + 1]) - prefix[pr]);
        const int n_tiles = (s_hi - s_lo + kTcRows - 1) / kTcRows;
        const int64_t row0 = p.lv.seq_row_off[b];
        const int N = (int)(p.lv.seq_row_off[b + 1] - row0);

        // ---- the sequence's queries into shared memory (heads beyond n_heads are zero) ----
        {
            const uint4 *qg = reinterpret_cast<const uint4 *>(p.q + (size_t)b * H * kRowDim);
            for (int e = tid; e < kHeads * kRowChunks; e += kTcThreads) {
                const int h = e / kRowChunks, c = e - h * kRowChunks;
                const uint4 v = h < H ? __ldg(qg + (size_t)h * kRowChunks + c) : make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4 *>(smem + kTcOffQ + (c >> 3) * kTcQColBytes + (h >> 3) * 1024 + (h & 7) * 128 + (((c & 7) ^ (h & 7)) << 4)) = v;
            }
        }
        proxy_fence();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();

        if (warp >= 5) {
            // ================= copies: warps 5-8 take even tiles, 9-12 odd tiles =================
            const int par = (warp - 5) >> 2, pw = (warp - 5) & 3, pt = pw * 32 + lane;      // pt: 0..127 inside the four warps
            const int jl = lane & 7, rl = lane >> 3;        // a warp instruction copies 128 bytes of each of four rows
            const int2 *line = kAll ? nullptr : p.row_meta + row0 + (int64_t)b * p.suffix_cap;
            const float *bias_g = kAll ? nullptr : p.seg_bias + (size_t)b * p.seg_cap * kHeads;
            for (int i = 0; i < n_tiles; ++i) {
                const uint32_t g = gt0 + i;
                if ((int)(g & 1u) != par) continue;
                const int pos0 = s_lo + kTcRows * i;
                // source rows of this thread: rows 16 pw + 4 u + rl, u < 4, and row pt / 2 for the bias copy
                int src[4], seg_pt = 0;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int pos = pos0 + 16 * pw + 4 * u + rl;
                    if (pos >= s_hi) src[u] = -1;
                    else if (kAll) src[u] = pos < N ? (int)(row0 + pos) : (int)(kSrcSuffix | (uint32_t)(b * p.suffix_cap + pos - N));
                    else src[u] = __ldcg(line + pos).x;
                }
                const bool ok_pt = pos0 + (pt >> 1) < s_hi;
                if (!kAll && ok_pt) seg_pt = __ldcg(line + pos0 + (pt >> 1)).y;
                const bool tr = gt0 == 0 && i == 2 && pt == 0;
                tc_mark(p.trace, tr, 0);
                if (g >= 2) mbar_wait(bar0 + 8 * (kBarPvDone + par), (g >> 1) - 1, abort_flag, status);     // the stage is free
                tc_mark(p.trace, tr, 1);
                const uint32_t stage = smem_base + par * kTcStageBytes;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const bool valid = src[u] != -1;
                    const uint32_t s = (uint32_t)src[u];
                    const uint4 *gp = !valid ? rows_g
                                             : ((s & kSrcSuffix) ? suffix_g + (size_t)(s & 0x7FFFFFFFu) * kRowChunks
                                                                 : rows_g + (size_t)s * kRowChunks);
                    const int r = 16 * pw + 4 * u + rl;
                    const uint32_t dst = stage + (r >> 3) * 1024 + (r & 7) * 128 + ((jl ^ (r & 7)) << 4);
                    const int bytes = valid ? 16 : 0;
#pragma unroll
                    for (int ac = 0; ac < kRowDim / 64; ++ac) cp_async16(dst + ac * kTcColBytes, gp + 8 * ac + jl, bytes);
                }
                if (!kAll) {                                // two threads copy a row's 16 corrections
                    const uint32_t bdst = smem_base + kTcOffBias + ((par * kTcRows + (pt >> 1)) * kBiasPitch + 8 * (pt & 1)) * 4;
                    const float *bsrc = ok_pt ? bias_g + (size_t)seg_pt * kHeads + 8 * (pt & 1) : reinterpret_cast<const float *>(rows_g);
#pragma unroll
                    for (int u = 0; u < 2; ++u) cp_async16(bdst + 16 * u, bsrc + 4 * u, ok_pt ? 16 : 0);
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                tc_mark(p.trace, tr, 2);
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                tc_mark(p.trace, tr, 3);
                proxy_fence();
                mbar_arrive(bar0 + 8 * (kBarFull + par));
            }
        } else if (warp == 4) {
            // ================= tensor-core instructions, one lane =================
            if (lane == 0) {
                // S^T of the next tile and O^T of the current one are issued as soon as their inputs are
                // there, whichever comes first: waiting for the next tile's rows must not hold back the
                // PV product that frees the stage the tile after it will be copied into.
                int s_next = 0, pv_next = 0, idle = 0;
                while (pv_next < n_tiles) {
                    bool progressed = false;
                    if (s_next < n_tiles) {
                        const uint32_t g = gt0 + s_next, bpar = g & 1u;
                        if (mbar_test(bar0 + 8 * (kBarFull + bpar), g >> 1, abort_flag)
                            && (g < 2 || mbar_test(bar0 + 8 * (kBarSFree + bpar), (g >> 1) - 1, abort_flag))) {
                            tc_fence_after();
                            // one descriptor per operand; a step only moves its start-address field (a single
                            // thread issues everything, so the instructions between two MMAs are what this costs)
                            const uint64_t da = tc_desc_sw128(smem_base + bpar * kTcStageBytes, 16, 1024);
                            const uint64_t dq = tc_desc_sw128(smem_base + kTcOffQ, 16, 1024);
#pragma unroll
                            for (int ks = 0; ks < kRowDim / 16; ++ks)
                                tc_mma(tmem + 64 * bpar, da + (uint64_t)(((ks >> 2) * kTcColBytes + (ks & 3) * 32) >> 4),
                                       dq + (uint64_t)(((ks >> 2) * kTcQColBytes + (ks & 3) * 32) >> 4), idesc_s, ks > 0 ? 1u : 0u);
                            tc_commit(bar0 + 8 * (kBarSReady + bpar));
                            tc_mark(p.trace, gt0 == 0 && s_next == 2, 4);
                            ++s_next;
                            progressed = true;
                        }
                    }
                    if (pv_next < s_next) {
                        const uint32_t g = gt0 + pv_next, bpar = g & 1u;
                        if (mbar_test(bar0 + 8 * (kBarPReady + bpar), g >> 1, abort_flag)) {
                            tc_fence_after();
                            const uint64_t dv = tc_desc_sw128(smem_base + bpar * kTcStageBytes, kTcColBytes, 1024);
                            const uint64_t dp = tc_desc(smem_base + kTcOffP + bpar * 4096, 128, 1024);
                            const uint32_t first = pv_next > 0 ? 1u : 0u;
#pragma unroll
                            for (int k4 = 0; k4 < kTcRows / 16; ++k4) {
#pragma unroll
                                for (int term = 0; term < 2; ++term) {
#pragma unroll
                                    for (int mt = 0; mt < 4; ++mt)
                                        tc_mma(tmem + kTcColO + 16 * mt, dv + (uint64_t)((2 * mt * kTcColBytes + 2 * k4 * 1024) >> 4),
                                               dp + (uint64_t)((term * 2048 + k4 * 256) >> 4), idesc_o, (k4 > 0 || term > 0) ? 1u : first);
                                }
                            }
                            tc_commit(bar0 + 8 * (kBarPvDone + bpar));
                            tc_mark(p.trace, gt0 == 0 && pv_next == 2, 9);
                            ++pv_next;
                            progressed = true;
                        }
                    }
                    if (progressed) {
                        idle = 0;
                    } else if (++idle > kTcWaitLimit) {
                        *abort_flag = 1;
                        if (status != nullptr) atomicOr(status, 4);
                    }
                }
            }
        } else {
            // ================= softmax: thread (warp w, lane l < 16) owns row 16 w + l of a tile =================
            const bool has_row = lane < 16;
            const int trow = warp * 16 + lane;
            const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
            float m_ref[kHeads], l_part[kHeads];
#pragma unroll
            for (int h = 0; h < kHeads; ++h) { m_ref[h] = -CUDART_INF_F; l_part[h] = 0.f; }
            for (int i = 0; i < n_tiles; ++i) {
                const uint32_t g = gt0 + i, bpar = g & 1u;
                const int nv = min(kTcRows, s_hi - (s_lo + kTcRows * i));
                const bool tr = gt0 == 0 && i == 2 && tid == 0;
                mbar_wait(bar0 + 8 * (kBarSReady + bpar), g >> 1, abort_flag, status);
                tc_mark(p.trace, tr, 5);
                tc_fence_after();
                uint32_t sv[16];
                tc_ld16(lane_addr + 64 * bpar, sv);
                tc_fence_before();
                mbar_arrive(bar0 + 8 * (kBarSFree + bpar));
                float x[kHeads], mx[kHeads];
                const float *bias_s = reinterpret_cast<const float *>(smem + kTcOffBias) + (bpar * kTcRows + trow) * kBiasPitch;
                const bool live = has_row && trow < nv;
#pragma unroll
                for (int h = 0; h < kHeads; ++h) {
                    const float bia = (kAll || !live) ? 0.f : bias_s[h];
                    x[h] = live ? fmaf(__uint_as_float(sv[h]), p.qk_scale_log2, bia) : -CUDART_INF_F;
                    mx[h] = x[h];
                }
                // column maxima over the tile's rows: inside the warp, then across the four warps
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) {
#pragma unroll
                    for (int h = 0; h < kHeads; ++h) mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xFFFFFFFFu, mx[h], o));
                }
                if (lane == 0) {
#pragma unroll
                    for (int h = 0; h < kHeads; ++h) red_max[(bpar * 4 + warp) * 16 + h] = mx[h];
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                tc_mark(p.trace, tr, 6);
                bool grow = false;
#pragma unroll
                for (int h = 0; h < kHeads; ++h) {
                    const float *rm = red_max + bpar * 64 + h;
                    mx[h] = fmaxf(fmaxf(rm[0], rm[16]), fmaxf(rm[32], rm[48]));
                    grow = grow || mx[h] > m_ref[h] + 8.f;                   // also: first finite maximum of a head
                }
                if (grow) {                                                   // the same decision in all 128 threads
                    float alpha[kHeads];
#pragma unroll
                    for (int h = 0; h < kHeads; ++h) {
                        const float mn = fmaxf(m_ref[h], mx[h]);
                        alpha[h] = ex2(m_ref[h] - (mn == -CUDART_INF_F ? 0.f : mn));
                        m_ref[h] = mn;
                        l_part[h] *= alpha[h];
                    }
                    if (i > 0) {                                              // O^T holds the earlier tiles: scale its columns
                        mbar_wait(bar0 + 8 * (kBarPvDone + ((g - 1) & 1u)), (g - 1) >> 1, abort_flag, status);
                        tc_fence_after();
#pragma unroll
                        for (int mt = 0; mt < 4; ++mt) {
                            uint32_t ov[16];
                            tc_ld16(lane_addr + kTcColO + 16 * mt, ov);
#pragma unroll
                            for (int h = 0; h < kHeads; ++h) ov[h] = __float_as_uint(__uint_as_float(ov[h]) * alpha[h]);
                            tc_st16(lane_addr + kTcColO + 16 * mt, ov);
                        }
                        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                    }
                }
                tc_mark(p.trace, tr, 7);
                if (g >= 2) mbar_wait(bar0 + 8 * (kBarPvDone + bpar), (g >> 1) - 1, abort_flag, status);      // P^T buffer is free
                uint32_t hi_w[8], lo_w[8];
#pragma unroll
                for (int h = 0; h < kHeads; h += 2) {
                    const float u0 = m_ref[h] == -CUDART_INF_F ? 0.f : m_ref[h], u1 = m_ref[h + 1] == -CUDART_INF_F ? 0.f : m_ref[h + 1];
                    const float p0 = ex2(x[h] - u0), p1 = ex2(x[h + 1] - u1);
                    l_part[h] += p0;
                    l_part[h + 1] += p1;
                    const uint32_t hw = pack_bf16(p0, p1);
                    hi_w[h >> 1] = hw;
                    lo_w[h >> 1] = pack_bf16(p0 - bf16_lo(hw), p1 - bf16_hi(hw));
                }
                if (has_row) {
                    // P^T as an MN-major operand: element (head h, row r) at (h / 8) * 1024 + (r / 8) * 128 + (r % 8) * 16 + (h % 8) * 2
                    unsigned char *pb = smem + kTcOffP + bpar * 4096 + (trow >> 3) * 128 + (trow & 7) * 16;
                    *reinterpret_cast<uint4 *>(pb) = make_uint4(hi_w[0], hi_w[1], hi_w[2], hi_w[3]);
                    *reinterpret_cast<uint4 *>(pb + 1024) = make_uint4(hi_w[4], hi_w[5], hi_w[6], hi_w[7]);
                    *reinterpret_cast<uint4 *>(pb + 2048) = make_uint4(lo_w[0], lo_w[1], lo_w[2], lo_w[3]);
                    *reinterpret_cast<uint4 *>(pb + 3072) = make_uint4(lo_w[4], lo_w[5], lo_w[6], lo_w[7]);
                }
                proxy_fence();
                tc_fence_before();
                mbar_arrive(bar0 + 8 * (kBarPReady + bpar));
                tc_mark(p.trace, tr, 8);
                if (i == 3 && gt0 == 0 && tid == 0) tc_mark(p.trace, true, 10);
            }
            // ---- the share's partial result: (m, l) per head and O^T from tensor memory ----
            const uint32_t g_last = gt0 + n_tiles - 1;
            mbar_wait(bar0 + 8 * (kBarPvDone + (g_last & 1u)), g_last >> 1, abort_flag, status);
            tc_fence_after();
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) {
#pragma unroll
                for (int h = 0; h < kHeads; ++h) l_part[h] += __shfl_xor_sync(0xFFFFFFFFu, l_part[h], o);
            }
            if (lane == 0) {
#pragma unroll
                for (int h = 0; h < kHeads; ++h) red_sum[warp * 16 + h] = l_part[h];
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            float *slot = p.partials + (size_t)(blockIdx.x + b) * kHeads * kLatPartialStride;
            if (tid < kHeads) {
                slot[(size_t)tid * kLatPartialStride] = m_ref[tid];
                slot[(size_t)tid * kLatPartialStride + 1] = red_sum[tid] + red_sum[16 + tid] + red_sum[32 + tid] + red_sum[48 + tid];
            }
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                uint32_t ov[16];
                tc_ld16(lane_addr + kTcColO + 16 * mt, ov);
                const int dim = 128 * mt + tid;                               // tensor-memory lane = value column inside the M tile
#pragma unroll
                for (int h = 0; h < kHeads; ++h) slot[(size_t)h * kLatPartialStride + 4 + dim] = __uint_as_float(ov[h]);
            }
        }
        gt0 += (uint32_t)n_tiles;
        tc_fence_before();
        __syncthreads();                                    // the share is done: queries, P^T and tensor memory may be reused
        tc_fence_after();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcColumns));
}

}  // namespace
