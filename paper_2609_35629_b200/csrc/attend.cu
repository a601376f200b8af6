// Exact attention over a read plan (Algorithm 1, the reads and the estimator):
// every member row of every selected team enters head h's sums with weight e^{s_i} / c_g
// (applied as s_i - log c_g, so the same correction enters the mass and the value sum), every
// suffix row with weight e^{s_i}; Eq. (method-estimate).
//
// Work split, two ways (split-K by rows, never by teams; one CTA per SM):
//   static   a fixed number of CTAs per (sequence, KV head) pair. Every CTA of a pair first
//            builds the pair's read plan in shared memory from the heads' samples (pairplan.cuh;
//            the dense kernel's plan is trivial), then takes its share of the pair's rows. No
//            plan kernel, no global plan: the shortest path for few pairs (a kernel boundary or
//            a counter in global memory costs about a microsecond, the redundant build less).
//   dynamic  the rows of all pairs form one global row space cut into equal contiguous ranges;
//            plans come from a plan kernel through global memory. Best balance for many pairs.
// Inside a CTA each warp takes a contiguous run of 16-row blocks and streams them through a
// private two-slot ring in shared memory with 16-byte asynchronous copies (a whole 256-byte row
// per half warp, XOR swizzled so that ldmatrix is bank-conflict free), one block ahead of the one
// it is evaluating, together with the block's per-row head masks and corrections; completion is
// tracked with cp.async groups, so the kernel has no spin-wait.
//
// Arithmetic. The GQA group is a real MMA tile: the query heads of the KV head (at most 8)
// are the M rows of S^T = q K^T (mma.sync m16n8k16, bf16 inputs, fp32 accumulation), so one
// row of K serves every head at once; a team contributes to a head only where the head
// selected it (mask), with the head's own correction. The weights are split into two bf16
// terms (p = p_hi + p_lo) so that O^T += V^T P^T keeps fp32-level accuracy.
//
// Each CTA leaves one online-softmax partial per pair it touched; a second, small kernel merges
// every pair's partials by log-sum-exp (the split-softmax reduction). A kernel boundary costs less
// here than any counter the CTAs of one launch could meet at, and it needs no state between calls.
#include <math_constants.h>

#include "common.cuh"
#include "pairplan.cuh"

namespace santapp {

namespace {

constexpr int kWarps = 12;
constexpr int kAttendThreads = kWarps * 32;
constexpr int kBlockRows = 16;                              // rows per block (one warp, one MMA K step)
constexpr int kSlots = 2;                                   // ring slots per warp
constexpr int kRowBytes = kHeadDim * 2;                     // one bf16 row
constexpr int kTileBytes = kBlockRows * kRowBytes;          // K tile or V tile of a block
constexpr int kSlotBytes = 2 * kTileBytes;                  // K tile then V tile
constexpr int kPairMax = 512;                               // pairs whose offsets are staged at a time (dynamic split)
constexpr int kMaxAttendGrid = 512;
constexpr uint32_t kNoRow = 0xFFFFFFFFu;

// ---- primitives ----
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros instead.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
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
// D += A (16x16, row) * B (16x8, col), bf16 (or fp16) inputs, fp32 accumulation.
template <bool kHalf>
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1)
{
    if constexpr (kHalf)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// (lo, hi) -> two 16-bit elements with lo in the low half, round to nearest even.
template <bool kHalf>
__device__ __forceinline__ uint32_t pack_x2(float lo, float hi)
{
    uint32_t r;
    if constexpr (kHalf) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    else                 asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// fp16 holds nothing below 2^-24, so the weights of rows that follow a much larger score in the
// same warp's stream would vanish when they are rounded for the value product (a bounded loss: a
// warp streams at most a few thousand rows). With fp16 inputs the weights (and with them the
// running sum and the accumulators, consistently, so the factor cancels in U / Z and in every
// merge) are carried multiplied by 2^15: the largest is 32768, the smallest kept 2^-39 of the
// running maximum. bf16 has the exponent range of fp32 and needs no such shift.
template <bool kHalf> constexpr float kWeightShift = kHalf ? 15.f : 0.f;

// ---- shared memory carve-up (dynamic) ----
template <int G>
struct Smem {
    static constexpr size_t ring = 0;                                           // [warps][kSlots][kSlotBytes]
    static constexpr size_t ring_bytes = (size_t)kWarps * kSlots * kSlotBytes;
    static constexpr size_t logc_tab = ring + ring_bytes;                       // float [warps][kSlots][16][8]
    static constexpr size_t mask_tab = logc_tab + (size_t)kWarps * kSlots * kBlockRows * kMaxGroup * 4;
    static constexpr size_t seg_prefix = mask_tab + kWarps * kSlots * kBlockRows;   // int [kSegMax + 1]
    static constexpr size_t seg_row = seg_prefix + (kSegMax + 3) * 4;           // int [kSegMax]
    static constexpr size_t seg_mask = seg_row + (kSegMax + 3) * 4;             // uint [kSegMax]
    static constexpr size_t pair_prefix = (seg_mask + (kSegMax + 3) * 4 + 15) / 16 * 16;   // int64 [kPairMax + 1]
    static constexpr size_t pair_nseg = pair_prefix + (kPairMax + 1) * 8;       // int [kPairMax]
    static constexpr size_t misc = pair_nseg + kPairMax * 4;                    // flags, then scan scratch [40]
    static constexpr size_t total = misc + 64 + 160;
    // aliases of the ring: plan scratch before a pair's rows are streamed, merge scratch after
    static_assert(sizeof(PlanScratch) <= ring_bytes, "plan scratch must fit in the ring");
    static constexpr int red_pitch = kHeadDim + 4;                              // floats per (warp, head) row: the 4 extra
                                                                                //   spread the heads of a store over the banks
    static constexpr size_t red_acc = ring;                                     // float [warps][G][red_pitch]
    static constexpr size_t red_m = red_acc + (size_t)kWarps * G * red_pitch * 4;  // float [warps][G]
    static constexpr size_t red_l = red_m + (size_t)kWarps * G * 4;
    static_assert(red_l + (size_t)kWarps * G * 4 <= ring_bytes, "merge scratch must fit in the ring");
    static_assert(total <= 227 * 1024, "shared memory budget");
};

template <int G, bool kAll, bool kStatic, bool kHalf>
__global__ void __launch_bounds__(kAttendThreads, 1)
attend_kernel(AttendParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    using S = Smem<G>;
    int *seg_prefix = reinterpret_cast<int *>(smem + S::seg_prefix);
    int *seg_row = reinterpret_cast<int *>(smem + S::seg_row);
    uint32_t *seg_mask = reinterpret_cast<uint32_t *>(smem + S::seg_mask);
    int64_t *pair_prefix = reinterpret_cast<int64_t *>(smem + S::pair_prefix);
    int *pair_nseg = reinterpret_cast<int *>(smem + S::pair_nseg);
    int *misc = reinterpret_cast<int *>(smem + S::misc);
    int *scan_scratch = misc + 16;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;                 // MMA fragment coordinates
    const int hw = lane >> 4, chunk = lane & 15;           // copy coordinates: row parity, 16-byte chunk
    trace_mark(p.in.trace, 3, 0);
    const uint32_t ring_w = smem_u32(smem + S::ring) + (uint32_t)warp * kSlots * kSlotBytes;
    float *logc_w = reinterpret_cast<float *>(smem + S::logc_tab) + warp * kSlots * kBlockRows * kMaxGroup;
    unsigned char *mask_w = smem + S::mask_tab + warp * kSlots * kBlockRows;
    const int cap = p.plan.seg_cap;

    // ---- which (pair, row range) spans this CTA works on ----
    int pair, sub = 0;
    int pair_base = 0;                                     // first pair of the staged window (dynamic split)
    auto stage_pairs = [&](int base) {                     // all threads: stage pairs [base, base + kPairMax]
        __syncthreads();
        const int n = min(kPairMax, p.n_pairs - base);
        for (int i = tid; i <= n; i += kAttendThreads) pair_prefix[i] = p.plan.pair_row_prefix[base + i];
        for (int i = tid; i < n; i += kAttendThreads) pair_nseg[i] = p.plan.pair_nseg[base + i];
        __syncthreads();
        pair_base = base;
    };
    // Batches of at most kPairMax pairs: the row prefix over the pairs is summed here from the
    // pairs' row counts (thread t owns pairs 2t and 2t + 1); block 0 leaves it in global memory
    // for the merge kernel.
    auto stage_all_pairs = [&]() {
        static_assert(2 * kAttendThreads >= kPairMax, "two pairs per thread");
        const int i0 = 2 * tid, i1 = 2 * tid + 1;
        const int v0 = i0 < p.n_pairs ? __ldcg(p.plan.pair_rows + i0) : 0;
        const int v1 = i1 < p.n_pairs ? __ldcg(p.plan.pair_rows + i1) : 0;
        if (i0 < p.n_pairs) pair_nseg[i0] = __ldcg(p.plan.pair_nseg + i0);
        if (i1 < p.n_pairs) pair_nseg[i1] = __ldcg(p.plan.pair_nseg + i1);
        int total;
        const int excl = block_exclusive_scan(v0 + v1, scan_scratch, total);
        if (i0 <= p.n_pairs) pair_prefix[i0] = excl;
        if (i1 <= p.n_pairs) pair_prefix[i1] = excl + v0;
        if (blockIdx.x == 0) {
            if (i0 <= p.n_pairs) p.plan.pair_row_prefix[i0] = excl;
            if (i1 <= p.n_pairs) p.plan.pair_row_prefix[i1] = excl + v0;
        }
        __syncthreads();
        pair_base = 0;
    };
    uint32_t r0 = 0, r1 = 0;                               // dynamic split: this item's range of the padded row line (< 2^32)
    int item = blockIdx.x;                                 // dynamic split: fixed range (< gridDim.x) or tail chunk
    int next_chunk = 0;                                    // thread 0: the tail chunk taken from the counter for later
    RangeSplit &sp = *reinterpret_cast<RangeSplit *>(misc + 8);   // the same in every thread: kept in shared memory
    const bool windowed = p.n_pairs > kPairMax;
    if (kStatic) {
        pair = blockIdx.x / p.ctas_per_pair;
        sub = blockIdx.x - pair * p.ctas_per_pair;
        if (pair >= p.n_pairs) return;
    } else {
        // pair_prefix / pair_nseg hold a window of kPairMax pairs starting at pair_base; batches of up
        // to kPairMax pairs are staged whole, before anything else is waited for
        if (!windowed) stage_all_pairs();
        const int64_t all_rows = windowed ? p.plan.pair_row_prefix[p.n_pairs] : pair_prefix[p.n_pairs];
        // Rows of all pairs laid end to end, with a gap of span_penalty_rows after every pair: a CTA
        // whose range crosses from one pair into the next pays the fixed cost of a second span
        // (tables, pipeline refill, merge) out of its row budget, so ranges cost about equal time.
        __syncthreads();
        if (tid == 0) sp = make_range_split(all_rows, p.n_pairs, p.span_penalty_rows, p.min_rows_per_cta, (int)gridDim.x);
        __syncthreads();
    }

  for (;;) {                                               // items of this block (one, for the fixed split)
    if (!kStatic) {
        // the next tail chunk is asked for now and looked at when this item is done
        if (tid == 0 && sp.n_tail > 0) next_chunk = atomicAdd(p.plan.tail_counter, 1);
        {
            const bool fixed = item < (int)gridDim.x;
            const uint64_t lo64 = fixed ? (uint64_t)item * sp.fixed_rows
                                        : (uint64_t)sp.fixed_end + (uint64_t)(item - (int)gridDim.x) * sp.chunk_rows;
            const uint64_t end = fixed ? sp.fixed_end : sp.total;
            const uint64_t hi64 = min(lo64 + (fixed ? sp.fixed_rows : sp.chunk_rows), end);
            if (lo64 >= hi64) goto item_done;
            r0 = (uint32_t)lo64;
            r1 = (uint32_t)hi64;
        }
        // first pair of the range: the largest i with prefix[i] + penalty * i <= r0
        int lo = 0, hi = p.n_pairs;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            const int64_t start = (windowed ? p.plan.pair_row_prefix[mid] : pair_prefix[mid])
                                  + (int64_t)p.span_penalty_rows * mid;
            if (start <= (int64_t)r0) lo = mid; else hi = mid;
        }
        if (windowed) stage_pairs(lo);
        pair = lo;
    }

    while (true) {
        int a, bnd, nseg, slot_id;
        uint32_t pb = 0, pe = 0;
        const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;
        const float *g_logc = p.plan.seg_logc + (size_t)pair * cap * kMaxGroup;
        // A fragments of q for the 8 k-steps: head g (zero rows for g >= G and for M rows 8..15);
        // requested first, so that they arrive while the plan is being set up
        uint32_t qa[8][2];
        {
            const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
                p.q + ((size_t)b * p.bv.n_q + (size_t)j * G + (g < G ? g : 0)) * kHeadDim);
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                qa[s][0] = g < G ? __ldg(qrow + 8 * s + c) : 0u;
                qa[s][1] = g < G ? __ldg(qrow + 8 * s + 4 + c) : 0u;
            }
        }

        if (kStatic) {
            int rows;
            if (!kAll) {
                PlanScratch &scratch = *reinterpret_cast<PlanScratch *>(smem + S::ring);
                build_pair_plan<kAttendThreads>(p.in, pair, p.max_words, scratch, seg_prefix, seg_row, seg_mask,
                                                p.plan.seg_logc + (size_t)pair * cap * kMaxGroup, nseg, rows, sub == 0);
            } else {
                __syncthreads();
                if (tid == 0) {
                    const int64_t row0 = p.bv.seq_row_off[b];
                    const int N = (int)(p.bv.seq_row_off[b + 1] - row0);
                    int t = 0;
                    if (p.in.suffix_len != nullptr && p.in.suffix_cap > 0)
                        t = max(0, min(p.in.suffix_len[b], p.in.suffix_cap));
                    const uint32_t all_heads = (1u << G) - 1u;
                    seg_prefix[0] = 0;
                    seg_row[0] = (int32_t)row0;
                    seg_mask[0] = all_heads;
                    int ns = 1, rw = N;
                    if (t > 0) {
                        seg_prefix[1] = rw;
                        seg_row[1] = pair * p.in.suffix_cap;
                        seg_mask[1] = all_heads | kSrcSuffix;
                        rw += t;
                        ns = 2;
                    }
                    seg_prefix[ns] = rw;
                    misc[2] = ns;
                    misc[3] = rw;
                }
                __syncthreads();
                nseg = misc[2];
                rows = misc[3];
            }
            const int per_cta = max((rows + p.ctas_per_pair - 1) / p.ctas_per_pair, p.min_rows_per_cta);
            a = sub * per_cta;
            bnd = min(a + per_cta, rows);
            slot_id = pair * p.ctas_per_pair + sub;
            if (a >= rows) {                               // more CTAs than this pair needs: an empty partial
                if (tid < G) {
                    float *part = p.partials + ((size_t)slot_id * G + tid) * kPartialStride;
                    part[0] = -CUDART_INF_F;
                    part[1] = 0.f;
                }
                return;
            }
        } else {
            // this pair's rows occupy [pb, pe) of the padded row line
            if (pair - pair_base >= kPairMax) stage_pairs(pair);           // walked off the staged window
            pb = (uint32_t)(pair_prefix[pair - pair_base] + (int64_t)p.span_penalty_rows * pair);
            pe = pb + (uint32_t)(pair_prefix[pair - pair_base + 1] - pair_prefix[pair - pair_base]);
            a = (int)(max(r0, pb) - pb);
            bnd = (int)(min(r1, pe) - pb);
            if (a >= bnd) {                                // the range starts in the gap behind this pair
                r0 = pe + p.span_penalty_rows;
                if (r0 >= r1 || pair + 1 >= p.n_pairs) goto item_done;
                ++pair;
                continue;
            }
            nseg = pair_nseg[pair - pair_base];
            slot_id = item + pair;                         // item c's partial of pair i lives in slot c + i
            __syncthreads();                               // the previous span is done with the tables
            // one round trip: every load is issued before the first store
            const int32_t *g_prefix = p.plan.seg_prefix + (size_t)pair * (cap + 1);
            const int32_t *g_row = p.plan.seg_row + (size_t)pair * cap;
            const uint32_t *g_mask = p.plan.seg_mask + (size_t)pair * cap;
            for (int i0 = 0; i0 <= nseg; i0 += kAttendThreads) {
                const int i = i0 + tid;
                int v_prefix = 0, v_row = 0;
                uint32_t v_mask = 0u;
                if (i <= nseg) v_prefix = g_prefix[i];
                if (i < nseg) { v_row = g_row[i]; v_mask = g_mask[i]; }
                if (i <= nseg) seg_prefix[i] = v_prefix;
                if (i < nseg) { seg_row[i] = v_row; seg_mask[i] = v_mask; }
            }
        }
        __syncthreads();
        trace_mark(p.in.trace, 3, 1);

        const unsigned char *k_plane = reinterpret_cast<const unsigned char *>(p.k_packed)
                                       + (size_t)j * p.bv.rows_total * kRowBytes;
        const unsigned char *v_plane = reinterpret_cast<const unsigned char *>(p.v_packed)
                                       + (size_t)j * p.bv.rows_total * kRowBytes;
        const unsigned char *k_suf = reinterpret_cast<const unsigned char *>(p.k_suffix);
        const unsigned char *v_suf = reinterpret_cast<const unsigned char *>(p.v_suffix);

        // this warp's contiguous run of blocks: [blk0, blk0 + nb)
        const int n_blk = (bnd - a + kBlockRows - 1) / kBlockRows;
        const int per = n_blk / kWarps, rem = n_blk - per * kWarps;
        const int nb = per + (warp < rem ? 1 : 0);
        const int blk0 = warp * per + min(warp, rem);

        // segment cursor of row (lane & 15) of the current block; rows advance by 16 per block
        int cur = 0;
        if (nb > 0) {
            const int pos = min(a + blk0 * kBlockRows + (lane & 15), bnd - 1);
            int lo = 0, hi = nseg;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (seg_prefix[mid] <= pos) lo = mid; else hi = mid;
            }
            cur = lo;
        }

        // Issue the copies of this warp's block i (if it exists) into ring slot i % kSlots and
        // close a group: K and V rows, and for each row its head mask and corrections.
        auto issue = [&](int i) {
            if (i < nb) {
                const int slot = i % kSlots;
                const int pos0 = a + (blk0 + i) * kBlockRows;
                const int r = lane & 15;
                const int pos = pos0 + r;
                uint32_t info = kNoRow;                    // row index in its buffer, bit 31: suffix buffer
                if (pos < bnd) {
                    while (pos >= seg_prefix[cur + 1]) ++cur;
                    const uint32_t mk = seg_mask[cur];
                    info = (uint32_t)(seg_row[cur] + (pos - seg_prefix[cur])) | (mk & kSrcSuffix);
                    if (lane < 16) {
                        mask_w[slot * kBlockRows + r] = (unsigned char)(mk & 0xFFu);
                        if (!kAll) {
                            const uint32_t dst = smem_u32(logc_w + (slot * kBlockRows + r) * kMaxGroup);
                            cp_async16(dst, g_logc + (size_t)cur * kMaxGroup, 16u);
                            cp_async16(dst + 16, g_logc + (size_t)cur * kMaxGroup + 4, 16u);
                        }
                    }
                } else if (lane < 16) {
                    mask_w[slot * kBlockRows + r] = 0;
                }
                const uint32_t k_dst = ring_w + slot * kSlotBytes;
#pragma unroll
                for (int piece = 0; piece < kBlockRows / 2; ++piece) {
                    const int row = 2 * piece + hw;
                    const uint32_t ri = __shfl_sync(0xFFFFFFFFu, info, row);
                    const bool valid = ri != kNoRow;
                    const size_t off = (size_t)(ri & 0x7FFFFFFFu) * kRowBytes + chunk * 16;
                    const bool suf = (ri & kSrcSuffix) != 0u;
                    const unsigned char *ks = valid ? (suf ? k_suf : k_plane) + off : k_plane;
                    const unsigned char *vs = valid ? (suf ? v_suf : v_plane) + off : v_plane;
                    const uint32_t dst = k_dst + row * kRowBytes + ((chunk ^ (row & 7)) << 4);
                    cp_async16(dst, ks, valid ? 16u : 0u);
                    cp_async16(dst + kTileBytes, vs, valid ? 16u : 0u);
                }
            }
            cp_async_commit();
        };

        // online-softmax state of head g (replicated over the quad) and O^T fragments:
        // o[t][r]: d = 16 t + g + 8 (r >> 1), head = 2 c + (r & 1)
        float m_run = -CUDART_INF_F, l_run = 0.f;
        float o[8][4];
#pragma unroll
        for (int t = 0; t < 8; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }
        const float qk = p.qk_scale_log2;

        issue(0);
        for (int i = 0; i < nb; ++i) {
            issue(i + 1);
            cp_async_wait_group<1>();                      // block i has landed (this lane's copies)
            __syncwarp();                                  // ... and every other lane's
            if (i == 0) trace_mark(p.in.trace, 3, 2);
            const int slot = i % kSlots;
            const uint32_t k_addr = ring_w + slot * kSlotBytes;
            const uint32_t v_addr = k_addr + kTileBytes;

            // the four (row, head g) entries of this thread: rows 2c, 2c+1, 8+2c, 9+2c
            bool on[4];
            float lc[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int r = 2 * c + (e & 1) + 8 * (e >> 1);
                const uint32_t mk = mask_w[slot * kBlockRows + r];
                on[e] = (g < G) && ((mk >> g) & 1u);
                lc[e] = (!kAll && on[e]) ? logc_w[(slot * kBlockRows + r) * kMaxGroup + g] : 0.f;
            }

            // S^T = q K^T for the two 8-row groups, two accumulators each to shorten the chain
            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
            float s2[4] = {0.f, 0.f, 0.f, 0.f}, s3[4] = {0.f, 0.f, 0.f, 0.f};
            {
                const int lrow = lane & 7, lmat = lane >> 3;
#pragma unroll
                for (int sp = 0; sp < 4; ++sp) {
                    uint32_t kb0[4], kb1[4];
                    const int ch = 4 * sp + lmat;
                    ldmatrix_x4(kb0, k_addr + lrow * kRowBytes + ((ch ^ lrow) << 4));
                    ldmatrix_x4(kb1, k_addr + (8 + lrow) * kRowBytes + ((ch ^ lrow) << 4));
                    mma_16816<kHalf>(s0, qa[2 * sp][0], 0u, qa[2 * sp][1], 0u, kb0[0], kb0[1]);
                    mma_16816<kHalf>(s1, qa[2 * sp][0], 0u, qa[2 * sp][1], 0u, kb1[0], kb1[1]);
                    mma_16816<kHalf>(s2, qa[2 * sp + 1][0], 0u, qa[2 * sp + 1][1], 0u, kb0[2], kb0[3]);
                    mma_16816<kHalf>(s3, qa[2 * sp + 1][0], 0u, qa[2 * sp + 1][1], 0u, kb1[2], kb1[3]);
                }
            }
            float sc[4];
            sc[0] = on[0] ? fmaf(s0[0] + s2[0], qk, -lc[0]) : -CUDART_INF_F;
            sc[1] = on[1] ? fmaf(s0[1] + s2[1], qk, -lc[1]) : -CUDART_INF_F;
            sc[2] = on[2] ? fmaf(s1[0] + s3[0], qk, -lc[2]) : -CUDART_INF_F;
            sc[3] = on[3] ? fmaf(s1[1] + s3[1], qk, -lc[3]) : -CUDART_INF_F;
            float mloc = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
            mloc = fmaxf(mloc, __shfl_xor_sync(0xFFFFFFFFu, mloc, 1));
            mloc = fmaxf(mloc, __shfl_xor_sync(0xFFFFFFFFu, mloc, 2));
            const float m_new = fmaxf(m_run, mloc);
            const bool grew = m_new > m_run;
            if (__any_sync(0xFFFFFFFFu, grew)) {
                const float f = grew ? exp2f(m_run - m_new) : 1.f;              // exp2f(-inf) = 0 on first rows
                l_run *= f;
                const float fe = __shfl_sync(0xFFFFFFFFu, f, 8 * c);            // head 2c lives in lanes 8c..8c+3
                const float fo = __shfl_sync(0xFFFFFFFFu, f, 8 * c + 4);        // head 2c+1
#pragma unroll
                for (int t = 0; t < 8; ++t) { o[t][0] *= fe; o[t][1] *= fo; o[t][2] *= fe; o[t][3] *= fo; }
                m_run = m_new;
            }
            float pw[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) pw[e] = on[e] ? exp2f(sc[e] - m_run + kWeightShift<kHalf>) : 0.f;
            l_run += (pw[0] + pw[1]) + (pw[2] + pw[3]);
            // P^T as B fragments, split in two bf16 terms
            const uint32_t ph0 = pack_x2<kHalf>(pw[0], pw[1]), ph1 = pack_x2<kHalf>(pw[2], pw[3]);
            const uint32_t pl0 = pack_x2<kHalf>(pw[0] - elem_lo<kHalf>(ph0), pw[1] - elem_hi<kHalf>(ph0));
            const uint32_t pl1 = pack_x2<kHalf>(pw[2] - elem_lo<kHalf>(ph1), pw[3] - elem_hi<kHalf>(ph1));

            // O^T += V^T P^T
            {
                const int lrow = lane & 7, lmat = lane >> 3;
                const int vrow = (lmat >> 1) * 8 + lrow;
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    uint32_t va[4];
                    const int ch = 2 * t + (lmat & 1);
                    ldmatrix_x4_trans(va, v_addr + vrow * kRowBytes + ((ch ^ lrow) << 4));
                    mma_16816<kHalf>(o[t], va[0], va[1], va[2], va[3], ph0, ph1);
                    mma_16816<kHalf>(o[t], va[0], va[1], va[2], va[3], pl0, pl1);
                }
            }
            __syncwarp();                                  // the slot may be refilled by the next issue
        }
        cp_async_wait_group<0>();
        __syncthreads();                                   // every block of the span is consumed
        trace_mark(p.in.trace, 3, 3);

        // ---- merge the warps into one partial (the ring is free: reuse it) ----
        float(*red_acc)[G][S::red_pitch] = reinterpret_cast<float(*)[G][S::red_pitch]>(smem + S::red_acc);
        float(*red_m)[G] = reinterpret_cast<float(*)[G]>(smem + S::red_m);
        float(*red_l)[G] = reinterpret_cast<float(*)[G]>(smem + S::red_l);
        l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 1);
        l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 2);
        if (c == 0 && g < G) { red_m[warp][g] = m_run; red_l[warp][g] = l_run; }
        if (nb > 0) {
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
        // thread (h, lane) merges four output columns of head h over the warps
        float *part = p.partials + (size_t)slot_id * G * kPartialStride;
        if (warp < G) {
            const int h = warp;
            float mh = -CUDART_INF_F;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) mh = fmaxf(mh, red_m[w][h]);
            float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
            float den = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float mw = red_m[w][h];
                if (mw > -CUDART_INF_F) {                  // warps without rows for this head left no data
                    const float f = exp2f(mw - mh);
                    const float4 v = *reinterpret_cast<const float4 *>(&red_acc[w][h][4 * lane]);
                    num.x = fmaf(f, v.x, num.x);
                    num.y = fmaf(f, v.y, num.y);
                    num.z = fmaf(f, v.z, num.z);
                    num.w = fmaf(f, v.w, num.w);
                    den = fmaf(f, red_l[w][h], den);
                }
            }
            *reinterpret_cast<float4 *>(part + h * kPartialStride + 4 + 4 * lane) = num;
            if (lane == 0) { part[h * kPartialStride] = mh; part[h * kPartialStride + 1] = den; }
        }

        // ---- next span ----
        if (kStatic) {
            trace_mark(p.in.trace, 3, 5);
            return;                                        // one span per CTA
        } else {
            if (pb + bnd < pe) goto item_done;             // the range ended inside this pair
            r0 = pe + p.span_penalty_rows;                 // first row of the next pair
            if (r0 >= r1 || pair + 1 >= p.n_pairs) goto item_done;
            ++pair;
        }
    }
item_done:
    if (kStatic) return;
    if (sp.n_tail == 0) return;
    __syncthreads();                                       // also: every warp is done with the previous span's scratch
    if (tid == 0) misc[5] = next_chunk;
    __syncthreads();
    if (misc[5] >= sp.n_tail) {
        // Out of chunks: the block leaves. The last block to leave resets both counters, so that the
        // kernel can be launched again on the same plans.
        if (tid == 0) {
            const int left = atomicAdd(p.plan.tail_counter + 1, 1);
            if (left == (int)gridDim.x - 1) {
                p.plan.tail_counter[0] = 0;
                p.plan.tail_counter[1] = 0;
            }
        }
        return;
    }
    item = (int)gridDim.x + misc[5];
  }
}

// Log-sum-exp merge of a pair's partials (the split-softmax reduction): one block per (query head
// of the group, pair). Thread (part, lane) takes the partials part, part + kParts, ...
// (at most kDepth of them in flight at once) for four output columns. Every step is laid out
// for a short dependent chain: all loads first, one block-wide maximum, weights relative to it
// (independent of each other), sums across the parts by the first four warps.
template <int kParts, bool kStatic>
__global__ void __launch_bounds__(kParts * 32)
merge_kernel(AttendParams p, int attend_grid)
{
    __shared__ float red_m[kParts], red_l[kParts];
    __shared__ __align__(16) float red_acc[kParts][kHeadDim];
    const int G = p.bv.group;
    const int h = blockIdx.x, pair = blockIdx.y;
    const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;
    const int part = threadIdx.x >> 5, lane = threadIdx.x & 31;
    trace_mark(p.in.trace, 4, 0);
    // the pair's partials: slots [first_slot, first_slot + n_fixed), then [tail_slot, tail_slot + n - n_fixed)
    int first_slot, n, n_fixed, tail_slot = 0;
    if (kStatic) {
        first_slot = pair * p.ctas_per_pair;
        n = n_fixed = p.ctas_per_pair;
    } else {
        // the attention kernel's split: rows of all pairs end to end with a gap behind each; item c
        // (fixed range or tail chunk) left its partial of pair i in slot c + i
        const int64_t pre0 = p.plan.pair_row_prefix[pair], pre1 = p.plan.pair_row_prefix[pair + 1];
        const RangeSplit sp = make_range_split(p.plan.pair_row_prefix[p.n_pairs], p.n_pairs, p.span_penalty_rows,
                                               p.min_rows_per_cta, attend_grid);
        const uint32_t pb = (uint32_t)(pre0 + (int64_t)p.span_penalty_rows * pair);
        const uint32_t pe = pb + (uint32_t)(pre1 - pre0);
        n_fixed = 0;
        first_slot = pair;
        if (pe > pb && pb < sp.fixed_end) {
            const int c_lo = (int)(pb / sp.fixed_rows), c_hi = (int)((min(pe, sp.fixed_end) - 1u) / sp.fixed_rows);
            first_slot = c_lo + pair;
            n_fixed = c_hi - c_lo + 1;
        }
        n = n_fixed;
        if (pe > pb && pe > sp.fixed_end) {
            const int j_lo = (int)((max(pb, sp.fixed_end) - sp.fixed_end) / sp.chunk_rows);
            const int j_hi = (int)((pe - 1u - sp.fixed_end) / sp.chunk_rows);
            tail_slot = attend_grid + j_lo + pair;
            n += j_hi - j_lo + 1;
        }
    }
    const size_t stride = (size_t)G * kPartialStride;
    const float *base = p.partials + (size_t)h * kPartialStride;
    auto slot_of = [&](int i) { return (size_t)(i < n_fixed ? first_slot + i : tail_slot + (i - n_fixed)); };
    constexpr int kDepth = 4;                              // partials a thread has in flight: one round trip for n <= 4 kParts
    float m_run = -CUDART_INF_F, l_run = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i0 = part; i0 < n; i0 += kParts * kDepth) {   // one trip unless n > kDepth * kParts
        float2 ml[kDepth];
        float4 v[kDepth];
#pragma unroll
        for (int u = 0; u < kDepth; ++u) {
            const int i = i0 + u * kParts;
            ml[u] = make_float2(-CUDART_INF_F, 0.f);
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < n) {
                ml[u] = __ldcg(reinterpret_cast<const float2 *>(base + slot_of(i) * stride));
                v[u] = __ldcg(reinterpret_cast<const float4 *>(base + slot_of(i) * stride + 4) + lane);
            }
        }
        float m_new = m_run;
#pragma unroll
        for (int u = 0; u < kDepth; ++u) m_new = fmaxf(m_new, ml[u].x);
        if (m_new > -CUDART_INF_F) {
            const float f = exp2f(m_run - m_new);          // 0 on the first trip
            acc.x *= f; acc.y *= f; acc.z *= f; acc.w *= f;
            l_run *= f;
#pragma unroll
            for (int u = 0; u < kDepth; ++u) {
                // a partial without rows for this head (m = -inf) holds no data
                const float w = ml[u].x > -CUDART_INF_F ? exp2f(ml[u].x - m_new) : 0.f;
                acc.x = fmaf(w, ml[u].x > -CUDART_INF_F ? v[u].x : 0.f, acc.x);
                acc.y = fmaf(w, ml[u].x > -CUDART_INF_F ? v[u].y : 0.f, acc.y);
                acc.z = fmaf(w, ml[u].x > -CUDART_INF_F ? v[u].z : 0.f, acc.z);
                acc.w = fmaf(w, ml[u].x > -CUDART_INF_F ? v[u].w : 0.f, acc.w);
                l_run = fmaf(w, ml[u].y, l_run);
            }
            m_run = m_new;
        }
    }
    if (lane == 0) red_m[part] = m_run;
    __syncthreads();
    float m_all = -CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < kParts; ++i) m_all = fmaxf(m_all, red_m[i]);
    const float f = m_run > -CUDART_INF_F ? exp2f(m_run - m_all) : 0.f;
    *reinterpret_cast<float4 *>(&red_acc[part][4 * lane]) = make_float4(acc.x * f, acc.y * f, acc.z * f, acc.w * f);
    if (lane == 0) red_l[part] = l_run * f;
    __syncthreads();
    if (threadIdx.x < kHeadDim) {
        const int d = threadIdx.x;
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int i = 0; i < kParts; ++i) { num += red_acc[i][d]; den += red_l[i]; }
        const float ov = num / den;
        p.out[((size_t)b * p.bv.n_q + (size_t)j * G + h) * kHeadDim + d] = ov;
        if (p.status && !isfinite(ov)) atomicOr(p.status, 1);
    }
    trace_mark(p.in.trace, 4, 1);
}

template <int G, bool kHalf>
cudaError_t launch_attend_g(const AttendParams &p, bool all_heads, bool static_split, int grid, cudaStream_t s)
{
    const size_t smem = Smem<G>::total;
    static std::atomic<unsigned long long> done[4];
    const void *fns[4] = {(const void *)attend_kernel<G, true, true, kHalf>, (const void *)attend_kernel<G, true, false, kHalf>,
                          (const void *)attend_kernel<G, false, true, kHalf>, (const void *)attend_kernel<G, false, false, kHalf>};
    const int which = (all_heads ? 0 : 2) + (static_split ? 0 : 1);
    cudaError_t err = ensure_dynamic_smem(fns[which], (int)smem, done[which]);
    if (err != cudaSuccess) return err;
    if (all_heads) {
        if (static_split) return launch_kernel(attend_kernel<G, true, true, kHalf>, dim3(grid), dim3(kAttendThreads), smem, s, p);
        return launch_kernel(attend_kernel<G, true, false, kHalf>, dim3(grid), dim3(kAttendThreads), smem, s, p);
    }
    if (static_split) return launch_kernel(attend_kernel<G, false, true, kHalf>, dim3(grid), dim3(kAttendThreads), smem, s, p);
    return launch_kernel(attend_kernel<G, false, false, kHalf>, dim3(grid), dim3(kAttendThreads), smem, s, p);
}

}  // namespace

int attend_grid_size()
{
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms > kMaxAttendGrid ? kMaxAttendGrid : sms;
}

int attend_max_segments() { return kSegMax; }
int attend_max_pairs() { return 65535; }                   // a grid dimension of the merge kernel
int attend_pairs_staged() { return kPairMax; }

cudaError_t launch_merge(const AttendParams &p, bool static_split, int attend_grid, cudaStream_t s)
{
    // few pairs: many partials each (16 warps share them); many pairs: a handful each
    const dim3 blocks(p.bv.group, p.n_pairs);
    const bool wide = static_split || p.n_pairs * 8 <= attend_grid;
    if (static_split) return launch_kernel(merge_kernel<16, true>, blocks, dim3(16 * 32), 0, s, p, attend_grid);
    if (wide) return launch_kernel(merge_kernel<16, false>, blocks, dim3(16 * 32), 0, s, p, attend_grid);
    return launch_kernel(merge_kernel<4, false>, blocks, dim3(4 * 32), 0, s, p, attend_grid);
}

cudaError_t launch_attend(const AttendParams &p, bool all_heads, bool static_split, int grid, cudaStream_t s)
{
    switch (p.bv.group) {
        case 1: return p.bv.elem ? launch_attend_g<1, true>(p, all_heads, static_split, grid, s)
                                 : launch_attend_g<1, false>(p, all_heads, static_split, grid, s);
        case 2: return p.bv.elem ? launch_attend_g<2, true>(p, all_heads, static_split, grid, s)
                                 : launch_attend_g<2, false>(p, all_heads, static_split, grid, s);
        case 3: return p.bv.elem ? launch_attend_g<3, true>(p, all_heads, static_split, grid, s)
                                 : launch_attend_g<3, false>(p, all_heads, static_split, grid, s);
        case 4: return p.bv.elem ? launch_attend_g<4, true>(p, all_heads, static_split, grid, s)
                                 : launch_attend_g<4, false>(p, all_heads, static_split, grid, s);
        case 5: return p.bv.elem ? launch_attend_g<5, true>(p, all_heads, static_split, grid, s)
                                 : launch_attend_g<5, false>(p, all_heads, static_split, grid, s);
        case 6: return p.bv.elem ? launch_attend_g<6, true>(p, all_heads, static_split, grid, s)
                                 : launch_attend_g<6, false>(p, all_heads, static_split, grid, s);
        case 7: return p.bv.elem ? launch_attend_g<7, true>(p, all_heads, static_split, grid, s)
                                 : launch_attend_g<7, false>(p, all_heads, static_split, grid, s);
        case 8: return p.bv.elem ? launch_attend_g<8, true>(p, all_heads, static_split, grid, s)
                                 : launch_attend_g<8, false>(p, all_heads, static_split, grid, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace santapp
