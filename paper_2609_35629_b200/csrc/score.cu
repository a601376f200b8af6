// Representative scoring for SANTA++ decode attention (Algorithm 1, routing logits and their
// Gumbel perturbation), in fp32 on tensor cores:
//   Y32_{h,g} = log n_g + q_h . l_g * scale + G_{h,g}          (Eq. method-routing plus noise)
// for every query head h of a KV head and every team g, one representative key l_g per team.
// These scores only choose which teams are re-evaluated exactly (see pairplan.cuh); the sample
// itself is decided in fp64 there.
//
// The GQA group is the M tile of S^T = q K^T (mma.sync m16n8k16, bf16 inputs, fp32
// accumulation). A lane feeds the tensor core 16-byte pieces of the representative keys exactly
// as they lie in memory: the contraction index is permuted consistently on both operands, so
// no transpose is needed. Small grids load the pieces straight from global memory; large grids
// stream whole tiles (16 keys = one contiguous 4 KB run) into shared memory with bulk
// asynchronous copies that complete on mbarriers, three tiles ahead.
#include "common.cuh"

namespace santapp {

namespace {

constexpr int kScoreThreads = 256;
constexpr int kScoreTeamsPerWarp = 16;
constexpr int kScoreTeamsPerCta = kScoreTeamsPerWarp * (kScoreThreads / 32);

template <bool kHalf>
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    // A rows 8..15 are zero (a1 = a3 = 0): only heads 0..7 exist
    if constexpr (kHalf)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                     "{%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Bulk asynchronous copy (the TMA engine's untiled form) of a contiguous run of bytes into shared
// memory, completion counted in bytes on an mbarrier; addresses and size are multiples of 16.
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_copy_to_shared(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

constexpr int kScoreStages = 3;                                 // tiles in flight per warp (pipelined variant)
constexpr int kScoreKeyRingBytes = kScoreStages * (kScoreThreads / 32) * 4096;
constexpr int kScoreCsrRingBytes = kScoreStages * (kScoreThreads / 32) * 128;                       // row offsets
constexpr int kSeqTableCap = 2048;                              // sequences whose first tile slot is kept in shared memory
constexpr int kScoreSeqTableBytes = ((kSeqTableCap + 1) * 4 + 15) / 16 * 16;
constexpr int kScoreBarrierBytes = kScoreStages * (kScoreThreads / 32) * 8;                         // one mbarrier per (warp, stage)
constexpr int kScoreRingBytes = kScoreKeyRingBytes + kScoreCsrRingBytes + kScoreSeqTableBytes + kScoreBarrierBytes;
constexpr int kScoreWaitPolls = 1 << 22;                        // bound on the polls of one mbarrier wait

// Gumbel(0,1) in fp32 from a 32-bit word: u = (x + 0.5) / 2^32, G = -log(-log u), to an absolute
// error well inside the additive term of the guard (see score_guard in pairplan.cuh).
// Lower half of the range (u <= 1/2): -log u >= 0.69 from the fast logarithm (3 ulp there).
// Upper half: u = 1 - z with z = (2^32 - x - 0.5) / 2^32 in (0, 1/2]; -log(1 - z) from four series
// terms when z < 2^-6 (relative truncation z^4 / 5 < 1.2e-8), else from the fast logarithm, whose
// absolute error 2^-21.4 is then below 2.3e-5 of the result. The outer logarithm sees values in
// (1e-10, 23) where the fast logarithm is accurate to 3 ulp or 2^-21.4 absolute.
__device__ __forceinline__ float gumbel32_from_word(uint32_t x)
{
    // straight-line: both halves are evaluated and one is selected, so lanes never diverge
    const bool upper = x >= 0x80000000u;
    const float u = ((float)x + 0.5f) * 2.3283064365386963e-10f;
    const float z = ((float)(~x) + 0.5f) * 2.3283064365386963e-10f;      // 1 - u
    const float by_log = -__logf(upper ? 1.f - z : u);
    const float by_series = z * (1.f + z * (0.5f + z * (0.33333334f + z * 0.25f)));
    const float nl = (upper && z < 0.015625f) ? by_series : by_log;
    return -__logf(nl);
}

// A fragments of q for the GQA group of (b, j): k-step s of thread column c covers dims
// (c + 4 (s / 2)) * 8 + 4 (s % 2) + {0,1} (a0) and + {2,3} (a2); the B fragments use the same
// permutation of the 128 dims, so a lane feeds the tensor core the 16-byte pieces c, c+4, c+8,
// c+12 of a key row exactly as they lie in memory.
template <int G>
__device__ __forceinline__ void load_q_fragments(const ScoreParams &p, int b, int j, int g, int c, uint32_t (&qa)[8][2])
{
    const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
        p.q + ((size_t)b * p.bv.n_q + (size_t)j * G + (g < G ? g : 0)) * kHeadDim);
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        const int w = (c + 4 * (s >> 1)) * 4 + 2 * (s & 1);
        qa[s][0] = g < G ? __ldg(qrow + w) : 0u;
        qa[s][1] = g < G ? __ldg(qrow + w + 1) : 0u;
    }
}

// Scores of one tile of 16 teams (two n-tiles of 8; B row n = team base + 8 t + g) from the key
// pieces kb of this lane: writes Y32 for the G heads and the tile's maximum per head.
// csr_tile points at the 17 row offsets of the tile's teams (global or shared memory).
template <int G, bool kHalf>
__device__ __forceinline__ void score_tile(const ScoreParams &p, int b, int j, int64_t team0, int M, int base,
                                           const int32_t *csr_tile, const uint4 (&kb)[2][4], const uint32_t (&qa)[8][2],
                                           uint32_t step, float scale, int g, int c)
{
    const uint32_t head = (uint32_t)(j * G + (g < G ? g : 0));
    float *y = p.y32 + (size_t)head * p.bv.teams_total + team0;
    // team sizes of this lane's four teams (teams base + 8 t + 2 c, + 1)
    int n_team[2][2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int t0 = base + 8 * t + 2 * c, o = 8 * t + 2 * c;
        const int r0 = t0 < M ? csr_tile[o] : 0, r1 = t0 < M ? csr_tile[o + 1] : 1, r2 = t0 + 1 < M ? csr_tile[o + 2] : 2;
        n_team[t][0] = r1 - r0;
        n_team[t][1] = r2 - r1;
    }
    float acc[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            mma_16816<kHalf>(acc[t], qa[2 * i][0], qa[2 * i][1], kb[t][i].x, kb[t][i].y);
            mma_16816<kHalf>(acc[t], qa[2 * i + 1][0], qa[2 * i + 1][1], kb[t][i].z, kb[t][i].w);
        }
    }
    // One Philox block covers four consecutive teams of a head: teams base + 8 t + {0..3} belong
    // to thread columns 0 and 1, + {4..7} to columns 2 and 3. The even column computes the block
    // of n-tile 0, the odd one that of n-tile 1, and the two exchange halves.
    const int my_t = c & 1;
    const uint4 words = philox4x32_10(
        make_uint4((uint32_t)(base + 8 * my_t + 4 * (c >> 1)) >> 2, step, head, p.stream_base + (uint32_t)b),
        p.seed_lo, p.seed_hi);
    // this lane needs words {2 (c & 1), 2 (c & 1) + 1} of both n-tiles' blocks
    uint32_t w[2][2];
    {
        const uint32_t give0 = (c & 1) ? words.x : words.z, give1 = (c & 1) ? words.y : words.w;
        const uint32_t got0 = __shfl_xor_sync(0xFFFFFFFFu, give0, 1), got1 = __shfl_xor_sync(0xFFFFFFFFu, give1, 1);
        const uint32_t keep0 = (c & 1) ? words.z : words.x, keep1 = (c & 1) ? words.w : words.y;
        w[0][0] = my_t ? got0 : keep0;
        w[0][1] = my_t ? got1 : keep1;
        w[1][0] = my_t ? keep0 : got0;
        w[1][1] = my_t ? keep1 : got1;
    }
    // acc[t][0], acc[t][1]: head g, teams base + 8 t + 2 c, + 1
    float blk_max = -INFINITY;
    if (g < G) {
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int t0 = base + 8 * t + 2 * c;
            const float y0 = __logf((float)n_team[t][0]) + acc[t][0] * scale + gumbel32_from_word(w[t][0]);
            const float y1 = __logf((float)n_team[t][1]) + acc[t][1] * scale + gumbel32_from_word(w[t][1]);
            if (t0 < M) { y[t0] = y0; blk_max = fmaxf(blk_max, y0); }
            if (t0 + 1 < M) { y[t0 + 1] = y1; blk_max = fmaxf(blk_max, y1); }
        }
    }
    // largest score of the 16-team block, per head (the quad of a head holds its 16 scores)
    blk_max = fmaxf(blk_max, __shfl_xor_sync(0xFFFFFFFFu, blk_max, 1));
    blk_max = fmaxf(blk_max, __shfl_xor_sync(0xFFFFFFFFu, blk_max, 2));
    if (g < G && c == 0)
        p.ymax[(size_t)head * p.ymax_stride + (size_t)(team0 >> 4) + b + (base >> 4)] = blk_max;
}

__device__ __forceinline__ void clear_control(const ScoreParams &p, int tid)
{
    // The first block clears the tickets the later kernels of this call count on.
    for (int i = tid; i < p.n_pairs; i += kScoreThreads) p.ctl.attend_ticket[i] = 0;
    if (tid == 0) {
        *p.ctl.plan_ticket = 0;
        if (p.status) *p.status = 0;
    }
}

// Small grids: one warp per tile of 16 teams, keys straight into registers (the shortest path).
template <int G, bool kHalf>
__global__ void __launch_bounds__(kScoreThreads, 2)
score32_kernel(ScoreParams p)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    const int pair = blockIdx.y;
    const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;
    if (blockIdx.x == 0 && blockIdx.y == 0) clear_control(p, tid);

    const int64_t team0 = p.bv.seq_team_off[b];
    const int M = (int)(p.bv.seq_team_off[b + 1] - team0);
    if (p.n_sample >= M) return;                       // every team is read; nothing is drawn
    const int base = (blockIdx.x * (kScoreThreads / 32) + warp) * kScoreTeamsPerWarp;
    if (base >= M) return;
    uint32_t qa[8][2];
    load_q_fragments<G>(p, b, j, g, c, qa);
    const uint16_t *rep = p.rep_keys + ((size_t)j * p.bv.teams_total + team0) * kHeadDim;
    uint4 kb[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const uint4 *row = reinterpret_cast<const uint4 *>(rep + (size_t)min(base + 8 * t + g, M - 1) * kHeadDim);
#pragma unroll
        for (int i = 0; i < 4; ++i) kb[t][i] = __ldg(row + c + 4 * i);
    }
    const uint32_t step = p.step + (p.step_dev ? *p.step_dev : 0u);
    const int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    score_tile<G, kHalf>(p, b, j, team0, M, base, csr + base, kb, qa, step, (float)p.scale, g, c);
}

// Where a tile index of the flat kernel lies: tiles are the slots of the block-maximum table,
// n_kv * ymax_stride of them; sequence b owns slots [(seq_team_off[b] >> 4) + b, ... + ceil(M / 16)),
// the few slots between sequences are empty.
struct TileCursor {
    int j, s;                       // KV head and slot of the current tile
    int b, slot_lo, slot_hi, M;     // sequence owning the slot range [slot_lo, slot_hi)
    int64_t team0;
};

__device__ __forceinline__ TileCursor cursor_at(const ScoreParams &p, long long ti)
{
    TileCursor cur;
    cur.j = (int)(ti / p.ymax_stride);
    cur.s = (int)(ti - (long long)cur.j * p.ymax_stride);
    cur.b = 0; cur.slot_lo = 0; cur.slot_hi = 0; cur.M = 0; cur.team0 = 0;      // empty range: located on first use
    return cur;
}

// Tile under the cursor: true with its first team in `base` when it has teams to score.
// seq_slot: first slot of every sequence in shared memory (nullptr: read the offsets from global
// memory instead, for batches beyond kSeqTableCap).
__device__ __forceinline__ bool locate_tile(const ScoreParams &p, const int *seq_slot, TileCursor &cur, int &base)
{
    const int s = cur.s;
    if (s < cur.slot_lo || s >= cur.slot_hi) {
        int lo = 0, hi = p.bv.n_seqs - 1;              // largest b with start(b) <= s
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            const int start = seq_slot ? seq_slot[mid] : (int)(p.bv.seq_team_off[mid] >> 4) + mid;
            if (start <= s) lo = mid; else hi = mid - 1;
        }
        cur.b = lo;
        cur.team0 = p.bv.seq_team_off[lo];
        const int64_t next0 = p.bv.seq_team_off[lo + 1];
        cur.M = (int)(next0 - cur.team0);
        cur.slot_lo = (int)(cur.team0 >> 4) + lo;
        cur.slot_hi = lo + 1 < p.bv.n_seqs ? (int)(next0 >> 4) + lo + 1 : p.ymax_stride;
    }
    base = (s - cur.slot_lo) * 16;
    return base < cur.M && p.n_sample < cur.M;
}

__device__ __forceinline__ void advance(const ScoreParams &p, TileCursor &cur)
{
    if (++cur.s == p.ymax_stride) { cur.s = 0; ++cur.j; cur.slot_lo = cur.slot_hi = 0; }
}

// Large grids: two resident blocks per SM, every warp walks an equal contiguous share of all
// tiles. The keys of the next kScoreStages tiles are in flight: lane 0 issues one bulk copy per
// tile (16 keys are one contiguous run) that completes on the stage's mbarrier; the tile's 17 row
// offsets travel as per-lane 4-byte cp.async copies (their address is only 4-byte aligned).
// Every wait on an mbarrier is bounded; on expiry the warp raises status bit 2 and stops.
template <int G, bool kHalf>
__global__ void __launch_bounds__(kScoreThreads, 2)
score32_flat_kernel(ScoreParams p)
{
    extern __shared__ uint4 score_ring[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    if (blockIdx.x == 0) clear_control(p, tid);

    const long long n_tiles = (long long)p.bv.n_kv * p.ymax_stride;
    const long long n_warps = (long long)gridDim.x * (kScoreThreads / 32), gw = (long long)blockIdx.x * (kScoreThreads / 32) + warp;
    const long long t_lo = gw * n_tiles / n_warps, t_hi = (gw + 1) * n_tiles / n_warps;
    const uint32_t step = p.step + (p.step_dev ? *p.step_dev : 0u);
    const float scale = (float)p.scale;

    // keys of the tile in stage s: [warp][s] 16 rows of 256 bytes, as in global memory
    auto tile_of = [&](int s) { return score_ring + (warp * kScoreStages + s) * 256; };
    // completion barrier of stage s, initialised by lane 0
    const uint32_t bars = (uint32_t)__cvta_generic_to_shared(reinterpret_cast<unsigned char *>(score_ring) + kScoreKeyRingBytes
                                                             + kScoreCsrRingBytes + kScoreSeqTableBytes)
                          + (uint32_t)warp * kScoreStages * 8;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kScoreStages; ++s) mbar_init(bars + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // the tile's 17 row offsets, copied by lanes 0..16: [warp][s][32]
    int32_t *csr_ring = reinterpret_cast<int32_t *>(reinterpret_cast<unsigned char *>(score_ring) + kScoreKeyRingBytes)
                        + warp * kScoreStages * 32;
    // first slot of every sequence, for the searches of locate_tile
    int *seq_slot = reinterpret_cast<int *>(reinterpret_cast<unsigned char *>(score_ring) + kScoreKeyRingBytes
                                            + kScoreCsrRingBytes);       // kScoreSeqTableBytes
    if (p.bv.n_seqs <= kSeqTableCap) {
        for (int i = tid; i < p.bv.n_seqs; i += kScoreThreads) seq_slot[i] = (int)(p.bv.seq_team_off[i] >> 4) + i;
        __syncthreads();
    } else {
        seq_slot = nullptr;
    }
    TileCursor ahead = cursor_at(p, t_lo), here = ahead;
    long long t_ahead = t_lo;                                   // tile index under `ahead`
    auto issue_tile = [&](int s) {
        int base;
        if (t_ahead < t_hi && locate_tile(p, seq_slot, ahead, base)) {
            // the tile's keys are one contiguous run: a single bulk copy by lane 0
            if (lane == 0) {
                const uint16_t *src = p.rep_keys + ((size_t)ahead.j * p.bv.teams_total + ahead.team0 + base) * kHeadDim;
                const uint32_t bytes = (uint32_t)min(kScoreTeamsPerWarp, ahead.M - base) * kHeadDim * 2;
                mbar_expect_tx(bars + 8 * s, bytes);
                bulk_copy_to_shared((uint32_t)__cvta_generic_to_shared(tile_of(s)), src, bytes, bars + 8 * s);
            }
            if (lane <= 16 && base + lane <= ahead.M) {
                const int32_t *csr = p.team_row_start + (size_t)ahead.j * (p.bv.teams_total + p.bv.n_seqs) + ahead.team0
                                     + ahead.b + base + lane;
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(
                                 csr_ring + s * 32 + lane)), "l"(csr) : "memory");
            }
        }
        cp_async_commit();                                       // one group per tile, empty or not
        ++t_ahead;
        advance(p, ahead);
    };
#pragma unroll
    for (int s = 0; s < kScoreStages; ++s) issue_tile(s);

    uint32_t qa[8][2];
    int q_b = -1, q_j = -1;
    int stage = 0;
    uint32_t phases = 0u;                                        // bit s: parity of the next completion of stage s
    for (long long ti = t_lo; ti < t_hi; ++ti) {
        cp_async_wait_group<kScoreStages - 1>();                 // this lane's row offset of tile ti has landed
        __syncwarp();                                            // the row offsets come from other lanes
        int base;
        if (locate_tile(p, seq_slot, here, base)) {
            // wait for the tile's keys; the wait is bounded: on expiry the kernel flags it and stops
            int polls = 0;
            while (!mbar_try_wait(bars + 8 * stage, (phases >> stage) & 1u)) {
                if (++polls >= kScoreWaitPolls) break;
            }
            if (polls >= kScoreWaitPolls) {
                if (lane == 0 && p.status) atomicOr(p.status, 4);
                break;
            }
            phases ^= 1u << stage;
            if (here.b != q_b || here.j != q_j) {
                load_q_fragments<G>(p, here.b, here.j, g, c, qa);
                q_b = here.b;
                q_j = here.j;
            }
            uint4 kb[2][4];
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int i = 0; i < 4; ++i) kb[t][i] = tile_of(stage)[(8 * t + g) * 16 + c + 4 * i];
            score_tile<G, kHalf>(p, here.b, here.j, here.team0, here.M, base, csr_ring + stage * 32, kb, qa, step, scale, g, c);
        }
        __syncwarp();                                            // every lane is done with the stage's row offsets
        // refill the stage just consumed (its pieces are in registers and already used above)
        issue_tile(stage);
        advance(p, here);
        stage = stage + 1 == kScoreStages ? 0 : stage + 1;
    }
    cp_async_wait_group<0>();
}

// One block per (sequence, KV head): largest |element| among the pair's representative keys.
__global__ void __launch_bounds__(256)
rep_abs_max_kernel(BatchView bv, const uint16_t *rep_keys, float *rep_abs_max)
{
    __shared__ uint32_t red[8];
    const int b = blockIdx.x, j = blockIdx.y;
    const int64_t team0 = bv.seq_team_off[b];
    const int64_t n = (bv.seq_team_off[b + 1] - team0) * kHeadDim / 2;     // 32-bit words
    const uint32_t *w = reinterpret_cast<const uint32_t *>(rep_keys + ((size_t)j * bv.teams_total + team0) * kHeadDim);
    uint32_t m = 0u;                                       // bf16 and fp16 magnitudes order like integers
    for (int64_t i = threadIdx.x; i < n; i += blockDim.x) {
        const uint32_t v = w[i];
        m = max(m, max(v & 0x7FFFu, (v >> 16) & 0x7FFFu));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) m = max(m, red[i]);
        rep_abs_max[(size_t)j * bv.n_seqs + b] = bv.elem ? elem_to_float<true>((uint16_t)m) : __uint_as_float(m << 16);
    }
}

template <int G, bool kHalf>
cudaError_t launch_score32_g(const ScoreParams &p, int max_teams, cudaStream_t s)
{
    const long long ctas1 = (long long)((max_teams + kScoreTeamsPerCta - 1) / kScoreTeamsPerCta) * p.n_pairs;
    if (ctas1 < 2 * 148) {
        dim3 grid((max_teams + kScoreTeamsPerCta - 1) / kScoreTeamsPerCta, p.n_pairs);
        score32_kernel<G, kHalf><<<grid, kScoreThreads, 0, s>>>(p);
        return cudaGetLastError();
    }
    static std::atomic<unsigned long long> done;
    cudaError_t e = ensure_dynamic_smem((const void *)score32_flat_kernel<G, kHalf>, kScoreRingBytes, done);
    if (e != cudaSuccess) return e;
    score32_flat_kernel<G, kHalf><<<2 * attend_grid_size(), kScoreThreads, kScoreRingBytes, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score32(const ScoreParams &p, int max_teams_per_seq, cudaStream_t s)
{
    switch (p.bv.group) {
        case 1: return p.bv.elem ? launch_score32_g<1, true>(p, max_teams_per_seq, s)
                                 : launch_score32_g<1, false>(p, max_teams_per_seq, s);
        case 2: return p.bv.elem ? launch_score32_g<2, true>(p, max_teams_per_seq, s)
                                 : launch_score32_g<2, false>(p, max_teams_per_seq, s);
        case 3: return p.bv.elem ? launch_score32_g<3, true>(p, max_teams_per_seq, s)
                                 : launch_score32_g<3, false>(p, max_teams_per_seq, s);
        case 4: return p.bv.elem ? launch_score32_g<4, true>(p, max_teams_per_seq, s)
                                 : launch_score32_g<4, false>(p, max_teams_per_seq, s);
        case 5: return p.bv.elem ? launch_score32_g<5, true>(p, max_teams_per_seq, s)
                                 : launch_score32_g<5, false>(p, max_teams_per_seq, s);
        case 6: return p.bv.elem ? launch_score32_g<6, true>(p, max_teams_per_seq, s)
                                 : launch_score32_g<6, false>(p, max_teams_per_seq, s);
        case 7: return p.bv.elem ? launch_score32_g<7, true>(p, max_teams_per_seq, s)
                                 : launch_score32_g<7, false>(p, max_teams_per_seq, s);
        case 8: return p.bv.elem ? launch_score32_g<8, true>(p, max_teams_per_seq, s)
                                 : launch_score32_g<8, false>(p, max_teams_per_seq, s);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_rep_abs_max(const BatchView &bv, const uint16_t *rep_keys, float *rep_abs_max, cudaStream_t s)
{
    rep_abs_max_kernel<<<dim3(bv.n_seqs, bv.n_kv), 256, 0, s>>>(bv, rep_keys, rep_abs_max);
    return cudaGetLastError();
}

}  // namespace santapp
