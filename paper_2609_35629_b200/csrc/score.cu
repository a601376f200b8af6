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
#include "score_tile.cuh"

namespace santapp {

namespace {

constexpr int kScoreThreads = 256;
constexpr int kScoreTeamsPerCta = kScoreTeamsPerWarp * (kScoreThreads / 32);

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

__device__ __forceinline__ ScoreCtx score_ctx(const ScoreParams &p)
{
    ScoreCtx c;
    c.y32 = p.y32;
    c.y_stride = p.y_stride;
    c.n_q = p.bv.n_q;
    c.n_seqs = p.bv.n_seqs;
    c.q = p.q;
    c.seed_lo = p.seed_lo;
    c.seed_hi = p.seed_hi;
    c.stream_base = p.stream_base;
    c.tune_flags = p.tune_flags;
    return c;
}

// Small grids: one warp per tile of 16 teams, keys straight into registers (the shortest path).
template <int G, bool kHalf>
__global__ void __launch_bounds__(kScoreThreads, 2)
score32_kernel(ScoreParams p)
{
    __shared__ uint4 philox_words[kScoreThreads / 32][32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    const int pair = blockIdx.y;
    const int b = pair / p.bv.n_kv, j = pair - b * p.bv.n_kv;
    trace_mark(p.trace, 0, 0);

    const int64_t team0 = p.bv.seq_team_off[b];
    const int M = (int)(p.bv.seq_team_off[b + 1] - team0);
    if (p.n_sample >= M) return;                       // every team is read; nothing is drawn
    const int base = (blockIdx.x * (kScoreThreads / 32) + warp) * kScoreTeamsPerWarp;
    if (base >= M) return;
    const ScoreCtx ctx = score_ctx(p);
    uint32_t qa[8][2];
    load_q_fragments<G>(ctx, b, j, g, c, qa);
    const uint16_t *rep = p.rep_keys + ((size_t)j * p.bv.teams_total + team0) * kHeadDim;
    uint4 kb[2][4];
    load_key_pieces(rep, base, M, g, c, kb);
    const uint32_t step = p.step + (p.step_dev ? *p.step_dev : 0u);
    const int32_t *csr = p.team_row_start + (size_t)j * (p.bv.teams_total + p.bv.n_seqs) + team0 + b;
    TileScores ts;
    uint32_t *words = reinterpret_cast<uint32_t *>(philox_words[warp]);
    score_tile_front<G, kHalf>(ctx, b, j, M, base, csr + base, kb, qa, step, g, c, words, ts);
    __syncwarp();                                      // every lane's Philox words are in shared memory
    score_tile_back<G>(ts, (float)p.scale, g, c, words);
    trace_mark(p.trace, 0, 1);
}

// Where a tile index of the flat kernel lies: every KV head has tile_stride tile slots, n_kv *
// tile_stride in all; sequence b owns slots [(seq_team_off[b] >> 4) + b, ... + ceil(M / 16)),
// the few slots between sequences are empty.
struct TileCursor {
    int j, s;                       // KV head and slot of the current tile
    int b, slot_lo, slot_hi, M;     // sequence owning the slot range [slot_lo, slot_hi)
    int64_t team0;
};

__device__ __forceinline__ TileCursor cursor_at(const ScoreParams &p, long long ti)
{
    TileCursor cur;
    cur.j = (int)(ti / p.tile_stride);
    cur.s = (int)(ti - (long long)cur.j * p.tile_stride);
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
        cur.slot_hi = lo + 1 < p.bv.n_seqs ? (int)(next0 >> 4) + lo + 1 : p.tile_stride;
    }
    base = (s - cur.slot_lo) * 16;
    return base < cur.M && p.n_sample < cur.M;
}

__device__ __forceinline__ void advance(const ScoreParams &p, TileCursor &cur)
{
    if (++cur.s == p.tile_stride) { cur.s = 0; ++cur.j; cur.slot_lo = cur.slot_hi = 0; }
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
    __shared__ uint4 philox_words[kScoreThreads / 32][32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    const long long n_tiles = (long long)p.bv.n_kv * p.tile_stride;
    const long long n_warps = (long long)gridDim.x * (kScoreThreads / 32), gw = (long long)blockIdx.x * (kScoreThreads / 32) + warp;
    const long long t_lo = gw * n_tiles / n_warps, t_hi = (gw + 1) * n_tiles / n_warps;
    const float scale = (float)p.scale;
    const ScoreCtx ctx = score_ctx(p);

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
    const uint32_t step = p.step + (p.step_dev ? *p.step_dev : 0u);
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
    uint32_t pending = 0u;                                       // bit s: a bulk copy into stage s is in flight
    auto issue_tile = [&](int s) {
        int base;
        if (t_ahead < t_hi && locate_tile(p, seq_slot, ahead, base)) {
            pending |= 1u << s;
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
    uint32_t *words = reinterpret_cast<uint32_t *>(philox_words[warp]);
#ifdef SANTAPP_TUNE
    long long tk[4] = {0, 0, 0, 0}, tk0 = clock64();
#define SCORE_TICK(i) { const long long now = clock64(); tk[i] += now - tk0; tk0 = now; }
#else
#define SCORE_TICK(i)
#endif
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
                // Never expected. The step is marked invalid; before the warp leaves it waits (again
                // with a limit) for the copies it still has in flight, so that none of them lands
                // in shared memory that no longer belongs to this block.
                if (lane == 0 && p.status) atomicOr(p.status, 4);
                for (int s = 0; s < kScoreStages; ++s) {
                    if (!((pending >> s) & 1u)) continue;
                    for (int again = 0; again < kScoreWaitPolls; ++again)
                        if (mbar_try_wait(bars + 8 * s, (phases >> s) & 1u)) break;
                }
                break;
            }
            pending &= ~(1u << stage);
            phases ^= 1u << stage;
            SCORE_TICK(0)
            if (here.b != q_b || here.j != q_j) {
                load_q_fragments<G>(ctx, here.b, here.j, g, c, qa);
                q_b = here.b;
                q_j = here.j;
            }
            uint4 kb[2][4];
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int i = 0; i < 4; ++i) kb[t][i] = tile_of(stage)[(8 * t + g) * 16 + c + 4 * i];
            SCORE_TICK(1)
            TileScores ts;
            score_tile_front<G, kHalf>(ctx, here.b, here.j, here.M, base, csr_ring + stage * 32, kb, qa, step, g, c, words, ts);
            __syncwarp();                                        // every lane's Philox words are in shared memory
            score_tile_back<G>(ts, scale, g, c, words);
            SCORE_TICK(2)
        }
        __syncwarp();                                            // every lane is done with the stage's row offsets and the words
        // refill the stage just consumed (its pieces are in registers and already used above)
        issue_tile(stage);
        advance(p, here);
        stage = stage + 1 == kScoreStages ? 0 : stage + 1;
        SCORE_TICK(3)
    }
    cp_async_wait_group<0>();
#ifdef SANTAPP_TUNE
    if (p.trace && lane == 0 && blockIdx.x < 8) {
        unsigned long long *o = p.trace + ((size_t)blockIdx.x * 8 + warp) * 8;
        o[0] = (unsigned long long)(t_hi - t_lo);
        for (int i = 0; i < 4; ++i) o[1 + i] = (unsigned long long)tk[i];
    }
#endif
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
    if (ctas1 < 2 * attend_grid_size()) {
        dim3 grid((max_teams + kScoreTeamsPerCta - 1) / kScoreTeamsPerCta, p.n_pairs);
        return launch_kernel(score32_kernel<G, kHalf>, grid, dim3(kScoreThreads), 0, s, p);
    }
    static std::atomic<unsigned long long> done;
    cudaError_t e = ensure_dynamic_smem((const void *)score32_flat_kernel<G, kHalf>, kScoreRingBytes, done);
    if (e != cudaSuccess) return e;
    return launch_kernel(score32_flat_kernel<G, kHalf>, dim3(2 * attend_grid_size()), dim3(kScoreThreads), kScoreRingBytes, s, p);
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
