// Shared declarations of the SANTA++ decode-attention kernels (sm_100a).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "santapp.h"

namespace santapp {

constexpr int kHeadDim = 128;
constexpr int kMaxGroup = 8;            // query heads per KV head
constexpr int kMaxParent = 512;
constexpr int kMaxTeamsPerSeq = 65536;  // the union plan keeps one bit and a prefix word per 32 teams in shared memory
constexpr uint32_t kSrcSuffix = 0x80000000u;   // segment flag: rows live in the suffix buffers

constexpr int kPartialStride = 132;     // floats per (slot, head): m, l, 2 pad, acc[128]
constexpr int kTraceSlots = 16;         // device-timer marks per block (diagnostic trace)
constexpr int kTraceBlocks = 256;       // blocks of a kernel that leave marks; kernel k writes from block slot k * kTraceBlocks

// ---------------------------------------------------------------------------------------------
// Device-side views. Plain structs passed by value to kernels.
// ---------------------------------------------------------------------------------------------

struct BatchView {
    int n_seqs, n_q, n_kv, group;
    const int64_t *seq_row_off;     // [n_seqs + 1]
    const int64_t *seq_team_off;    // [n_seqs + 1] team slots of each sequence
    const int32_t *team_count;      // [n_kv][n_seqs] teams a pair really has, or null: every slot is a team
    int64_t rows_total, teams_total;
    int elem;                       // element type of q / K / V / representative keys: 0 bf16, 1 fp16
};

// Teams of (sequence b, KV head j): the first `pair_team_count` slots of the sequence's range (a
// count outside [0, slots] is clamped, so a corrupt table cannot send a kernel past the records).
__device__ __forceinline__ int pair_team_count(const BatchView &bv, int b, int j)
{
    const int slots = (int)(bv.seq_team_off[b + 1] - bv.seq_team_off[b]);
    return bv.team_count ? min(max(bv.team_count[(size_t)j * bv.n_seqs + b], 0), slots) : slots;
}

// Read plan of one (sequence, KV head) pair: the union of the teams its query heads selected,
// in ascending team id, optionally followed by one suffix segment.
struct PlanView {
    int seg_cap;                    // segments reserved per pair
    int32_t *seg_prefix;            // [n_pairs][seg_cap + 1] exclusive prefix of segment rows
    int32_t *seg_row;               // [n_pairs][seg_cap] first row (global row of the KV plane, or
                                    //   row of the suffix buffer when kSrcSuffix is set in seg_mask)
    uint32_t *seg_mask;             // [n_pairs][seg_cap] bit h: head h of the group selected the team
    float *seg_logc;                // [n_pairs][seg_cap][kMaxGroup] log2(e) * log c_g per selecting head
    int32_t *pair_nseg;             // [n_pairs]
    int32_t *pair_rows;             // [n_pairs] rows of the pair's plan (prompt union + suffix)
    int32_t *pair_union_rows;       // [n_pairs] prompt rows only
    int64_t *pair_row_prefix;       // [n_pairs + 1] exclusive prefix of pair_rows over pairs
    int32_t *tail_counter;          // [2] equal-range split: next tail chunk to hand out, and the count of
                                    //   blocks that have left; zeroed with the plans, both reset themselves
};

// Equal-range split of the attention kernel: the padded row line [0, total) is cut into one fixed
// range per block over its first part and, when the ranges are long enough to pay for it, into
// small chunks over its last part (about a sixth), which blocks take from a counter as they
// finish: blocks do not all stream at the same speed, and the chunks even out their finish.
struct RangeSplit {
    uint32_t total;                 // rows of the padded line (< 2^32: rows_total < 2^31, gaps add at most 2^26 * 16)
    uint32_t fixed_rows;            // rows per fixed range
    uint32_t fixed_end;             // the fixed ranges cover [0, fixed_end)
    uint32_t chunk_rows;            // rows per tail chunk
    int n_tail;                     // tail chunks covering [fixed_end, total)
};
__host__ __device__ __forceinline__ RangeSplit make_range_split(int64_t all_rows, int n_pairs, int span_penalty_rows,
                                                                int min_rows_per_cta, int grid)
{
    RangeSplit sp;
    sp.total = (uint32_t)(all_rows + (int64_t)span_penalty_rows * (n_pairs - 1));
    uint32_t per = (sp.total + (uint32_t)grid - 1u) / (uint32_t)grid;
    if (per < (uint32_t)min_rows_per_cta) per = (uint32_t)min_rows_per_cta;
    if (per < 2048u) {                                      // short ranges: a chunk's fixed cost would not pay
        sp.fixed_rows = per;
        sp.fixed_end = sp.total;
        sp.chunk_rows = 1u;
        sp.n_tail = 0;
        return sp;
    }
    sp.fixed_rows = per - per / 6u;
    const uint64_t covered = (uint64_t)sp.fixed_rows * (uint32_t)grid;
    sp.fixed_end = covered < sp.total ? (uint32_t)covered : sp.total;
    const uint32_t tail = sp.total - sp.fixed_end;
    uint32_t chunk = (tail + 2u * (uint32_t)grid - 1u) / (2u * (uint32_t)grid);
    if (chunk < 256u) chunk = 256u;
    sp.chunk_rows = chunk;
    sp.n_tail = (int)((tail + chunk - 1u) / chunk);
    return sp;
}
constexpr int kMaxTailChunksPerBlock = 2;                   // n_tail <= 2 * grid (+ 1 by rounding)


// Scores of one (query head, sequence) form a row of y_stride floats, y_stride = the longest
// sequence's team slots rounded up to a multiple of 4: rows are 16-byte aligned and their address
// needs nothing that lives in device memory.
__host__ __device__ __forceinline__ int64_t score_row_stride(int max_teams_per_seq)
{
    return ((int64_t)max_teams_per_seq + 3) & ~(int64_t)3;
}

struct ScoreParams {
    BatchView bv;
    const uint16_t *rep_keys;       // [n_kv][teams_total][128]
    const int32_t *team_row_start;  // [n_kv][teams_total + n_seqs]
    const uint16_t *q;              // [n_seqs][n_q][128]
    float *y32;                     // [n_q][n_seqs][y_stride] fp32 perturbed routing scores (see score_row_stride)
    int64_t y_stride;
    int tile_stride;                // tile slots per KV head: sequence b's 16-team tiles start at
                                    //   seq_team_off[b] / 16 + b
    int n_sample;
    uint32_t seed_lo, seed_hi, step, stream_base;
    const uint32_t *step_dev;       // nullable: added to step
    double scale;
    int n_pairs;
    int32_t *status;                // nullable
    unsigned long long *trace;      // nullable, see trace_mark
    int tune_flags;                 // diagnostic builds only
};

// What the sampling step (headplan.cu) and the union step (pairplan.cuh) read and write.
struct PlanInputs {
    BatchView bv;
    const float *y32;               // [n_q][n_seqs][y_stride], see ScoreParams
    int64_t y_stride;
    const uint16_t *rep_keys;       // [n_kv][teams_total][128]
    const int32_t *team_row_start;  // [n_kv][teams_total + n_seqs]
    const float *rep_abs_max;       // [n_kv][n_seqs]
    const uint16_t *q;              // [n_seqs][n_q][128]
    int n_sample;
    uint32_t seed_lo, seed_hi, step, stream_base;
    const uint32_t *step_dev;       // nullable: added to step
    double scale;
    const int32_t *suffix_len;      // nullable
    int suffix_cap;
    int32_t *sel_team;              // [n_seqs][n_q][n_sample] sampled teams of each head, descending score
    float *sel_logc;                // [n_seqs][n_q][n_sample] log c_g of each
    int2 *sel_rows;                 // [n_seqs][n_q][n_sample] first packed row (local to the sequence), row count
    // diagnostics (nullable)
    int32_t *status;
    int32_t *dbg_sel_idx;
    float *dbg_sel_logc;
    double *dbg_tau;
    int32_t *dbg_union_rows;
    unsigned long long *trace;      // nullable: device-timer marks, kTraceSlots per block of a kernel
};

struct PlanParams {
    PlanInputs in;
    PlanView plan;
    int n_pairs;
};

struct AttendParams {
    BatchView bv;
    const uint16_t *k_packed, *v_packed;    // [n_kv][rows_total][128]
    const uint16_t *k_suffix, *v_suffix;    // [n_seqs][n_kv][suffix_cap][128]
    const uint16_t *q;
    float qk_scale_log2;            // scale * log2(e)
    PlanView plan;                  // plan in global memory (dynamic split); seg_logc in both modes
    PlanInputs in;                  // static split: the plan is built inside the kernel
    int n_pairs;
    float *partials;                // [slots][group][kPartialStride]
    float *out;                     // [n_seqs][n_q][128]
    int32_t *status;                // nullable
    int min_rows_per_cta;
    int span_penalty_rows;          // equal-range split: rows a second span costs a CTA (see attend.cu)
    int ctas_per_pair;              // static split: CTAs that share one (sequence, KV head) pair
    int max_words;                  // static split: 32-team words that cover the longest sequence's teams
};

// Kernels that need more than the default dynamic shared memory opt in once per device (the
// attribute belongs to the device's context). `done` has one bit per device ordinal below 64;
// higher ordinals simply set the attribute on every call.
inline cudaError_t ensure_dynamic_smem(const void *fn, int bytes, std::atomic<unsigned long long> &done)
{
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const unsigned long long bit = dev < 64 ? 1ull << dev : 0ull;
    if (bit && (done.load(std::memory_order_acquire) & bit)) return cudaSuccess;
    err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (err == cudaSuccess && bit) done.fetch_or(bit, std::memory_order_release);
    return err;
}

// Launch through cudaLaunchKernelEx so that the launch's own status comes back (no sticky-error read).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Per-thread bookkeeping behind santapp_last_cuda_error / santapp_last_launch_count / santapp_set_stage_mask
// (api.cu), for entry points defined in other files.
int note_cuda_failure(cudaError_t err, const char *where);     // records the text, returns SANTAPP_ERR_CUDA
void note_launch_count(int n);
int current_stage_mask();

// ---------------------------------------------------------------------------------------------
// Host launchers (each returns the cudaError_t of its launches).
// ---------------------------------------------------------------------------------------------
cudaError_t launch_score32(const ScoreParams &p, int max_teams_per_seq, cudaStream_t s);
cudaError_t launch_rep_abs_max(const BatchView &bv, const uint16_t *rep_keys, float *rep_abs_max, cudaStream_t s);
cudaError_t launch_headplan(const PlanInputs &in, cudaStream_t s);
cudaError_t launch_plan(const PlanParams &p, int max_teams_per_seq, cudaStream_t s);
cudaError_t launch_pair_prefix(const PlanParams &p, cudaStream_t s);
cudaError_t launch_dense_plan(const PlanParams &p, cudaStream_t s);
// split: 0 = rows of all pairs cut into equal ranges (plan read from global memory),
//        1 = a fixed number of CTAs per pair (plan built in the kernel; dense: trivial plan)
cudaError_t launch_attend(const AttendParams &p, bool all_heads, bool static_split, int grid, cudaStream_t s);
// log-sum-exp merge of the partials the attention kernel left (launched with `attend_grid` blocks)
cudaError_t launch_merge(const AttendParams &p, bool static_split, int attend_grid, cudaStream_t s);
int attend_grid_size();
int attend_max_segments();
int attend_max_pairs();
int attend_pairs_staged();

struct BuildParams {
    BatchView bv;
    int parent_size, reps;
    int teams_per_full_parent;              // min(R, P)
    const uint16_t *k_prompt, *v_prompt;    // [n_kv][rows_total][128] token order
    uint16_t *k_packed, *v_packed, *rep_keys;
    int32_t *team_row_start, *row_token;
    int32_t *team_count;                    // [n_kv][n_seqs] or null
    uint16_t *owner;                        // workspace [n_kv][rows_total]: team index inside the parent
    int max_parents_per_seq;
};
cudaError_t launch_build_teams(const BuildParams &p, cudaStream_t s);
cudaError_t launch_build_groups_mean(const BuildParams &p, cudaStream_t s);

// Nearest-centre assignment (last step of Algorithm 3).
struct AssignParams {
    int n_seqs, n_kv, max_rows_per_seq, elem;
    int64_t rows_total, centres_total;
    const int64_t *seq_row_off;             // device [n_seqs + 1]
    const int64_t *seq_centre_off;          // device [n_seqs + 1]
    const uint16_t *k_prompt;               // [n_kv][rows_total][128]
    const float *centres;                   // [n_kv][centres_total][128]
    int32_t *parent_of;                     // [n_kv][rows_total] out
};
cudaError_t launch_assign_parents(const AssignParams &p, cudaStream_t s);

// Team records from an arbitrary parent partition given as one label per token.
struct ParentBuildParams {
    BatchView bv;                           // seq_team_off: team slots per sequence
    int reps, max_labels_per_seq, max_rows_per_seq;
    bool mean_keys;                         // one group per parent routed by its mean key (reps = 1)
    int64_t labels_total;
    const uint16_t *k_prompt, *v_prompt;    // [n_kv][rows_total][128] token order
    const int32_t *parent_of;               // [n_kv][rows_total] label of each token
    const int64_t *seq_label_off;           // device [n_seqs + 1]
    uint16_t *k_packed, *v_packed, *rep_keys;
    int32_t *team_row_start, *row_token, *team_count;
    // workspace
    int32_t *parent_start;                  // [n_kv][labels_total + n_seqs] member-list offsets
    int32_t *parent_cursor;                 // [n_kv][labels_total] counts, then scatter cursors
    int32_t *parent_team_base;              // [n_kv][labels_total] first team of each parent
    int32_t *members;                       // [n_kv][rows_total] tokens ordered by (label, index)
    int32_t *team_of;                       // [n_kv][rows_total] team of each token
    double *mind;                           // [n_kv][rows_total] distance to the nearest representative
    int32_t *owner;                         // [n_kv][rows_total] its rank inside the parent
    unsigned char *is_rep;                  // [n_kv][rows_total]
    int32_t *team_cursor;                   // [n_kv][teams_total]
    int32_t *dest;                          // [n_kv][rows_total] packed position of each token
};
cudaError_t launch_build_teams_parents(const ParentBuildParams &p, cudaStream_t s);

// Minibatch k-means fit (second line of Algorithm 3), one problem per (sequence, KV head).
struct KmeansState {
    double ewa, ewa_min;                    // averaged per-point inertia and its minimum so far
    int bad, steps, stopped, pad;
};
struct KmeansParams {
    int n_seqs, n_kv, elem, max_rows_per_seq;
    int batch, patience;
    int no_host_poll;                       // never wait for the stream inside the call
    double ratio;
    uint32_t seed_lo, seed_hi, stream_base;
    int k_max, n_init_max, trials_max, t_max_max;   // maxima over the sequences
    int64_t rows_total, centres_total;
    const int64_t *seq_row_off, *seq_centre_off;    // device [n_seqs + 1]
    const int32_t *seq_n_init, *seq_trials, *seq_t_max;   // device [n_seqs]
    const uint16_t *k_prompt;               // [n_kv][rows_total][128]
    float *centres_out;                     // [n_kv][centres_total][128]
    int32_t *steps_out;                     // [n_kv][n_seqs] or null
    // workspace; "pairs" arrays are indexed by j * n_seqs + b
    int32_t *perm;                          // [n_kv][rows_total]
    double *closest;                        // [pairs][n_init_max]
    double *cand;                           // [pairs][trials_max][n_init_max]
    double *part;                           // [pairs][trials_max][ceil(n_init_max / 128)] block sums of the trials' potentials
    int32_t *pick;                          // [pairs][trials_max]
    double *centres64;                      // [n_kv][centres_total][128]
    double *count;                          // [n_kv][centres_total]
    int32_t *idx, *label;                   // [pairs][batch]
    double *dist;                           // [pairs][batch]
    double *dist_part;                      // [pairs][assign_split][batch] nearest centre inside each slice of the centres
    int32_t *label_part;                    // [pairs][assign_split][batch]
    int assign_split;                       // slices the centres are cut into for the nearest-centre search
    uint32_t *sorted;                       // [pairs][4096] minibatch slots ordered by (label, slot): label << 12 | slot, padded with ~0
    KmeansState *state;                     // [pairs]
    int *active;                            // [1] fits that still have steps to run
};
cudaError_t launch_kmeans_fit(const KmeansParams &p, cudaStream_t s);

// Per-sequence tables of the fit, handed to the device inside kernel arguments (a copy from host
// memory that is gone after the call would be read again by every replay of a captured graph).
constexpr int kKmTableChunk = 128;
struct KmTableChunk {
    int32_t first, n;                               // sequences [first, first + n); offsets also get entry first + n
    int64_t row_off[kKmTableChunk + 1], centre_off[kKmTableChunk + 1];
    int32_t n_init[kKmTableChunk], trials[kKmTableChunk], t_max[kKmTableChunk];
};
cudaError_t launch_kmeans_tables(const KmTableChunk &c, int64_t *row_off, int64_t *centre_off, int32_t *n_init,
                                 int32_t *trials, int32_t *t_max, cudaStream_t s);

// ---------------------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ float bf16_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }
__device__ __forceinline__ double bf16_to_double(uint16_t b) { return (double)bf16_to_float(b); }

// The same three conversions for either 16-bit element type (kHalf: IEEE fp16, else bf16).
template <bool kHalf>
__device__ __forceinline__ float elem_to_float(uint16_t b)
{
    if constexpr (kHalf) return __half2float(__ushort_as_half(b));
    else return bf16_to_float(b);
}
template <bool kHalf>
__device__ __forceinline__ float elem_lo(uint32_t w)
{
    if constexpr (kHalf) return __half2float(__ushort_as_half((unsigned short)(w & 0xFFFFu)));
    else return bf16_lo(w);
}
template <bool kHalf>
__device__ __forceinline__ float elem_hi(uint32_t w)
{
    if constexpr (kHalf) return __half2float(__ushort_as_half((unsigned short)(w >> 16)));
    else return bf16_hi(w);
}

// fp32 -> fp64 where it is written (the compiler would otherwise widen all of a point's values ahead of
// a loop over centres and keep them in local memory)
__device__ __forceinline__ double widen_here(float x)
{
    double r;
    asm volatile("cvt.f64.f32 %0, %1;" : "=d"(r) : "f"(x));
    return r;
}

// Squared distances (fp64, the 128 terms added in order) of kP points (rows of packed words in global
// memory, read eight values at a time, one read ahead) to kN candidate points held as doubles in
// shared memory: a candidate value serves all kP points and a point value is widened once for all
// candidates (widening runs at a quarter of the fp64 add rate). The loop is kept rolled: a warp runs
// it once, and a body unrolled over the whole row is fetched from instruction memory slower than it runs.
template <bool kHalf, int kP, int kN, int kD>
__device__ __forceinline__ void dist_points(const uint4 *const (&row)[kP], const double (*y_s)[kHeadDim], double (&d)[kP][kD])
{
    uint4 nxt[kP];
#pragma unroll
    for (int j = 0; j < kP; ++j) nxt[j] = row[j][0];
#pragma unroll 1
    for (int qd = 0; qd < 16; ++qd) {
        uint32_t xw[kP][4];
#pragma unroll
        for (int j = 0; j < kP; ++j) {
            xw[j][0] = nxt[j].x; xw[j][1] = nxt[j].y; xw[j][2] = nxt[j].z; xw[j][3] = nxt[j].w;
            if (qd + 1 < 16) nxt[j] = row[j][qd + 1];
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            double2 y[kN];
#pragma unroll
            for (int v = 0; v < kN; ++v) y[v] = *reinterpret_cast<const double2 *>(&y_s[v][8 * qd + 2 * t]);
#pragma unroll
            for (int j = 0; j < kP; ++j) {
                const double x0 = widen_here(elem_lo<kHalf>(xw[j][t])), x1 = widen_here(elem_hi<kHalf>(xw[j][t]));
#pragma unroll
                for (int v = 0; v < kN; ++v) {
                    const double e = __dsub_rn(x0, y[v].x);
                    d[j][v] = __dadd_rn(d[j][v], __dmul_rn(e, e));
                }
#pragma unroll
                for (int v = 0; v < kN; ++v) {
                    const double e = __dsub_rn(x1, y[v].y);
                    d[j][v] = __dadd_rn(d[j][v], __dmul_rn(e, e));
                }
            }
        }
    }
}

template <bool kHalf>
__device__ __forceinline__ double elem_to_double(uint16_t b) { return (double)elem_to_float<kHalf>(b); }
// fp64 -> fp32 (to nearest) -> the 16-bit element type (to nearest even): how a computed routing key is stored.
template <bool kHalf>
__device__ __forceinline__ uint16_t double_to_elem(double v)
{
    const float f = __double2float_rn(v);
    if constexpr (kHalf) return __half_as_ushort(__float2half_rn(f));
    const uint32_t bits = __float_as_uint(f);
    return (uint16_t)((bits + 0x7FFFu + ((bits >> 16) & 1u)) >> 16);
}

// Philox4x32-10: 128-bit counter, 64-bit key, four 32-bit words.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c;
}

// Gumbel(0,1) from a 32-bit word: u = (x + 0.5) / 2^32 in (0,1), G = -log(-log u), in fp64.
__device__ __forceinline__ double gumbel_from_word(uint32_t x)
{
    const double u = ((double)x + 0.5) * (1.0 / 4294967296.0);
    return -log(-log(u));
}

__device__ __forceinline__ uint32_t pick_word(const uint4 &w, int i)
{
    return i == 0 ? w.x : (i == 1 ? w.y : (i == 2 ? w.z : w.w));
}

// Diagnostic: thread 0 of a block notes the device timer (ns) in slot `slot` of its block's marks.
__device__ __forceinline__ void trace_mark(unsigned long long *trace, int kernel, int slot)
{
    const unsigned blk = blockIdx.x + blockIdx.y * gridDim.x;
    if (trace != nullptr && threadIdx.x == 0 && blk < (unsigned)kTraceBlocks) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        trace[((size_t)kernel * kTraceBlocks + blk) * kTraceSlots + slot] = t;
    }
}

// Order-preserving map from a double to an unsigned 64-bit key (larger double <=> larger key).
__device__ __forceinline__ unsigned long long sortable_key(double v)
{
    const unsigned long long b = (unsigned long long)__double_as_longlong(v);
    return (b & 0x8000000000000000ull) ? ~b : (b | 0x8000000000000000ull);
}
__device__ __forceinline__ double key_to_double(unsigned long long k)
{
    const unsigned long long b = (k & 0x8000000000000000ull) ? (k & 0x7FFFFFFFFFFFFFFFull) : ~k;
    return __longlong_as_double((long long)b);
}

// Exclusive prefix sum of one int per thread over the block; returns the thread's offset and the
// block total. `scratch` needs 33 ints of shared memory. blockDim.x is a multiple of 32, <= 1024.
__device__ __forceinline__ int block_exclusive_scan(int v, int *scratch, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();                       // scratch may still be read from a previous call
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < n_warps ? scratch[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
            if (lane >= o) wi += t;
        }
        scratch[lane] = wi - w;            // exclusive offset of each warp
        if (lane == 31) scratch[32] = wi;  // block total
    }
    __syncthreads();
    total = scratch[32];
    return scratch[warp] + incl - v;
}

}  // namespace santapp
