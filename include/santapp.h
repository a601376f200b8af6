/*
 * santapp.h — C ABI of the SANTA++ decode-attention library for NVIDIA B200 (sm_100a).
 *
 * Three operations, named after the paper's statement of the problem:
 *
 *   santapp_build_teams        once after prefill, per sequence and KV head: contiguous
 *                              parent groups (Algorithm 4), actual-key representatives and
 *                              nearest-representative teams (Algorithm 2), written out as a
 *                              team-contiguous copy of K/V with CSR row offsets (the packed
 *                              copy of the appendix "Triton decode kernels").
 *   santapp_decode_attn        per generated token: SANTA++ attention for every query head
 *                              (Algorithm 1) under the GQA rule of the Method section.
 *   santapp_dense_decode_attn  full-cache attention, Eq. (method-attention), over the same
 *                              buffers: the in-library dense baseline.
 * Beside them: santapp_assign_parents and santapp_build_teams_parents (Algorithm 3 after the fit:
 * nearest-centre parents, then Algorithm 2 on parents of any size) and santapp_build_groups_mean
 * (the centroid-guided baseline of the routing diagnostic).
 *
 * Conventions
 *   - "device" pointers address GPU global memory of the current device; "host" pointers
 *     address CPU memory. The library allocates no device memory and keeps no state between
 *     calls (one exception, stated with it: santapp_dense_decode_attn_noalloc and its built-in
 *     array): the caller owns every buffer, including workspaces, whose sizes come from the
 *     *_sizes / *_workspace_bytes queries. A workspace needs no initialisation: every word a
 *     kernel reads was written earlier in the same call. Buffers should be 256-byte aligned; a bf16 / fp32 array or a
 *     workspace that is not at least 16-byte aligned (64-bit offset arrays: 8, 32-bit tables: 4)
 *     is refused with SANTAPP_ERR_INVALID_ARG.
 *   - bf16 tensors are raw 16-bit patterns. head_dim is 128. Query head h uses KV head
 *     h / (n_q_heads / n_kv_heads); at most 8 query heads per KV head.
 *   - A batch holds n_seqs independent sequences of prompt length prompt_len[b] >= 1; prompt
 *     rows of all sequences are concatenated: sequence b owns rows
 *     [seq_row_off[b], seq_row_off[b+1]) of each KV head's plane.
 *   - Team ids are local to a (sequence, KV head), numbered parent by parent and, inside a
 *     parent, in representative-selection order (the emission order of Algorithm 2).
 *   - Every call is asynchronous on `stream` (a cudaStream_t passed as void*; NULL is the
 *     legacy default stream) and returns SANTAPP_OK or a negative santapp_status. No call
 *     throws, aborts or traps. Argument errors are detected on the host before any launch.
 *
 * Random stream (the paper asks for independent Gumbel(0,1) draws; this is the library's
 * realisation): Philox4x32-10 with key = (seed low 32 bits, seed high 32 bits) and counter
 * (team_id / 4, step, query head index, stream_base + sequence index); team g takes word
 * g mod 4; u = (word + 0.5) / 2^32; G = -log(-log u). The draw is a pure function of
 * (seed, step, head, sequence stream, team), so a replayed step reproduces its sample.
 */
#ifndef SANTAPP_H
#define SANTAPP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum santapp_status {
    SANTAPP_OK = 0,
    SANTAPP_ERR_INVALID_ARG = -1,        /* null pointer, non-positive size, K < 1, R does not divide P, ... */
    SANTAPP_ERR_UNSUPPORTED = -2,        /* head_dim != 128, group size > 8, parent_size > 512, too many teams */
    SANTAPP_ERR_WORKSPACE_TOO_SMALL = -3,
    SANTAPP_ERR_CUDA = -4,               /* a CUDA runtime call or launch failed; see santapp_last_cuda_error */
    SANTAPP_ERR_STATIC_SCRATCH = -5      /* the problem needs more scratch than the built-in array holds */
} santapp_status;

typedef void *santapp_stream;            /* cudaStream_t */

/* 16-bit element type of the inputs. Wherever this header says "bf16" for q, K, V, the suffix or
 * the representative keys, the tensor holds raw 16-bit patterns of this type. Outputs are fp32 and
 * every accumulation is fp32 or fp64 for both. The paper's own runs use fp16 inputs
 * (Appendix "Kernel evaluation protocol and profiling"). */
typedef enum santapp_elem { SANTAPP_BF16 = 0, SANTAPP_FP16 = 1 } santapp_elem;

/* Problem geometry (host struct). */
typedef struct santapp_geom {
    int32_t n_seqs;            /* B: sequences in the batch                         */
    int32_t n_q_heads;         /* Hq                                               */
    int32_t n_kv_heads;        /* Hkv; must divide Hq                              */
    int32_t head_dim;          /* d; 128                                           */
    int32_t parent_size;       /* P: nominal parent size (Algorithm 4), <= 512      */
    int32_t reps_per_parent;   /* R: maximum representatives per parent; divides P  */
    int32_t elem_type;         /* santapp_elem of q, K, V and the representative keys */
} santapp_geom;

/* Sizes derived from the geometry and the prompt lengths (host struct, output). */
typedef struct santapp_sizes {
    int64_t rows_total;              /* sum_b prompt_len[b]                                          */
    int64_t teams_total;             /* sum_b M_b, M_b = sum over parents of min(R, parent rows)     */
    int32_t max_teams_per_seq;       /* max_b M_b                                                    */
    int32_t max_rows_per_seq;        /* max_b prompt_len[b]                                          */
    int64_t team_row_start_elems;    /* n_kv_heads * (teams_total + n_seqs) int32 elements           */
    size_t build_workspace_bytes;    /* workspace santapp_build_teams needs                          */
} santapp_sizes;

/*
 * Team records (Section "Preparing parent groups and teams"; packed layout of the appendix
 * "Triton decode kernels"). All pointers are device pointers, caller-allocated. After
 * santapp_build_teams they are immutable: memberships and representative keys stay fixed
 * for the whole decode.
 */
typedef struct santapp_teams {
    void *k_packed;            /* bf16 [n_kv_heads][rows_total][d]: each team's members occupy a
                                  contiguous row range, teams in id order, members by token index   */
    void *v_packed;            /* bf16, same layout                                                 */
    void *rep_keys;            /* bf16 [n_kv_heads][teams_total][d]: frozen representative keys      */
    int32_t *team_row_start;   /* int32 [n_kv_heads][teams_total + n_seqs]: for sequence b the
                                  M_b + 1 CSR offsets start at element seq_team_off[b] + b; values
                                  are row offsets local to the sequence (0 .. prompt_len[b])         */
    int32_t *row_token;        /* int32 [n_kv_heads][rows_total]: prompt token index (local to its
                                  sequence) of each packed row                                       */
    int64_t *seq_row_off;      /* int64 [n_seqs + 1] device copy of the row offsets                  */
    int64_t *seq_team_off;     /* int64 [n_seqs + 1] device copy of the team offsets                 */
    float *rep_abs_max;        /* fp32  [n_kv_heads][n_seqs]: largest |element| among the pair's
                                  representative keys (bounds the fp32 routing pass)                 */
    int32_t *team_count;       /* int32 [n_kv_heads][n_seqs], or NULL: the number of teams M of each
                                  (sequence, KV head). The offsets above reserve the same number of
                                  team slots for every KV head of a sequence; a pair whose parents
                                  yield fewer teams (santapp_build_teams_parents) uses the first M
                                  slots, and the slots behind them are empty teams (row offset =
                                  prompt length, representative key zero) that the decode ignores.
                                  NULL means every slot holds a team. Written by every builder
                                  when not NULL.                                                    */
    int64_t rows_total;        /* host scalars, as in santapp_sizes                                  */
    int64_t teams_total;
    int32_t max_teams_per_seq;
    int32_t max_rows_per_seq;
} santapp_teams;

/*
 * Optional per-step diagnostics (device pointers, each may be NULL).
 * With Ke = min(K, M_b): sel_idx/sel_logc hold Ke entries per head followed by -1 / 0 padding.
 */
typedef struct santapp_debug {
    int32_t *sel_idx;          /* int32 [n_seqs][n_q_heads][K]: sampled team ids in descending
                                  perturbed score; 0..M_b-1 when K >= M_b                            */
    float *sel_logc;           /* fp32  [n_seqs][n_q_heads][K]: log c_g, Eq. (method-inclusion)      */
    double *tau;               /* fp64  [n_seqs][n_q_heads]: (K+1)-st largest perturbed score; NaN
                                  when K >= M_b                                                      */
    int32_t *union_rows;       /* int32 [n_seqs][n_kv_heads]: distinct prompt rows read (u_c of the
                                  logical-access counter)                                            */
    int32_t *status;           /* int32 [1]: bit flags raised on the device (0 = clean);
                                  bit 0: non-finite output; bit 1: a head had fewer than K + 1
                                  comparable routing scores (non-finite q or keys): its sample was
                                  completed with arbitrary teams, the output is meaningless;
                                  bit 2: a bounded wait for an asynchronous copy expired in the
                                  scorer (never expected; the step's result is not valid).
                                  Cleared by the call itself before its first kernel                */
    uint64_t *trace;           /* uint64 [5][256][16] or NULL: device-timer readings (ns) that thread 0
                                  of the first 256 blocks of each kernel of the call notes at fixed
                                  points, [kernel][block][mark]; kernels in launch order: scoring,
                                  sampling, read plans, attention, merge. For latency breakdowns;
                                  not a stable interface                                             */
} santapp_debug;

/* Library version: major * 10000 + minor * 100 + patch. */
int santapp_version(void);

/* Text for a santapp_status value. The returned string is static. */
const char *santapp_strerror(int status);

/* Text of the last CUDA error a call on this thread ran into (static storage; "" if none). */
const char *santapp_last_cuda_error(void);

/*
 * Sizes for a batch (Algorithm 4: sequence b has ceil(prompt_len[b] / P) parents; Algorithm 2:
 * a parent of c rows yields min(R, c) teams).
 *   geom             host, in
 *   prompt_len_host  host int32 [n_seqs], in; every entry >= 1
 *   out              host, out
 */
int santapp_build_teams_sizes(const santapp_geom *geom, const int32_t *prompt_len_host,
                              santapp_sizes *out);

/*
 * Build the team records of one layer for every (sequence, KV head).
 * Algorithm 4 (contiguous parents of P tokens, last one possibly short), then Algorithm 2 per
 * parent: r = min(R, rows); first representative = the key nearest the parent mean; each later
 * one = the key farthest from its nearest chosen representative; every key joins its nearest
 * representative (squared Euclidean distance on the raw keys, evaluated in fp64); each
 * representative owns its own row. Ties: representative choices go to the smaller token index,
 * assignments to the earlier-selected representative.
 *   k_prompt, v_prompt   device bf16 [n_kv_heads][rows_total][d], token order, in (not modified)
 *   teams                host struct of device pointers, out: every array is overwritten; the
 *                        host scalars are filled in
 *   workspace            device, >= sizes.build_workspace_bytes; contents undefined afterwards
 * The call copies the (n_seqs + 1)-entry offset tables to the device with cudaMemcpyAsync from
 * pageable memory, which orders after prior work on `stream`; it is a preparation call, outside
 * the per-token path.
 */
int santapp_build_teams(const santapp_geom *geom, const int32_t *prompt_len_host,
                        const void *k_prompt, const void *v_prompt,
                        santapp_teams *teams, void *workspace, size_t workspace_bytes,
                        santapp_stream stream);

/*
 * Centroid-guided grouping, the baseline the paper's routing diagnostic compares the team variant
 * with (Section "How closely routing follows dense attention"; appendix on the KL variants): one
 * group per parent, routed by the arithmetic mean of its keys instead of an actual key; routing
 * logit, sampling, correction and estimator are those of Algorithm 1, so the records are consumed by
 * santapp_decode_attn unchanged. The paper forms the groups by k-means; this call uses the
 * contiguous parents of Algorithm 4 (group size = geom->parent_size, last one possibly short).
 * The mean of a parent is the fp64 sum of its keys in token order divided by their number, stored
 * in the element type (fp64 to fp32 to nearest, fp32 to bf16 or fp16 to nearest even). Rows keep their token order.
 * geom->reps_per_parent must be 1 (sizes then come from santapp_build_teams_sizes as usual).
 * Arguments, ownership and errors as for santapp_build_teams.
 */
int santapp_build_groups_mean(const santapp_geom *geom, const int32_t *prompt_len_host,
                              const void *k_prompt, const void *v_prompt,
                              santapp_teams *teams, void *workspace, size_t workspace_bytes,
                              santapp_stream stream);

/*
 * Algorithm 3 (global k-means parents), first line: the number of centres to fit for a prompt of
 * prompt_len >= 2 keys and nominal parent size P: min(prompt_len, max(2, prompt_len / P)).
 * Returns 0 for arguments outside that range. Host arithmetic only.
 */
int32_t santapp_kmeans_parent_count(int32_t prompt_len, int32_t parent_size);

/*
 * Algorithm 3, the fit: minibatch k-means on the raw keys of each (sequence, KV head), squared
 * Euclidean distance, fp64 arithmetic. The paper fixes the routine's settings (the defaults named
 * below) and leaves its details to a library; this is the routine as built here:
 *   1. Initialisation sample: min(N, max(3 * batch, 3 * k)) distinct keys, the head of a
 *      Fisher-Yates shuffle of the token indices.
 *   2. Greedy k-means++ on the sample with 2 + floor(ln k) trials per centre: the first centre is
 *      a uniform sample point; each later one is the best of the trial points drawn with
 *      probability proportional to the squared distance to the nearest centre so far, best meaning
 *      the smallest resulting sum of nearest-centre distances over the sample. Sums over the
 *      sample (that potential, and the running sums of the draw) are taken in blocks of 128
 *      consecutive sample points: inside a block in order, then the block sums in order.
 *   3. At most max_iter * ceil(N / batch) steps; a step draws `batch` token indices uniformly with
 *      replacement, assigns each to its nearest centre (ties to the smaller index) and moves every
 *      centre that received points to the mean of all points it has received so far
 *      (cumulative count).
 *   4. At steps t with (t + 1) divisible by 10 + floor(smallest count), centres whose count is
 *      below reassignment_ratio * (largest count), at most batch / 2 of them, jump onto distinct
 *      points of the current minibatch and take the smallest count among the centres that stay.
 *   5. The per-point inertia of each minibatch feeds an exponentially weighted average with
 *      weight min(1, 2 * batch / (N + 1)); the fit stops after `patience` consecutive steps
 *      without a new minimum of that average. There is no centre-change criterion (tolerance 0).
 * Random choices are words of the library's Philox stream (top of this file) with counter
 * (slot, purpose, stream, step), key = seed, stream = stream_base + b * n_kv_heads + j for
 * sequence b and KV head j: a fit is a pure function of its arguments.
 *   n_centres_host   host int32 [n_seqs], in: k of sequence b, 1 <= k <= prompt_len[b]
 *                    (santapp_kmeans_parent_count gives the paper's choice)
 *   k_prompt         device [n_kv_heads][rows_total][d], token order, in
 *   centres          device fp32 [n_kv_heads][sum_b k_b][d], out (the fp64 centres rounded to nearest);
 *                    the layout santapp_assign_parents takes
 *   steps_run        device int32 [n_kv_heads][n_seqs] or NULL, out: minibatch steps each fit ran
 *   workspace        device, >= santapp_kmeans_fit_workspace_bytes(...)
 * batch_size > 4096, or an initialisation sample above 28544 keys (more than 9514 centres in a
 * sequence): SANTAPP_ERR_UNSUPPORTED. The call enqueues a few kernels per centre and per
 * step on `stream`. By default it waits for the stream every 16 steps to learn whether any fit
 * is still running (most stop long before the step limit), so it blocks the calling thread for
 * most of the fit; with opts->no_host_poll = 1 it never waits and enqueues every step up to the
 * limit instead (the result is the same: a stopped fit's later steps do nothing). In that mode the
 * call may be issued during a stream capture and the graph replayed: the per-sequence tables made
 * from the host arrays travel inside kernel arguments, nothing is copied from host memory. (The
 * other preparation calls that take host arrays -- the builders and santapp_assign_parents -- copy
 * their tables from host memory that is gone when they return: they must not be captured.)
 */
typedef struct santapp_kmeans_opts {
    int32_t batch_size;           /* paper: 4096 */
    int32_t max_iter;             /* paper: 100 */
    int32_t patience;             /* paper: 10 */
    int32_t no_host_poll;         /* 0: the call looks at the fits' stop flags every 16 steps (and waits for
                                     the stream to do so); 1: it never waits: every step up to the limit is
                                     enqueued, steps of a fit that has stopped return at once */
    double reassignment_ratio;    /* paper: 0.01; 0 switches reassignment off */
    uint64_t seed;                /* paper: 0 */
    uint32_t stream_base;
    uint32_t reserved2;           /* set to 0 */
} santapp_kmeans_opts;
size_t santapp_kmeans_fit_workspace_bytes(const santapp_geom *geom, const int32_t *prompt_len_host,
                                          const int32_t *n_centres_host, const santapp_kmeans_opts *opts);
int santapp_kmeans_fit(const santapp_geom *geom, const int32_t *prompt_len_host,
                       const int32_t *n_centres_host, const void *k_prompt,
                       const santapp_kmeans_opts *opts, float *centres, int32_t *steps_run,
                       void *workspace, size_t workspace_bytes, santapp_stream stream);

/*
 * Algorithm 3, the assignment that follows the fit: every key joins its nearest centre, squared
 * Euclidean distance evaluated in fp64 on the raw keys, ties going to the smaller centre index.
 * The centres are an input: santapp_kmeans_fit's output, or any other clustering's.
 *   n_centres_host   host int32 [n_seqs], in: centres of sequence b (>= 1), the same for every KV head
 *   k_prompt         device bf16 [n_kv_heads][rows_total][d], token order, in
 *   centres          device fp32 [n_kv_heads][sum_b n_centres[b]][d], in: sequence b's centres
 *                    start at the sum of the earlier sequences' counts
 *   parent_of        device int32 [n_kv_heads][rows_total], out: centre index (local to the
 *                    sequence) of each token; a centre that attracts no token simply does not occur
 *   workspace        device, >= santapp_assign_parents_workspace_bytes(geom) (offset tables)
 */
size_t santapp_assign_parents_workspace_bytes(const santapp_geom *geom);
int santapp_assign_parents(const santapp_geom *geom, const int32_t *prompt_len_host,
                           const int32_t *n_centres_host, const void *k_prompt, const float *centres,
                           int32_t *parent_of, void *workspace, size_t workspace_bytes,
                           santapp_stream stream);

/*
 * Sizes for team records built from an arbitrary parent partition: sequence b, whose tokens carry
 * parent labels in [0, n_parents[b]), gets min(prompt_len[b], n_parents[b] * R) team slots per KV
 * head (a parent of c tokens yields min(R, c) teams; empty parents yield none).
 * geom->parent_size is not used by the parent-based calls beyond the general checks.
 */
int santapp_parent_teams_sizes(const santapp_geom *geom, const int32_t *prompt_len_host,
                               const int32_t *n_parents_host, santapp_sizes *out);

/*
 * Build the team records of one layer from a given parent partition (the partition Algorithm 3
 * returns, or any other): Algorithm 2 on parents of any size. Parents are ordered by label, labels
 * without a token are omitted, and each (sequence, KV head) has its own partition, so the number of
 * teams may differ between the KV heads of a sequence: teams->team_count (required here) receives
 * it, and unused slots are left as empty teams.
 *   n_parents_host   host int32 [n_seqs], in: size of sequence b's label range (>= 1)
 *   parent_of        device int32 [n_kv_heads][rows_total], in: label of each token, local to its
 *                    sequence; values outside [0, n_parents[b]) are clamped into the range
 *   teams, workspace as for santapp_build_teams, with sizes from santapp_parent_teams_sizes
 * Arithmetic, tie rules and the packed layout are those of santapp_build_teams.
 */
int santapp_build_teams_parents(const santapp_geom *geom, const int32_t *prompt_len_host,
                                const int32_t *n_parents_host, const void *k_prompt,
                                const void *v_prompt, const int32_t *parent_of, santapp_teams *teams,
                                void *workspace, size_t workspace_bytes, santapp_stream stream);

/*
 * Centroid-guided groups on a given parent partition (the paper's baseline forms its groups by
 * k-means): as santapp_build_groups_mean, but one group per non-empty parent of `parent_of`, in label
 * order, members in token order. geom->reps_per_parent must be 1. Arguments,
 * sizes (santapp_parent_teams_sizes) and errors as for santapp_build_teams_parents.
 */
int santapp_build_groups_mean_parents(const santapp_geom *geom, const int32_t *prompt_len_host,
                                      const int32_t *n_parents_host, const void *k_prompt,
                                      const void *v_prompt, const int32_t *parent_of,
                                      santapp_teams *teams, void *workspace, size_t workspace_bytes,
                                      santapp_stream stream);

/* Workspace bytes santapp_decode_attn needs for n_sample = K on these team records. */
size_t santapp_decode_workspace_bytes(const santapp_geom *geom, const santapp_teams *teams,
                                      int32_t n_sample);

/*
 * One decode step of SANTA++ attention for all sequences and query heads (Algorithm 1).
 * Per query head h of sequence b, with the M_b teams of its KV head:
 *   K <- min(n_sample, M_b). If K = M_b every team is read with c_g = 1 and nothing is drawn.
 *   Otherwise phi_g = log n_g + q.l_g * scale (Eq. method-routing), Y_g = phi_g + Gumbel draw,
 *   S = the K largest Y (ties to the smaller team id), tau = the (K+1)-st largest,
 *   c_g = 1 - exp(-exp(phi_g - tau)) (Eq. method-inclusion). The sample is the fp64 one: an
 *   fp32 pass over all teams only narrows the field to the teams whose exact fp64 score can
 *   still be among the K+1 largest, and those are re-evaluated and ranked in fp64.
 *   out = U^ / Z^ of Eq. (method-estimate): every member of every selected team enters with
 *   weight e^{s_i} / c_g, every suffix row with weight e^{s_i}, s_i = q.k_i * scale
 *   (bf16 inputs, fp32 accumulation). Heads sharing a KV head sample independently; K/V rows
 *   of the union of their selections are read once.
 *   teams           host struct of device pointers, in
 *   q               device bf16 [n_seqs][n_q_heads][d], in (unscaled, post-RoPE)
 *   k_suffix,v_suffix device bf16 [n_seqs][n_kv_heads][suffix_cap][d], in: exact suffix of
 *                   generated tokens; may be NULL when suffix_cap == 0
 *   suffix_len_dev  device int32 [n_seqs], in: visible suffix rows per sequence (clamped to
 *                   [0, suffix_cap]); NULL means 0 everywhere
 *   n_sample        1 <= K <= 128, and (query heads per KV head) * min(K, M_b) <= 1024
 *                   (SANTAPP_ERR_UNSUPPORTED beyond; likewise for more than 65535 (sequence, KV
 *                   head) pairs in one call or more than 65536 teams in a sequence)
 *   seed, step, stream_base   random-stream key and counters (see top of file)
 *   step_dev        device uint32 [1] or NULL: when given, its value is added to `step` on the
 *                   device, so a captured CUDA graph can be replayed for successive tokens
 *   scale           logit scale; 0 means 1 / sqrt(d)
 *   out             device fp32 [n_seqs][n_q_heads][d], out
 *   dbg             host struct of device pointers or NULL
 *   workspace       device, >= santapp_decode_workspace_bytes(...); contents undefined on entry
 *                   and on exit; must not be shared by calls that may overlap on the GPU
 */
int santapp_decode_attn(const santapp_geom *geom, const santapp_teams *teams, const void *q,
                        const void *k_suffix, const void *v_suffix, const int32_t *suffix_len_dev,
                        int32_t suffix_cap, int32_t n_sample, uint64_t seed, uint32_t step,
                        const uint32_t *step_dev, uint32_t stream_base, float scale, float *out,
                        const santapp_debug *dbg, void *workspace, size_t workspace_bytes,
                        santapp_stream stream);

/* Workspace bytes santapp_dense_decode_attn needs. */
size_t santapp_dense_workspace_bytes(const santapp_geom *geom, const santapp_teams *teams);

/*
 * Dense decode attention, Eq. (method-attention), over all prompt rows (read from the packed
 * copy; attention does not depend on row order) and the visible suffix, for all sequences and
 * query heads. Arguments as in santapp_decode_attn.
 */
int santapp_dense_decode_attn(const santapp_geom *geom, const santapp_teams *teams, const void *q,
                              const void *k_suffix, const void *v_suffix,
                              const int32_t *suffix_len_dev, int32_t suffix_cap, float scale,
                              float *out, void *workspace, size_t workspace_bytes,
                              santapp_stream stream);

/*
 * Dense decode attention for callers that cannot hand the library a workspace. (The paper has
 * no counterpart: this entry point exists for deployment reasons only.)
 *
 * Who needs it: code that has no way to obtain device memory at the point of the call. Examples
 * are a serving loop whose device memory was handed over in full to another component's pool,
 * a plug-in host that forbids CUDA allocation calls inside its callbacks, and latency-critical
 * paths that must not run into the device-wide synchronisation an allocation can cause. For
 * them the scratch memory santapp_dense_decode_attn would take as `workspace` lives inside the
 * library: one array of SANTAPP_STATIC_SCRATCH_BYTES bytes in device global memory, part of
 * the library image, so every GPU that loads the library holds it until the process exits.
 * The call makes no allocation of any kind (no cudaMalloc, cudaFree, or allocating library
 * routine); inputs and outputs are still the caller's buffers.
 *
 * Computes exactly what santapp_dense_decode_attn computes, with the same arguments minus the
 * workspace pair.
 *   - Limit: if santapp_dense_workspace_bytes(geom, teams) exceeds SANTAPP_STATIC_SCRATCH_BYTES
 *     the call returns SANTAPP_ERR_STATIC_SCRATCH and launches nothing (the text of
 *     santapp_last_cuda_error says how many bytes were needed). On a 148-SM GPU with 7 query
 *     heads per KV head the 2 MiB array covers about 110 (sequence, KV head) pairs.
 *   - Set-up: the first call on each device looks up the array's device address (the device
 *     must be current, as for every call) and remembers it for the life of the process. Make
 *     that first call outside any stream capture. The remembered address belongs to the
 *     device's context: after a cudaDeviceReset it is stale, and the library must be reloaded
 *     before this entry point is used again on that device.
 *   - Sharing: every call on a device uses the same array, which keeps whatever the previous
 *     call left in it. Nothing in it has to be cleared between calls: the kernels write every
 *     table they read, and there are no counters. Two calls that can overlap on the GPU (different
 *     streams without an ordering between them) race on the array and must not be issued.
 */
#define SANTAPP_STATIC_SCRATCH_BYTES (2u << 20)
int santapp_dense_decode_attn_noalloc(const santapp_geom *geom, const santapp_teams *teams,
                                      const void *q, const void *k_suffix, const void *v_suffix,
                                      const int32_t *suffix_len_dev, int32_t suffix_cap,
                                      float scale, float *out, santapp_stream stream);

/*
 * Launch statistics of the most recent decode / dense call on this thread (host-side
 * bookkeeping, no device access): number of kernels launched by that call.
 */
int santapp_last_launch_count(void);

/*
 * Diagnostic: choose which stages the following santapp_decode_attn calls on this thread
 * launch, for timing one stage in isolation (the paper's "isolated-stage measurements").
 * Bit 0: representative scoring and perturbation; bit 1: sampling per query head, and the
 * read plans as a kernel of their own for batches of many (sequence, KV head) pairs (for few
 * pairs the union of the heads' samples is the first phase of the attention kernel);
 * bit 2: exact attention (each block leaves a partial result); bit 3: the merge of the partials
 * into the output. A stage that is skipped reuses what an earlier full call with the same
 * arguments left in the same workspace. The default, and the only setting that computes a
 * decode step, is SANTAPP_STAGE_ALL.
 */
enum { SANTAPP_STAGE_ROUTE = 1, SANTAPP_STAGE_SELECT = 2, SANTAPP_STAGE_ATTEND = 4, SANTAPP_STAGE_MERGE = 8,
       SANTAPP_STAGE_ALL = 15 };
void santapp_set_stage_mask(int mask);

#ifdef __cplusplus
}
#endif
#endif /* SANTAPP_H */
