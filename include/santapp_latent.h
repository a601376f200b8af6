/*
 * santapp_latent.h — C ABI of the shared-latent variant of the SANTA++ decode step (sm_100a).
 *
 * The paper's appendix "Token sparsity after latent compression" applies Algorithm 1 to a cache
 * that stores ONE row per token, shared by all query heads: a content latent (512 values)
 * followed by a rotary-position key (64 values), bf16. Teams are formed once per layer from the
 * content latents alone and are shared by the heads; every head scores a team's representative
 * with its own (absorbed) query against the representative's whole row, draws its own sample and
 * keeps its own inclusion corrections; a row is read when ANY head selected its team (the union
 * of Eq. (mla-logical-access)); a head's logit against a row is its query against the whole row,
 * its value the row's latent part. The paper reports this variant by logical access only and
 * names no kernel for it; the entry points here are the same three operations as in santapp.h
 * for that row format:
 *
 *   santapp_latent_build_teams        contiguous parents (Algorithm 4) and Algorithm 2 on the
 *                                     content latents, rows packed team by team
 *   santapp_latent_decode_attn        Algorithm 1 for all heads of all sequences, union over heads
 *   santapp_latent_dense_decode_attn  Eq. (method-attention) over all rows: the dense baseline
 *
 * Conventions are those of santapp.h (device / host pointers, caller-owned buffers and
 * workspaces that need no initialisation, asynchronous on `stream`, negative santapp_status on
 * error, argument errors found on the host before any launch, the Philox stream with the query
 * head index in the counter and stream = stream_base + sequence index). Status values, the
 * stream type and santapp_debug come from santapp.h.
 */
#ifndef SANTAPP_LATENT_H
#define SANTAPP_LATENT_H

#include "santapp.h"

#ifdef __cplusplus
extern "C" {
#endif

#define SANTAPP_LATENT_DIM 512          /* content latent values per row                         */
#define SANTAPP_LATENT_ROPE_DIM 64      /* rotary key values per row                             */
#define SANTAPP_LATENT_ROW 576          /* values per stored row                                 */
#define SANTAPP_LATENT_MAX_HEADS 16     /* query heads sharing a row                             */
#define SANTAPP_LATENT_MAX_PARENT 32    /* parent size P                                         */

/* Geometry (host struct). */
typedef struct santapp_latent_geom {
    int32_t n_seqs;            /* B                                                              */
    int32_t n_heads;           /* query heads that share every row: 1..16                        */
    int32_t parent_size;       /* P <= 32 (the paper's study uses 16)                            */
    int32_t reps_per_parent;   /* R, divides P (the paper's study uses 4)                        */
} santapp_latent_geom;

/*
 * Team records of one layer (device pointers, caller-allocated, immutable after the build).
 * Element counts come from santapp_latent_sizes.
 */
typedef struct santapp_latent_teams {
    void *rows_packed;         /* bf16 [rows_total][576]: each team's members contiguous, teams in
                                  id order, members by token index                               */
    void *rep_rows;            /* bf16 [teams_total][576]: the representatives' rows (frozen
                                  routing keys); 32-byte aligned (the scorer reads 32 bytes at a
                                  time), every other array as in santapp.h                       */
    int32_t *team_row_start;   /* int32 [teams_total + n_seqs]: sequence b's M_b + 1 CSR offsets
                                  start at seq_team_off[b] + b; values are local to the sequence */
    int32_t *row_token;        /* int32 [rows_total]: token index (local) of each packed row      */
    int64_t *seq_row_off;      /* int64 [n_seqs + 1]                                              */
    int64_t *seq_team_off;     /* int64 [n_seqs + 1]                                              */
    float *rep_abs_max;        /* fp32 [n_seqs]: largest |value| among a sequence's representative
                                  rows (bounds the fp32 routing pass)                            */
    int64_t rows_total;        /* host scalars                                                    */
    int64_t teams_total;
    int32_t max_teams_per_seq;
    int32_t max_rows_per_seq;
} santapp_latent_teams;

/* rows_total, teams_total, the maxima, and the build workspace (santapp_sizes, with
 * team_row_start_elems = teams_total + n_seqs). prompt_len_host: host int32 [n_seqs], each >= 1. */
int santapp_latent_sizes(const santapp_latent_geom *geom, const int32_t *prompt_len_host,
                         santapp_sizes *out);

/*
 * Algorithm 4 and Algorithm 2 on the content latents (columns 0..511 of each row; the rotary
 * columns take no part in distances or means): arithmetic, tie rules and team numbering as in
 * santapp_build_teams (fp64 distances in a fixed order).
 *   rows_prompt   device bf16 [rows_total][576], token order, in
 *   teams         out: every array overwritten, host scalars filled in
 *   workspace     device, >= sizes.build_workspace_bytes
 */
int santapp_latent_build_teams(const santapp_latent_geom *geom, const int32_t *prompt_len_host,
                               const void *rows_prompt, santapp_latent_teams *teams,
                               void *workspace, size_t workspace_bytes, santapp_stream stream);

size_t santapp_latent_decode_workspace_bytes(const santapp_latent_geom *geom,
                                             const santapp_latent_teams *teams, int32_t n_sample,
                                             int32_t suffix_cap);

/*
 * One decode step (Algorithm 1 per head; the sample is the fp64 one, obtained as in
 * santapp_decode_attn: an fp32 tensor-core pass over all representatives narrows the field, the
 * candidates are re-evaluated and ranked in fp64).
 *   q             device bf16 [n_seqs][n_heads][576]: each head's query against a whole row
 *   suffix_rows   device bf16 [n_seqs][suffix_cap][576] or NULL when suffix_cap == 0: rows of the
 *                 generated tokens, attended exactly by every head
 *   suffix_len_dev device int32 [n_seqs] or NULL (= 0): visible suffix rows, clamped to [0, suffix_cap]
 *   n_sample      1 <= K <= 256 teams per head (the paper's budgets S = 128, 256, 512, 1024 with
 *                 P = 16, R = 4 are K = 32, 64, 128, 256)
 *   scale         logit scale, > 0 (the model's; there is no default for this row format)
 *   out           device fp32 [n_seqs][n_heads][512]
 *   dbg           as in santapp_decode_attn with n_q_heads = n_heads and one KV head; `trace` is
 *                 not written
 * More than 4096 sequences in one call or more than 65536 teams in a sequence:
 * SANTAPP_ERR_UNSUPPORTED.
 */
int santapp_latent_decode_attn(const santapp_latent_geom *geom, const santapp_latent_teams *teams,
                               const void *q, const void *suffix_rows, const int32_t *suffix_len_dev,
                               int32_t suffix_cap, int32_t n_sample, uint64_t seed, uint32_t step,
                               const uint32_t *step_dev, uint32_t stream_base, float scale, float *out,
                               const santapp_debug *dbg, void *workspace, size_t workspace_bytes,
                               santapp_stream stream);

size_t santapp_latent_dense_workspace_bytes(const santapp_latent_geom *geom,
                                            const santapp_latent_teams *teams);

/* Dense attention of every head over every row of its sequence and the visible suffix. */
int santapp_latent_dense_decode_attn(const santapp_latent_geom *geom, const santapp_latent_teams *teams,
                                     const void *q, const void *suffix_rows,
                                     const int32_t *suffix_len_dev, int32_t suffix_cap, float scale,
                                     float *out, void *workspace, size_t workspace_bytes,
                                     santapp_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* SANTAPP_LATENT_H */
