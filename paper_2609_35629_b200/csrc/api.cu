// C ABI of the SANTA++ decode-attention library: argument checks, workspace carving, launches.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "common.cuh"

using namespace santapp;

namespace {

thread_local char g_cuda_error[256] = "";
thread_local int g_launches = 0;
thread_local int g_stage_mask = SANTAPP_STAGE_ALL;

int cuda_fail(cudaError_t err, const char *where)
{
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", where, cudaGetErrorString(err));
    return SANTAPP_ERR_CUDA;
}

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

}  // namespace

// The same bookkeeping for entry points that live in other files.
namespace santapp {
int note_cuda_failure(cudaError_t err, const char *where) { return cuda_fail(err, where); }
void note_launch_count(int n) { g_launches = n; }
int current_stage_mask() { return g_stage_mask; }
}  // namespace santapp

namespace {

// Device arrays are read and written 16 bytes at a time (8 for the 64-bit offsets, 4 for the 32-bit
// tables): a pointer that is not aligned accordingly would fault on the device, so it is refused here.
inline bool misaligned(const void *p, size_t a) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) % a) != 0; }

int check_geom(const santapp_geom *g)
{
    if (!g) return SANTAPP_ERR_INVALID_ARG;
    if (g->n_seqs < 1 || g->n_q_heads < 1 || g->n_kv_heads < 1 || g->parent_size < 1 || g->reps_per_parent < 1)
        return SANTAPP_ERR_INVALID_ARG;
    if (g->n_q_heads % g->n_kv_heads != 0) return SANTAPP_ERR_INVALID_ARG;
    if (g->elem_type != SANTAPP_BF16 && g->elem_type != SANTAPP_FP16) return SANTAPP_ERR_INVALID_ARG;
    if (g->parent_size % g->reps_per_parent != 0) return SANTAPP_ERR_INVALID_ARG;   // R divides P
    if (g->head_dim != kHeadDim) return SANTAPP_ERR_UNSUPPORTED;
    if (g->n_q_heads / g->n_kv_heads > kMaxGroup) return SANTAPP_ERR_UNSUPPORTED;
    if (g->parent_size > kMaxParent) return SANTAPP_ERR_UNSUPPORTED;
    return SANTAPP_OK;
}

int teams_in_sequence(int N, int P, int R)
{
    const int full = N / P, tail = N % P;
    return full * (R < P ? R : P) + (tail ? (R < tail ? R : tail) : 0);
}

int check_teams(const santapp_geom *g, const santapp_teams *t)
{
    if (!t) return SANTAPP_ERR_INVALID_ARG;
    if (!t->k_packed || !t->v_packed || !t->rep_keys || !t->team_row_start || !t->seq_row_off || !t->seq_team_off
        || !t->rep_abs_max)
        return SANTAPP_ERR_INVALID_ARG;
    if (misaligned(t->k_packed, 16) || misaligned(t->v_packed, 16) || misaligned(t->rep_keys, 16)
        || misaligned(t->team_row_start, 4) || misaligned(t->row_token, 4) || misaligned(t->seq_row_off, 8)
        || misaligned(t->seq_team_off, 8) || misaligned(t->rep_abs_max, 4) || misaligned(t->team_count, 4))
        return SANTAPP_ERR_INVALID_ARG;
    if (t->rows_total < g->n_seqs || t->teams_total < g->n_seqs || t->max_teams_per_seq < 1)
        return SANTAPP_ERR_INVALID_ARG;
    if (t->rows_total >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    if (t->max_teams_per_seq > kMaxTeamsPerSeq) return SANTAPP_ERR_UNSUPPORTED;
    return SANTAPP_OK;
}

BatchView make_view(const santapp_geom *g, const santapp_teams *t)
{
    BatchView bv;
    bv.n_seqs = g->n_seqs;
    bv.n_q = g->n_q_heads;
    bv.n_kv = g->n_kv_heads;
    bv.group = g->n_q_heads / g->n_kv_heads;
    bv.seq_row_off = t->seq_row_off;
    bv.seq_team_off = t->seq_team_off;
    bv.team_count = t->team_count;
    bv.elem = g->elem_type;
    bv.rows_total = t->rows_total;
    bv.teams_total = t->teams_total;
    return bv;
}

// Workspace layout shared by the sparse and the dense call. Offsets in bytes.
struct DecodeLayout {
    size_t counter, y32, sel_team, sel_logc, sel_rows, seg_prefix, seg_row, seg_mask, seg_logc, pair_nseg, pair_rows, pair_prefix, partials, total;
    int seg_cap, grid, n_pairs, ctas_per_pair, tile_stride;
    int64_t y_stride;
    bool static_split;
};

DecodeLayout decode_layout(const santapp_geom *g, const santapp_teams *t, int K, bool dense, int grid)
{
    DecodeLayout L;
    const int G = g->n_q_heads / g->n_kv_heads;
    L.n_pairs = g->n_seqs * g->n_kv_heads;
    L.grid = grid;
    // few pairs: a fixed number of CTAs per pair and the plan built inside the attention kernel;
    // many pairs: equal row ranges over a plan in global memory
    int static_factor = 9;
#ifdef SANTAPP_TUNE
    if (const char *e = getenv("SANTAPP_STATIC_FACTOR")) static_factor = atoi(e);
#endif
    L.static_split = (int64_t)L.n_pairs * static_factor <= grid;
    L.ctas_per_pair = L.static_split ? grid / L.n_pairs : 1;
    int64_t cap = dense ? 1 : (int64_t)G * K;
    if (cap > t->max_teams_per_seq) cap = t->max_teams_per_seq;
    L.seg_cap = (int)cap + 1;                                   // + the suffix segment
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    L.counter = take(sizeof(int32_t) * 2);
    L.y_stride = score_row_stride(t->max_teams_per_seq);
    L.y32 = take(dense ? 0 : sizeof(float) * (size_t)g->n_q_heads * (size_t)g->n_seqs * (size_t)L.y_stride);
    L.tile_stride = (int)(t->teams_total / 16 + g->n_seqs + 1);
    L.sel_team = take(dense ? 0 : sizeof(int32_t) * (size_t)g->n_seqs * g->n_q_heads * K);
    L.sel_logc = take(dense ? 0 : sizeof(float) * (size_t)g->n_seqs * g->n_q_heads * K);
    L.sel_rows = take(dense ? 0 : sizeof(int2) * (size_t)g->n_seqs * g->n_q_heads * K);
    L.seg_prefix = take(sizeof(int32_t) * (size_t)L.n_pairs * (L.seg_cap + 1));
    L.seg_row = take(sizeof(int32_t) * (size_t)L.n_pairs * L.seg_cap);
    L.seg_mask = take(sizeof(uint32_t) * (size_t)L.n_pairs * L.seg_cap);
    L.seg_logc = take(sizeof(float) * (size_t)L.n_pairs * L.seg_cap * kMaxGroup);
    L.pair_nseg = take(sizeof(int32_t) * (size_t)L.n_pairs);
    L.pair_rows = take(sizeof(int32_t) * (size_t)L.n_pairs);
    L.pair_prefix = take(sizeof(int64_t) * ((size_t)L.n_pairs + 1));
    // one partial per (block or tail chunk, pair it touches)
    L.partials = take(sizeof(float) * ((size_t)grid * (1 + kMaxTailChunksPerBlock) + 1 + L.n_pairs) * G * kPartialStride);
    L.total = off;
    return L;
}

void fill_plan(const DecodeLayout &L, char *ws, PlanView &plan)
{
    plan.seg_cap = L.seg_cap;
    plan.seg_prefix = reinterpret_cast<int32_t *>(ws + L.seg_prefix);
    plan.seg_row = reinterpret_cast<int32_t *>(ws + L.seg_row);
    plan.seg_mask = reinterpret_cast<uint32_t *>(ws + L.seg_mask);
    plan.seg_logc = reinterpret_cast<float *>(ws + L.seg_logc);
    plan.pair_nseg = reinterpret_cast<int32_t *>(ws + L.pair_nseg);
    plan.pair_rows = reinterpret_cast<int32_t *>(ws + L.pair_rows);
    plan.pair_union_rows = nullptr;
    plan.pair_row_prefix = reinterpret_cast<int64_t *>(ws + L.pair_prefix);
    plan.tail_counter = reinterpret_cast<int32_t *>(ws + L.counter);
}

}  // namespace

extern "C" {

int santapp_version(void) { return 100; }

const char *santapp_strerror(int status)
{
    switch (status) {
        case SANTAPP_OK: return "ok";
        case SANTAPP_ERR_INVALID_ARG: return "invalid argument";
        case SANTAPP_ERR_UNSUPPORTED: return "unsupported configuration";
        case SANTAPP_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case SANTAPP_ERR_CUDA: return "CUDA error";
        case SANTAPP_ERR_STATIC_SCRATCH: return "problem needs more scratch than the built-in array holds";
        default: return "unknown status";
    }
}

const char *santapp_last_cuda_error(void) { return g_cuda_error; }

int santapp_last_launch_count(void) { return g_launches; }

void santapp_set_stage_mask(int mask) { g_stage_mask = mask & SANTAPP_STAGE_ALL; }

int santapp_build_teams_sizes(const santapp_geom *geom, const int32_t *prompt_len_host, santapp_sizes *out)
{
    int rc = check_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if (!prompt_len_host || !out) return SANTAPP_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    for (int b = 0; b < geom->n_seqs; ++b) {
        const int N = prompt_len_host[b];
        if (N < 1) return SANTAPP_ERR_INVALID_ARG;
        const int M = teams_in_sequence(N, geom->parent_size, geom->reps_per_parent);
        out->rows_total += N;
        out->teams_total += M;
        if (M > out->max_teams_per_seq) out->max_teams_per_seq = M;
        if (N > out->max_rows_per_seq) out->max_rows_per_seq = N;
    }
    if (out->rows_total >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    out->team_row_start_elems = (int64_t)geom->n_kv_heads * (out->teams_total + geom->n_seqs);
    out->build_workspace_bytes = align_up(sizeof(uint16_t) * (size_t)geom->n_kv_heads * (size_t)out->rows_total);
    return SANTAPP_OK;
}

}  // extern "C"

namespace {

// Both builders: checks, offset tables, host scalars, then the kernels of the chosen grouping.
int build_records(const santapp_geom *geom, const int32_t *prompt_len_host, const void *k_prompt,
                  const void *v_prompt, santapp_teams *teams, void *workspace, size_t workspace_bytes,
                  santapp_stream stream, bool mean_groups)
{
    santapp_sizes sz;
    int rc = santapp_build_teams_sizes(geom, prompt_len_host, &sz);
    if (rc != SANTAPP_OK) return rc;
    if (!k_prompt || !v_prompt || !teams || !workspace) return SANTAPP_ERR_INVALID_ARG;
    if (!teams->k_packed || !teams->v_packed || !teams->rep_keys || !teams->team_row_start || !teams->row_token
        || !teams->seq_row_off || !teams->seq_team_off || !teams->rep_abs_max)
        return SANTAPP_ERR_INVALID_ARG;
    if (misaligned(k_prompt, 16) || misaligned(v_prompt, 16) || misaligned(workspace, 16)
        || misaligned(teams->k_packed, 16) || misaligned(teams->v_packed, 16) || misaligned(teams->rep_keys, 16)
        || misaligned(teams->team_row_start, 4) || misaligned(teams->row_token, 4) || misaligned(teams->seq_row_off, 8)
        || misaligned(teams->seq_team_off, 8) || misaligned(teams->rep_abs_max, 4)
        || misaligned(teams->team_count, 4))
        return SANTAPP_ERR_INVALID_ARG;
    if (workspace_bytes < sz.build_workspace_bytes) return SANTAPP_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    g_cuda_error[0] = 0;

    std::vector<int64_t> offs(2 * ((size_t)geom->n_seqs + 1));
    int64_t *row_off = offs.data(), *team_off = offs.data() + geom->n_seqs + 1;
    row_off[0] = team_off[0] = 0;
    int max_parents = 0;
    for (int b = 0; b < geom->n_seqs; ++b) {
        const int N = prompt_len_host[b];
        row_off[b + 1] = row_off[b] + N;
        team_off[b + 1] = team_off[b] + teams_in_sequence(N, geom->parent_size, geom->reps_per_parent);
        const int parents = (N + geom->parent_size - 1) / geom->parent_size;
        if (parents > max_parents) max_parents = parents;
    }
    const size_t ob = sizeof(int64_t) * ((size_t)geom->n_seqs + 1);
    cudaError_t err = cudaMemcpyAsync(teams->seq_row_off, row_off, ob, cudaMemcpyHostToDevice, s);
    if (err != cudaSuccess) return cuda_fail(err, "copy seq_row_off");
    err = cudaMemcpyAsync(teams->seq_team_off, team_off, ob, cudaMemcpyHostToDevice, s);
    if (err != cudaSuccess) return cuda_fail(err, "copy seq_team_off");

    teams->rows_total = sz.rows_total;
    teams->teams_total = sz.teams_total;
    teams->max_teams_per_seq = sz.max_teams_per_seq;
    teams->max_rows_per_seq = sz.max_rows_per_seq;

    BuildParams p;
    p.bv = make_view(geom, teams);
    p.parent_size = geom->parent_size;
    p.reps = geom->reps_per_parent;
    p.teams_per_full_parent = geom->reps_per_parent < geom->parent_size ? geom->reps_per_parent : geom->parent_size;
    p.k_prompt = static_cast<const uint16_t *>(k_prompt);
    p.v_prompt = static_cast<const uint16_t *>(v_prompt);
    p.k_packed = static_cast<uint16_t *>(teams->k_packed);
    p.v_packed = static_cast<uint16_t *>(teams->v_packed);
    p.rep_keys = static_cast<uint16_t *>(teams->rep_keys);
    p.team_row_start = teams->team_row_start;
    p.row_token = teams->row_token;
    p.team_count = teams->team_count;
    p.owner = static_cast<uint16_t *>(workspace);
    p.max_parents_per_seq = max_parents;
    err = mean_groups ? launch_build_groups_mean(p, s) : launch_build_teams(p, s);
    if (err != cudaSuccess) return cuda_fail(err, "build launch");
    err = launch_rep_abs_max(p.bv, p.rep_keys, teams->rep_abs_max, s);
    if (err != cudaSuccess) return cuda_fail(err, "rep_abs_max launch");
    return SANTAPP_OK;
}

}  // namespace

namespace {

// Workspace of santapp_build_teams_parents. Offsets in bytes.
struct ParentLayout {
    size_t label_off, parent_start, parent_cursor, parent_team_base, members, team_of, mind, owner, is_rep,
        team_cursor, dest, total;
};

ParentLayout parent_layout(int n_seqs, int n_kv, int64_t rows_total, int64_t labels_total, int64_t teams_total)
{
    ParentLayout L;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    const size_t H = (size_t)n_kv, R = (size_t)rows_total, Lt = (size_t)labels_total;
    L.label_off = take(sizeof(int64_t) * ((size_t)n_seqs + 1));
    L.parent_start = take(sizeof(int32_t) * H * (Lt + (size_t)n_seqs));
    L.parent_cursor = take(sizeof(int32_t) * H * Lt);
    L.parent_team_base = take(sizeof(int32_t) * H * Lt);
    L.members = take(sizeof(int32_t) * H * R);
    L.team_of = take(sizeof(int32_t) * H * R);
    L.mind = take(sizeof(double) * H * R);
    L.owner = take(sizeof(int32_t) * H * R);
    L.is_rep = take(H * R);
    L.team_cursor = take(sizeof(int32_t) * H * (size_t)teams_total);
    L.dest = take(sizeof(int32_t) * H * R);
    L.total = off;
    return L;
}

}  // namespace

extern "C" {

int32_t santapp_kmeans_parent_count(int32_t prompt_len, int32_t parent_size)
{
    if (prompt_len < 2 || parent_size < 1) return 0;
    int32_t m = prompt_len / parent_size;
    if (m < 2) m = 2;
    if (m > prompt_len) m = prompt_len;
    return m;
}

size_t santapp_assign_parents_workspace_bytes(const santapp_geom *geom)
{
    if (check_geom(geom) != SANTAPP_OK) return 0;
    return 2 * align_up(sizeof(int64_t) * ((size_t)geom->n_seqs + 1));
}

int santapp_assign_parents(const santapp_geom *geom, const int32_t *prompt_len_host, const int32_t *n_centres_host,
                           const void *k_prompt, const float *centres, int32_t *parent_of, void *workspace,
                           size_t workspace_bytes, santapp_stream stream)
{
    int rc = check_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if (!prompt_len_host || !n_centres_host || !k_prompt || !centres || !parent_of || !workspace)
        return SANTAPP_ERR_INVALID_ARG;
    if (misaligned(k_prompt, 16) || misaligned(centres, 4) || misaligned(parent_of, 4) || misaligned(workspace, 16))
        return SANTAPP_ERR_INVALID_ARG;
    if (workspace_bytes < santapp_assign_parents_workspace_bytes(geom)) return SANTAPP_ERR_WORKSPACE_TOO_SMALL;
    std::vector<int64_t> offs(2 * ((size_t)geom->n_seqs + 1));
    int64_t *row_off = offs.data(), *cen_off = offs.data() + geom->n_seqs + 1;
    row_off[0] = cen_off[0] = 0;
    int max_rows = 0;
    for (int b = 0; b < geom->n_seqs; ++b) {
        if (prompt_len_host[b] < 1 || n_centres_host[b] < 1) return SANTAPP_ERR_INVALID_ARG;
        row_off[b + 1] = row_off[b] + prompt_len_host[b];
        cen_off[b + 1] = cen_off[b] + n_centres_host[b];
        if (prompt_len_host[b] > max_rows) max_rows = prompt_len_host[b];
    }
    if (row_off[geom->n_seqs] >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    g_cuda_error[0] = 0;
    const size_t ob = sizeof(int64_t) * ((size_t)geom->n_seqs + 1);
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    int64_t *d_row_off = reinterpret_cast<int64_t *>(ws);
    int64_t *d_cen_off = reinterpret_cast<int64_t *>(ws + align_up(ob));
    cudaError_t err = cudaMemcpyAsync(d_row_off, row_off, ob, cudaMemcpyHostToDevice, s);
    if (err != cudaSuccess) return cuda_fail(err, "copy row offsets");
    err = cudaMemcpyAsync(d_cen_off, cen_off, ob, cudaMemcpyHostToDevice, s);
    if (err != cudaSuccess) return cuda_fail(err, "copy centre offsets");
    AssignParams p;
    p.n_seqs = geom->n_seqs;
    p.n_kv = geom->n_kv_heads;
    p.elem = geom->elem_type;
    p.max_rows_per_seq = max_rows;
    p.rows_total = row_off[geom->n_seqs];
    p.centres_total = cen_off[geom->n_seqs];
    p.seq_row_off = d_row_off;
    p.seq_centre_off = d_cen_off;
    p.k_prompt = static_cast<const uint16_t *>(k_prompt);
    p.centres = centres;
    p.parent_of = parent_of;
    err = launch_assign_parents(p, s);
    if (err != cudaSuccess) return cuda_fail(err, "assign_parents launch");
    return SANTAPP_OK;
}

int santapp_parent_teams_sizes(const santapp_geom *geom, const int32_t *prompt_len_host, const int32_t *n_parents_host,
                               santapp_sizes *out)
{
    int rc = check_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if (!prompt_len_host || !n_parents_host || !out) return SANTAPP_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    int64_t labels_total = 0;
    for (int b = 0; b < geom->n_seqs; ++b) {
        const int N = prompt_len_host[b];
        if (N < 1 || n_parents_host[b] < 1) return SANTAPP_ERR_INVALID_ARG;
        const int64_t want = (int64_t)n_parents_host[b] * geom->reps_per_parent;
        const int M = (int)(want < N ? want : N);
        labels_total += n_parents_host[b];
        out->rows_total += N;
        out->teams_total += M;
        if (M > out->max_teams_per_seq) out->max_teams_per_seq = M;
        if (N > out->max_rows_per_seq) out->max_rows_per_seq = N;
    }
    if (out->rows_total >= (int64_t)1 << 31 || labels_total >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    out->team_row_start_elems = (int64_t)geom->n_kv_heads * (out->teams_total + geom->n_seqs);
    out->build_workspace_bytes =
        parent_layout(geom->n_seqs, geom->n_kv_heads, out->rows_total, labels_total, out->teams_total).total;
    return SANTAPP_OK;
}

static int build_parent_records(const santapp_geom *geom, const int32_t *prompt_len_host,
                                const int32_t *n_parents_host, const void *k_prompt, const void *v_prompt,
                                const int32_t *parent_of, santapp_teams *teams, void *workspace,
                                size_t workspace_bytes, santapp_stream stream, bool mean_keys)
{
    santapp_sizes sz;
    int rc = santapp_parent_teams_sizes(geom, prompt_len_host, n_parents_host, &sz);
    if (rc != SANTAPP_OK) return rc;
    if (!k_prompt || !v_prompt || !parent_of || !teams || !workspace) return SANTAPP_ERR_INVALID_ARG;
    if (!teams->k_packed || !teams->v_packed || !teams->rep_keys || !teams->team_row_start || !teams->row_token
        || !teams->seq_row_off || !teams->seq_team_off || !teams->rep_abs_max || !teams->team_count)
        return SANTAPP_ERR_INVALID_ARG;
    if (misaligned(k_prompt, 16) || misaligned(v_prompt, 16) || misaligned(workspace, 16) || misaligned(parent_of, 4)
        || misaligned(teams->k_packed, 16) || misaligned(teams->v_packed, 16) || misaligned(teams->rep_keys, 16)
        || misaligned(teams->team_row_start, 4) || misaligned(teams->row_token, 4) || misaligned(teams->seq_row_off, 8)
        || misaligned(teams->seq_team_off, 8) || misaligned(teams->rep_abs_max, 4)
        || misaligned(teams->team_count, 4))
        return SANTAPP_ERR_INVALID_ARG;
    if (workspace_bytes < sz.build_workspace_bytes) return SANTAPP_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    g_cuda_error[0] = 0;

    const int B = geom->n_seqs;
    std::vector<int64_t> offs(3 * ((size_t)B + 1));
    int64_t *row_off = offs.data(), *team_off = row_off + B + 1, *label_off = team_off + B + 1;
    row_off[0] = team_off[0] = label_off[0] = 0;
    int max_labels = 0;
    for (int b = 0; b < B; ++b) {
        const int N = prompt_len_host[b];
        const int64_t want = (int64_t)n_parents_host[b] * geom->reps_per_parent;
        row_off[b + 1] = row_off[b] + N;
        team_off[b + 1] = team_off[b] + (want < N ? want : N);
        label_off[b + 1] = label_off[b] + n_parents_host[b];
        if (n_parents_host[b] > max_labels) max_labels = n_parents_host[b];
    }
    const ParentLayout L = parent_layout(B, geom->n_kv_heads, sz.rows_total, label_off[B], sz.teams_total);
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    const size_t ob = sizeof(int64_t) * ((size_t)B + 1);
    cudaError_t err = cudaMemcpyAsync(teams->seq_row_off, row_off, ob, cudaMemcpyHostToDevice, s);
    if (err != cudaSuccess) return cuda_fail(err, "copy seq_row_off");
    err = cudaMemcpyAsync(teams->seq_team_off, team_off, ob, cudaMemcpyHostToDevice, s);
    if (err != cudaSuccess) return cuda_fail(err, "copy seq_team_off");
    err = cudaMemcpyAsync(ws + L.label_off, label_off, ob, cudaMemcpyHostToDevice, s);
    if (err != cudaSuccess) return cuda_fail(err, "copy label offsets");

    teams->rows_total = sz.rows_total;
    teams->teams_total = sz.teams_total;
    teams->max_teams_per_seq = sz.max_teams_per_seq;
    teams->max_rows_per_seq = sz.max_rows_per_seq;

    ParentBuildParams p;
    p.bv = make_view(geom, teams);
    p.reps = geom->reps_per_parent;
    p.mean_keys = mean_keys;
    p.max_labels_per_seq = max_labels;
    p.max_rows_per_seq = sz.max_rows_per_seq;
    p.labels_total = label_off[B];
    p.k_prompt = static_cast<const uint16_t *>(k_prompt);
    p.v_prompt = static_cast<const uint16_t *>(v_prompt);
    p.parent_of = parent_of;
    p.seq_label_off = reinterpret_cast<const int64_t *>(ws + L.label_off);
    p.k_packed = static_cast<uint16_t *>(teams->k_packed);
    p.v_packed = static_cast<uint16_t *>(teams->v_packed);
    p.rep_keys = static_cast<uint16_t *>(teams->rep_keys);
    p.team_row_start = teams->team_row_start;
    p.row_token = teams->row_token;
    p.team_count = teams->team_count;
    p.parent_start = reinterpret_cast<int32_t *>(ws + L.parent_start);
    p.parent_cursor = reinterpret_cast<int32_t *>(ws + L.parent_cursor);
    p.parent_team_base = reinterpret_cast<int32_t *>(ws + L.parent_team_base);
    p.members = reinterpret_cast<int32_t *>(ws + L.members);
    p.team_of = reinterpret_cast<int32_t *>(ws + L.team_of);
    p.mind = reinterpret_cast<double *>(ws + L.mind);
    p.owner = reinterpret_cast<int32_t *>(ws + L.owner);
    p.is_rep = ws + L.is_rep;
    p.team_cursor = reinterpret_cast<int32_t *>(ws + L.team_cursor);
    p.dest = reinterpret_cast<int32_t *>(ws + L.dest);
    err = launch_build_teams_parents(p, s);
    if (err != cudaSuccess) return cuda_fail(err, "build_teams_parents launch");
    err = launch_rep_abs_max(p.bv, p.rep_keys, teams->rep_abs_max, s);
    if (err != cudaSuccess) return cuda_fail(err, "rep_abs_max launch");
    return SANTAPP_OK;
}

int santapp_build_teams_parents(const santapp_geom *geom, const int32_t *prompt_len_host, const int32_t *n_parents_host,
                                const void *k_prompt, const void *v_prompt, const int32_t *parent_of,
                                santapp_teams *teams, void *workspace, size_t workspace_bytes, santapp_stream stream)
{
    return build_parent_records(geom, prompt_len_host, n_parents_host, k_prompt, v_prompt, parent_of, teams, workspace,
                                workspace_bytes, stream, false);
}

int santapp_build_groups_mean_parents(const santapp_geom *geom, const int32_t *prompt_len_host,
                                      const int32_t *n_parents_host, const void *k_prompt, const void *v_prompt,
                                      const int32_t *parent_of, santapp_teams *teams, void *workspace,
                                      size_t workspace_bytes, santapp_stream stream)
{
    if (geom && geom->reps_per_parent != 1) return SANTAPP_ERR_INVALID_ARG;    // one group per parent
    return build_parent_records(geom, prompt_len_host, n_parents_host, k_prompt, v_prompt, parent_of, teams, workspace,
                                workspace_bytes, stream, true);
}

}  // extern "C"

namespace {

constexpr int kKmeansMaxSample = 28544;     // 223 KB of fp64 running sums (plus their block offsets): up to 9514 centres per sequence

struct KmeansLayout {
    size_t row_off, cen_off, tabs, perm, closest, cand, part, pick, centres64, count, idx, label, dist, dist_part, label_part, sorted, state, active, total;
    int k_max, n_init_max, trials_max, t_max_max, max_rows, assign_split;
    int64_t rows_total, centres_total;
};

// Per-sequence quantities of the fit and the workspace that holds its state. Returns a status.
int kmeans_layout(const santapp_geom *geom, const int32_t *prompt_len_host, const int32_t *n_centres_host,
                  const santapp_kmeans_opts *o, KmeansLayout *L, std::vector<int32_t> *tabs)
{
    int rc = check_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if (!prompt_len_host || !n_centres_host || !o) return SANTAPP_ERR_INVALID_ARG;
    if (o->batch_size < 1 || o->max_iter < 1 || o->patience < 1 || !(o->reassignment_ratio >= 0.0))
        return SANTAPP_ERR_INVALID_ARG;
    if (o->batch_size > 4096) return SANTAPP_ERR_UNSUPPORTED;
    const int B = geom->n_seqs;
    memset(L, 0, sizeof(*L));
    if (tabs) tabs->assign(3 * (size_t)B, 0);
    for (int b = 0; b < B; ++b) {
        const int N = prompt_len_host[b], k = n_centres_host[b];
        if (N < 1 || k < 1 || k > N) return SANTAPP_ERR_INVALID_ARG;
        int64_t n_init = 3 * (int64_t)(o->batch_size > k ? o->batch_size : k);
        if (n_init > N) n_init = N;
        const int trials = 2 + (int)floor(log((double)k));
        const int64_t t_max = (int64_t)o->max_iter * ((N + o->batch_size - 1) / o->batch_size);
        if (t_max > INT32_MAX) return SANTAPP_ERR_UNSUPPORTED;
        if (tabs) { (*tabs)[b] = (int32_t)n_init; (*tabs)[B + b] = trials; (*tabs)[2 * B + b] = (int32_t)t_max; }
        L->rows_total += N;
        L->centres_total += k;
        if (k > L->k_max) L->k_max = k;
        if (n_init > L->n_init_max) L->n_init_max = (int)n_init;
        if (trials > L->trials_max) L->trials_max = trials;
        if (t_max > L->t_max_max) L->t_max_max = (int)t_max;
        if (N > L->max_rows) L->max_rows = N;
    }
    if (L->rows_total >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    if (L->n_init_max > kKmeansMaxSample) return SANTAPP_ERR_UNSUPPORTED;   // its running sums live in shared memory
    const size_t H = (size_t)geom->n_kv_heads, pairs = H * (size_t)B;
    if (pairs > 65535) return SANTAPP_ERR_UNSUPPORTED;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes); return at; };
    L->row_off = take(sizeof(int64_t) * ((size_t)B + 1));
    L->cen_off = take(sizeof(int64_t) * ((size_t)B + 1));
    L->tabs = take(sizeof(int32_t) * 3 * (size_t)B);
    L->perm = take(sizeof(int32_t) * H * (size_t)L->rows_total);
    L->closest = take(sizeof(double) * pairs * (size_t)L->n_init_max);
    L->cand = take(sizeof(double) * pairs * (size_t)L->trials_max * (size_t)L->n_init_max);
    L->part = take(sizeof(double) * pairs * (size_t)L->trials_max * (((size_t)L->n_init_max + 127) / 128));
    L->pick = take(sizeof(int32_t) * pairs * (size_t)L->trials_max);
    L->centres64 = take(sizeof(double) * H * (size_t)L->centres_total * kHeadDim);
    L->count = take(sizeof(double) * H * (size_t)L->centres_total);
    L->idx = take(sizeof(int32_t) * pairs * (size_t)o->batch_size);
    L->label = take(sizeof(int32_t) * pairs * (size_t)o->batch_size);
    L->dist = take(sizeof(double) * pairs * (size_t)o->batch_size);
    // the nearest-centre search of a minibatch is cut into slices of the centres (about 128 each, at most 16)
    L->assign_split = L->k_max / 128 < 1 ? 1 : (L->k_max / 128 > 16 ? 16 : L->k_max / 128);
    L->dist_part = take(sizeof(double) * pairs * (size_t)L->assign_split * (size_t)o->batch_size);
    L->label_part = take(sizeof(int32_t) * pairs * (size_t)L->assign_split * (size_t)o->batch_size);
    L->sorted = take(sizeof(uint32_t) * pairs * 4096);
    L->state = take(sizeof(KmeansState) * pairs);
    L->active = take(sizeof(int));
    L->total = off;
    return SANTAPP_OK;
}

}  // namespace

extern "C" {

size_t santapp_kmeans_fit_workspace_bytes(const santapp_geom *geom, const int32_t *prompt_len_host,
                                          const int32_t *n_centres_host, const santapp_kmeans_opts *opts)
{
    KmeansLayout L;
    if (kmeans_layout(geom, prompt_len_host, n_centres_host, opts, &L, nullptr) != SANTAPP_OK) return 0;
    return L.total;
}

int santapp_kmeans_fit(const santapp_geom *geom, const int32_t *prompt_len_host, const int32_t *n_centres_host,
                       const void *k_prompt, const santapp_kmeans_opts *opts, float *centres, int32_t *steps_run,
                       void *workspace, size_t workspace_bytes, santapp_stream stream)
{
    KmeansLayout L;
    std::vector<int32_t> tabs;
    int rc = kmeans_layout(geom, prompt_len_host, n_centres_host, opts, &L, &tabs);
    if (rc != SANTAPP_OK) return rc;
    if (!k_prompt || !centres || !workspace) return SANTAPP_ERR_INVALID_ARG;
    if (misaligned(k_prompt, 16) || misaligned(centres, 4) || misaligned(steps_run, 4) || misaligned(workspace, 16))
        return SANTAPP_ERR_INVALID_ARG;
    if (workspace_bytes < L.total) return SANTAPP_ERR_WORKSPACE_TOO_SMALL;
    const int B = geom->n_seqs;
    std::vector<int64_t> offs(2 * ((size_t)B + 1));
    int64_t *row_off = offs.data(), *cen_off = row_off + B + 1;
    row_off[0] = cen_off[0] = 0;
    for (int b = 0; b < B; ++b) {
        row_off[b + 1] = row_off[b] + prompt_len_host[b];
        cen_off[b + 1] = cen_off[b] + n_centres_host[b];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    g_cuda_error[0] = 0;
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    cudaError_t err = cudaSuccess;
    {
        // the tables travel inside kernel arguments, a chunk of sequences per launch
        int32_t *t_dev = reinterpret_cast<int32_t *>(ws + L.tabs);
        for (int first = 0; first < B; first += kKmTableChunk) {
            KmTableChunk c;
            c.first = first;
            c.n = std::min(kKmTableChunk, B - first);
            for (int i = 0; i <= c.n; ++i) {
                c.row_off[i] = row_off[first + i];
                c.centre_off[i] = cen_off[first + i];
            }
            for (int i = 0; i < c.n; ++i) {
                c.n_init[i] = tabs[first + i];
                c.trials[i] = tabs[(size_t)B + first + i];
                c.t_max[i] = tabs[2 * (size_t)B + first + i];
            }
            err = launch_kmeans_tables(c, reinterpret_cast<int64_t *>(ws + L.row_off), reinterpret_cast<int64_t *>(ws + L.cen_off),
                                       t_dev, t_dev + B, t_dev + 2 * (size_t)B, s);
            if (err != cudaSuccess) return cuda_fail(err, "fit tables");
        }
    }

    KmeansParams p;
    p.n_seqs = B;
    p.n_kv = geom->n_kv_heads;
    p.elem = geom->elem_type;
    p.max_rows_per_seq = L.max_rows;
    p.batch = opts->batch_size;
    p.patience = opts->patience;
    p.no_host_poll = opts->no_host_poll != 0;
    p.ratio = opts->reassignment_ratio;
    p.seed_lo = (uint32_t)(opts->seed & 0xFFFFFFFFull);
    p.seed_hi = (uint32_t)(opts->seed >> 32);
    p.stream_base = opts->stream_base;
    p.k_max = L.k_max;
    p.n_init_max = L.n_init_max;
    p.trials_max = L.trials_max;
    p.t_max_max = L.t_max_max;
    p.rows_total = L.rows_total;
    p.centres_total = L.centres_total;
    p.seq_row_off = reinterpret_cast<const int64_t *>(ws + L.row_off);
    p.seq_centre_off = reinterpret_cast<const int64_t *>(ws + L.cen_off);
    const int32_t *t = reinterpret_cast<const int32_t *>(ws + L.tabs);
    p.seq_n_init = t;
    p.seq_trials = t + B;
    p.seq_t_max = t + 2 * B;
    p.k_prompt = static_cast<const uint16_t *>(k_prompt);
    p.centres_out = centres;
    p.steps_out = steps_run;
    p.perm = reinterpret_cast<int32_t *>(ws + L.perm);
    p.closest = reinterpret_cast<double *>(ws + L.closest);
    p.cand = reinterpret_cast<double *>(ws + L.cand);
    p.part = reinterpret_cast<double *>(ws + L.part);
    p.pick = reinterpret_cast<int32_t *>(ws + L.pick);
    p.centres64 = reinterpret_cast<double *>(ws + L.centres64);
    p.count = reinterpret_cast<double *>(ws + L.count);
    p.idx = reinterpret_cast<int32_t *>(ws + L.idx);
    p.label = reinterpret_cast<int32_t *>(ws + L.label);
    p.dist = reinterpret_cast<double *>(ws + L.dist);
    p.dist_part = reinterpret_cast<double *>(ws + L.dist_part);
    p.label_part = reinterpret_cast<int32_t *>(ws + L.label_part);
    p.assign_split = L.assign_split;
    p.sorted = reinterpret_cast<uint32_t *>(ws + L.sorted);
    p.state = reinterpret_cast<KmeansState *>(ws + L.state);
    p.active = reinterpret_cast<int *>(ws + L.active);
    err = launch_kmeans_fit(p, s);
    if (err != cudaSuccess) return cuda_fail(err, "kmeans_fit launch");
    return SANTAPP_OK;
}

}  // extern "C"

extern "C" {

int santapp_build_teams(const santapp_geom *geom, const int32_t *prompt_len_host, const void *k_prompt,
                        const void *v_prompt, santapp_teams *teams, void *workspace, size_t workspace_bytes,
                        santapp_stream stream)
{
    return build_records(geom, prompt_len_host, k_prompt, v_prompt, teams, workspace, workspace_bytes, stream, false);
}

int santapp_build_groups_mean(const santapp_geom *geom, const int32_t *prompt_len_host, const void *k_prompt,
                              const void *v_prompt, santapp_teams *teams, void *workspace, size_t workspace_bytes,
                              santapp_stream stream)
{
    if (geom && geom->reps_per_parent != 1) return SANTAPP_ERR_INVALID_ARG;    // one group per parent
    return build_records(geom, prompt_len_host, k_prompt, v_prompt, teams, workspace, workspace_bytes, stream, true);
}

size_t santapp_decode_workspace_bytes(const santapp_geom *geom, const santapp_teams *teams, int32_t n_sample)
{
    if (check_geom(geom) != SANTAPP_OK || !teams || n_sample < 1 || n_sample > 128) return 0;
    return decode_layout(geom, teams, n_sample, false, attend_grid_size()).total;
}

size_t santapp_dense_workspace_bytes(const santapp_geom *geom, const santapp_teams *teams)
{
    if (check_geom(geom) != SANTAPP_OK || !teams) return 0;
    return decode_layout(geom, teams, 1, true, attend_grid_size()).total;
}

int santapp_decode_attn(const santapp_geom *geom, const santapp_teams *teams, const void *q, const void *k_suffix,
                        const void *v_suffix, const int32_t *suffix_len_dev, int32_t suffix_cap, int32_t n_sample,
                        uint64_t seed, uint32_t step, const uint32_t *step_dev, uint32_t stream_base, float scale,
                        float *out,
                        const santapp_debug *dbg, void *workspace, size_t workspace_bytes, santapp_stream stream)
{
    g_launches = 0;
    int rc = check_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if ((rc = check_teams(geom, teams)) != SANTAPP_OK) return rc;
    if (!q || !out || !workspace) return SANTAPP_ERR_INVALID_ARG;
    if (misaligned(q, 16) || misaligned(out, 16) || misaligned(workspace, 16) || misaligned(k_suffix, 16)
        || misaligned(v_suffix, 16) || misaligned(suffix_len_dev, 4))
        return SANTAPP_ERR_INVALID_ARG;
    if (n_sample < 1 || suffix_cap < 0) return SANTAPP_ERR_INVALID_ARG;
    if (n_sample > 128) return SANTAPP_ERR_UNSUPPORTED;
    if (suffix_cap > 0 && suffix_len_dev && (!k_suffix || !v_suffix)) return SANTAPP_ERR_INVALID_ARG;
    if (!(scale >= 0.f) || isinf(scale)) return SANTAPP_ERR_INVALID_ARG;
    if ((int64_t)geom->n_seqs * geom->n_kv_heads * (int64_t)suffix_cap >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    const int grid = attend_grid_size();
    const DecodeLayout L = decode_layout(geom, teams, n_sample, false, grid);
    if (L.seg_cap > attend_max_segments() || L.n_pairs > attend_max_pairs()) return SANTAPP_ERR_UNSUPPORTED;
    if (workspace_bytes < L.total) return SANTAPP_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    g_cuda_error[0] = 0;
    char *ws = static_cast<char *>(workspace);
    const double sc = scale == 0.f ? 1.0 / sqrt((double)geom->head_dim) : (double)scale;

    PlanView plan;
    fill_plan(L, ws, plan);

    ScoreParams rp;
    rp.bv = make_view(geom, teams);
    rp.rep_keys = static_cast<const uint16_t *>(teams->rep_keys);
    rp.team_row_start = teams->team_row_start;
    rp.q = static_cast<const uint16_t *>(q);
    rp.y32 = reinterpret_cast<float *>(ws + L.y32);
    rp.y_stride = L.y_stride;
    rp.tile_stride = L.tile_stride;
    rp.n_sample = n_sample;
    rp.seed_lo = (uint32_t)(seed & 0xFFFFFFFFull);
    rp.seed_hi = (uint32_t)(seed >> 32);
    rp.step = step;
    rp.step_dev = step_dev;
    rp.stream_base = stream_base;
    rp.scale = sc;
    rp.n_pairs = L.n_pairs;
    rp.status = dbg ? dbg->status : nullptr;
    rp.trace = dbg ? reinterpret_cast<unsigned long long *>(dbg->trace) : nullptr;
    rp.tune_flags = 0;
#ifdef SANTAPP_TUNE
    if (const char *e = getenv("SANTAPP_SCORE_FLAGS")) rp.tune_flags = atoi(e);
#endif
    cudaError_t err = cudaSuccess;
    if (rp.status && g_stage_mask == SANTAPP_STAGE_ALL) {
        // diagnostics only: a node of its own, so that no kernel both clears and raises the flags
        err = cudaMemsetAsync(rp.status, 0, sizeof(int32_t), s);
        if (err != cudaSuccess) return cuda_fail(err, "status memset");
    }
    if (g_stage_mask & SANTAPP_STAGE_ROUTE) {
        err = launch_score32(rp, teams->max_teams_per_seq, s);
        if (err != cudaSuccess) return cuda_fail(err, "score launch");
        ++g_launches;
    }

    PlanParams pp;
    pp.in.bv = rp.bv;
    pp.in.y32 = rp.y32;
    pp.in.y_stride = L.y_stride;
    pp.in.rep_keys = rp.rep_keys;
    pp.in.team_row_start = teams->team_row_start;
    pp.in.rep_abs_max = teams->rep_abs_max;
    pp.in.q = rp.q;
    pp.in.n_sample = n_sample;
    pp.in.seed_lo = rp.seed_lo;
    pp.in.seed_hi = rp.seed_hi;
    pp.in.step = step;
    pp.in.step_dev = step_dev;
    pp.in.stream_base = stream_base;
    pp.in.scale = sc;
    pp.in.suffix_len = suffix_len_dev;
    pp.in.suffix_cap = suffix_cap;
    pp.in.sel_team = reinterpret_cast<int32_t *>(ws + L.sel_team);
    pp.in.sel_logc = reinterpret_cast<float *>(ws + L.sel_logc);
    pp.in.sel_rows = reinterpret_cast<int2 *>(ws + L.sel_rows);
    pp.in.status = dbg ? dbg->status : nullptr;
    pp.in.dbg_sel_idx = dbg ? dbg->sel_idx : nullptr;
    pp.in.dbg_sel_logc = dbg ? dbg->sel_logc : nullptr;
    pp.in.dbg_tau = dbg ? dbg->tau : nullptr;
    pp.in.dbg_union_rows = dbg ? dbg->union_rows : nullptr;
    pp.in.trace = rp.trace;
    pp.plan = plan;
    pp.n_pairs = L.n_pairs;
    if (g_stage_mask & SANTAPP_STAGE_SELECT) {
        err = launch_headplan(pp.in, s);
        if (err != cudaSuccess) return cuda_fail(err, "headplan launch");
        ++g_launches;
    }
    // few pairs: the plan is built inside the attention kernel (fixed CTAs per pair)
    if (!L.static_split && (g_stage_mask & SANTAPP_STAGE_SELECT)) {
        err = launch_plan(pp, teams->max_teams_per_seq, s);
        if (err != cudaSuccess) return cuda_fail(err, "plan launch");
        ++g_launches;
        if (L.n_pairs > attend_pairs_staged()) {                // else the attention kernel sums the pairs' rows itself
            err = launch_pair_prefix(pp, s);
            if (err != cudaSuccess) return cuda_fail(err, "pair prefix launch");
            ++g_launches;
        }
    }

    AttendParams ap;
    ap.bv = rp.bv;
    ap.k_packed = static_cast<const uint16_t *>(teams->k_packed);
    ap.v_packed = static_cast<const uint16_t *>(teams->v_packed);
    ap.k_suffix = static_cast<const uint16_t *>(k_suffix);
    ap.v_suffix = static_cast<const uint16_t *>(v_suffix);
    ap.q = rp.q;
    ap.qk_scale_log2 = (float)(sc * 1.4426950408889634);
    ap.plan = plan;
    ap.in = pp.in;
    ap.n_pairs = L.n_pairs;
    ap.partials = reinterpret_cast<float *>(ws + L.partials);
    ap.out = out;
    ap.status = rp.status;
    ap.min_rows_per_cta = 64;
    ap.span_penalty_rows = 640;                                 // measured: a second span costs about 8 us of one SM's bandwidth
#ifdef SANTAPP_TUNE
    if (const char *e = getenv("SANTAPP_SPAN_PENALTY")) ap.span_penalty_rows = atoi(e);
#endif
    ap.ctas_per_pair = L.ctas_per_pair;
    ap.max_words = (teams->max_teams_per_seq + 31) / 32;
    if (g_stage_mask & SANTAPP_STAGE_ATTEND) {
        const int launch_grid = L.static_split ? L.n_pairs * L.ctas_per_pair : grid;
        err = launch_attend(ap, false, L.static_split, launch_grid, s);
        if (err != cudaSuccess) return cuda_fail(err, "attend launch");
        ++g_launches;
    }
    if (g_stage_mask & SANTAPP_STAGE_MERGE) {
        const int launch_grid = L.static_split ? L.n_pairs * L.ctas_per_pair : grid;
        err = launch_merge(ap, L.static_split, launch_grid, s);
        if (err != cudaSuccess) return cuda_fail(err, "merge launch");
        ++g_launches;
    }
    return SANTAPP_OK;
}

int santapp_dense_decode_attn(const santapp_geom *geom, const santapp_teams *teams, const void *q,
                              const void *k_suffix, const void *v_suffix, const int32_t *suffix_len_dev,
                              int32_t suffix_cap, float scale, float *out, void *workspace, size_t workspace_bytes,
                              santapp_stream stream)
{
    g_launches = 0;
    int rc = check_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if ((rc = check_teams(geom, teams)) != SANTAPP_OK) return rc;
    if (!q || !out || !workspace) return SANTAPP_ERR_INVALID_ARG;
    if (misaligned(q, 16) || misaligned(out, 16) || misaligned(workspace, 16) || misaligned(k_suffix, 16)
        || misaligned(v_suffix, 16) || misaligned(suffix_len_dev, 4))
        return SANTAPP_ERR_INVALID_ARG;
    if (suffix_cap < 0) return SANTAPP_ERR_INVALID_ARG;
    if (suffix_cap > 0 && suffix_len_dev && (!k_suffix || !v_suffix)) return SANTAPP_ERR_INVALID_ARG;
    if (!(scale >= 0.f) || isinf(scale)) return SANTAPP_ERR_INVALID_ARG;
    if ((int64_t)geom->n_seqs * geom->n_kv_heads * (int64_t)suffix_cap >= (int64_t)1 << 31) return SANTAPP_ERR_UNSUPPORTED;
    const int grid = attend_grid_size();
    const DecodeLayout L = decode_layout(geom, teams, 1, true, grid);
    if (L.n_pairs > attend_max_pairs()) return SANTAPP_ERR_UNSUPPORTED;
    if (workspace_bytes < L.total) return SANTAPP_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    g_cuda_error[0] = 0;
    char *ws = static_cast<char *>(workspace);
    const double sc = scale == 0.f ? 1.0 / sqrt((double)geom->head_dim) : (double)scale;

    PlanView plan;
    fill_plan(L, ws, plan);

    PlanParams pp;
    memset(&pp, 0, sizeof(pp));
    pp.in.bv = make_view(geom, teams);
    pp.in.suffix_len = suffix_len_dev;
    pp.in.suffix_cap = suffix_cap;
    pp.plan = plan;
    pp.n_pairs = L.n_pairs;
    cudaError_t err;
    if (!L.static_split) {                                      // else the plan is trivial and built inside the kernel
        err = launch_dense_plan(pp, s);
        if (err != cudaSuccess) return cuda_fail(err, "dense_plan launch");
        ++g_launches;
        if (L.n_pairs > attend_pairs_staged()) {
            err = launch_pair_prefix(pp, s);
            if (err != cudaSuccess) return cuda_fail(err, "pair prefix launch");
            ++g_launches;
        }
    }

    AttendParams ap;
    ap.bv = pp.in.bv;
    ap.k_packed = static_cast<const uint16_t *>(teams->k_packed);
    ap.v_packed = static_cast<const uint16_t *>(teams->v_packed);
    ap.k_suffix = static_cast<const uint16_t *>(k_suffix);
    ap.v_suffix = static_cast<const uint16_t *>(v_suffix);
    ap.q = static_cast<const uint16_t *>(q);
    ap.qk_scale_log2 = (float)(sc * 1.4426950408889634);
    ap.plan = plan;
    ap.in = pp.in;
    ap.n_pairs = L.n_pairs;
    ap.partials = reinterpret_cast<float *>(ws + L.partials);
    ap.out = out;
    ap.status = nullptr;
    ap.min_rows_per_cta = 64;
    ap.span_penalty_rows = 1040;                                // measured on the dense path: about 13 us
#ifdef SANTAPP_TUNE
    if (const char *e = getenv("SANTAPP_SPAN_PENALTY_DENSE")) ap.span_penalty_rows = atoi(e);
#endif
    ap.ctas_per_pair = L.ctas_per_pair;
    const int launch_grid = L.static_split ? L.n_pairs * L.ctas_per_pair : grid;
    err = launch_attend(ap, true, L.static_split, launch_grid, s);
    if (err != cudaSuccess) return cuda_fail(err, "attend launch");
    ++g_launches;
    err = launch_merge(ap, L.static_split, launch_grid, s);
    if (err != cudaSuccess) return cuda_fail(err, "merge launch");
    ++g_launches;
    return SANTAPP_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Dense decode attention without a caller-provided workspace.
// ---------------------------------------------------------------------------------------------
namespace {

// Scratch for santapp_dense_decode_attn_noalloc. In host code this name is only a handle for
// the runtime's symbol lookup, never a device address; the address comes from
// cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[SANTAPP_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_scratch_addr[kMaxDevices];      // per device ordinal; null until looked up

}  // namespace

extern "C" int santapp_dense_decode_attn_noalloc(const santapp_geom *geom, const santapp_teams *teams,
                                                 const void *q, const void *k_suffix, const void *v_suffix,
                                                 const int32_t *suffix_len_dev, int32_t suffix_cap, float scale,
                                                 float *out, santapp_stream stream)
{
    int rc = check_geom(geom);
    if (rc != SANTAPP_OK) return rc;
    if ((rc = check_teams(geom, teams)) != SANTAPP_OK) return rc;
    const size_t need = santapp_dense_workspace_bytes(geom, teams);
    if (need > (size_t)SANTAPP_STATIC_SCRATCH_BYTES) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "built-in scratch holds %u bytes, this problem needs %zu",
                 (unsigned)SANTAPP_STATIC_SCRATCH_BYTES, need);
        return SANTAPP_ERR_STATIC_SCRATCH;
    }
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return cuda_fail(err, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return SANTAPP_ERR_UNSUPPORTED;
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (g_static_scratch_addr[dev] == nullptr) {
            // once per device, with that device current
            void *addr = nullptr;
            err = cudaGetSymbolAddress(&addr, g_static_scratch);
            if (err != cudaSuccess) return cuda_fail(err, "cudaGetSymbolAddress(static scratch)");
            g_static_scratch_addr[dev] = addr;
        }
        scratch = g_static_scratch_addr[dev];
    }
    return santapp_dense_decode_attn(geom, teams, q, k_suffix, v_suffix, suffix_len_dev, suffix_cap, scale, out,
                                     scratch, (size_t)SANTAPP_STATIC_SCRATCH_BYTES, stream);
}
