/*
 * SANTA++ decode attention — plain fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT CODE. This file is the slow, obviously
 * correct restatement of what the paper's method computes. Only the test
 * suite, the smoke check and the benchmark's cpu-baseline / reference arm may
 * call it. It shares no code, tables or helpers with the CUDA path.
 *
 * Every function follows one passage of the paper, in the paper's order and
 * notation, with no blocking, fusion or reordering:
 *   orc_dense_head            full-cache attention, Eq. (method-attention)
 *   orc_contiguous_parents    Algorithm 4 (contiguous parent partition)
 *   orc_build_teams           Algorithm 2 (actual-key teams from parents)
 *   orc_decode_head_given_gumbel / orc_decode_head
 *                             Algorithm 1 (SANTA++ attention, one query head),
 *                             routing weight Eq. (method-routing), inclusion
 *                             correction Eq. (method-inclusion), estimator
 *                             Eq. (method-estimate)
 *   orc_philox4x32_10, orc_uniform_open, orc_gumbel, orc_team_word
 *                             the reproducible Gumbel(0,1) stream (the paper
 *                             only asks for independent Gumbel draws; the
 *                             generator and its keying are this build's
 *                             reading and are documented with the function)
 *   orc_logical_access_*      logical KV-access counter, Eq. (qwen-logical-access)
 *   orc_team_budget           selected-team count, Eq. (method-budget)
 *   orc_mla_logical_access_pct   shared-row counter of a shared-latent cache, Eq. (mla-logical-access)
 *   orc_routing_kl            routing-agreement diagnostic, Eq. (diagnostic-kl)
 *   orc_group_mean_keys       centroid-guided baseline of the routing diagnostic: one group per
 *                             parent, routed by the arithmetic mean of its keys
 *   orc_group_mean_keys_parents   the same baseline on an arbitrary partition (k-means groups)
 *   orc_minibatch_kmeans      the fit of Algorithm 3 (minibatch k-means, greedy k-means++ start) in the
 *                             reading spelled out above the function
 *   orc_kmeans_parent_count, orc_nearest_centre_parents
 *                             Algorithm 3 without the fit: the number of centres, and the
 *                             nearest-centre partition with empty parents omitted
 *
 * Parity pins (tests marked "not gpu"): Philox words against an independent
 * library generator; Gumbel law by Kolmogorov-Smirnov and moments; first-draw
 * law and the every-key-its-own-team limit against softmax; K >= M against a
 * library softmax; inclusion probabilities against exact enumeration of the
 * successive-sampling law and against 1e5-draw frequencies; unbiasedness of
 * the two unnormalised sums by quadrature and Monte Carlo; Algorithm 2 on
 * hand-worked parents and duplicate keys; the accounting helpers against the
 * figures the paper prints; the routing KL against its closed forms (zero for
 * singleton teams, log N - H(p) for one team holding every key) and against a
 * numpy re-evaluation of the defining sum; the nearest-centre partition against a library
 * vector quantiser, hand-worked ties and empty centres, and brute force over all labellings; the
 * fit by recovery of separated blobs, the k = N and k = 1 special cases (the latter against the
 * mean of the recomputed draws), its step limits, the reassignment of a starved centre, and its
 * inertia against a library's minibatch and full-batch k-means.
 * Parity unpinned: nothing in this file. (Accuracy of the sampled output
 * against dense attention on real model data is outside what can be pinned
 * here; only the estimator identities are.)
 *
 * Build: gcc -O2 -ffp-contract=off -fPIC -shared [-fopenmp] (see build_oracle.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* Random stream                                                             */
/* ------------------------------------------------------------------------- */

/* Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw 2011): a 128-bit
 * counter and a 64-bit key give four 32-bit words. Each round multiplies two
 * counter words by fixed odd constants, swaps high/low halves into the other
 * lanes and xors in the key; the key is advanced by Weyl constants between
 * rounds. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t prod0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t prod1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
        uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 32-bit word that belongs to team g (0-based, local to its sequence and
 * KV head) for query head `head` at decode step `step` on stream `stream`:
 * key = (low, high) halves of the seed; counter = (g / 4, step, head, stream);
 * word g mod 4 of the block. Heads that share a KV head differ in the counter,
 * so their draws are independent, as the GQA rule of the Method section
 * requires. */
uint32_t orc_team_word(uint64_t seed, uint32_t step, uint32_t head, uint32_t stream, uint32_t g)
{
    uint32_t ctr[4] = { g >> 2, step, head, stream };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return out[g & 3u];
}

/* Uniform on the open interval: the centre of the x-th of 2^32 equal cells. */
double orc_uniform_open(uint32_t x)
{
    return ((double)x + 0.5) * (1.0 / 4294967296.0);
}

/* Standard Gumbel by inversion of the CDF exp(-exp(-x)) quoted in the
 * "Conditional inclusion correction" paragraph: G = -log(-log u). */
double orc_gumbel(uint32_t x)
{
    return -log(-log(orc_uniform_open(x)));
}

void orc_gumbel_many(uint64_t seed, uint32_t step, uint32_t head, uint32_t stream,
                     int32_t M, double *gumbel /* [M] */)
{
    for (int32_t g = 0; g < M; ++g)
        gumbel[g] = orc_gumbel(orc_team_word(seed, step, head, stream, (uint32_t)g));
}

/* ------------------------------------------------------------------------- */
/* Full-cache attention, Eq. (method-attention)                              */
/* ------------------------------------------------------------------------- */

static double dot(const double *a, const double *b, int d)
{
    double s = 0.0;
    for (int j = 0; j < d; ++j) s += a[j] * b[j];
    return s;
}

/* s_i = q.k_i * scale, Z = sum e^{s_i}, U = sum e^{s_i} v_i, o = U / Z over
 * the n rows of (k, v). Evaluated with the usual max shift, which cancels in
 * the ratio. */
void orc_dense_head(int d, const double *q, int64_t n, const double *k, const double *v,
                    double scale, double *o /* [d] */)
{
    double smax = -INFINITY;
    for (int64_t i = 0; i < n; ++i) {
        double s = dot(q, k + i * d, d) * scale;
        if (s > smax) smax = s;
    }
    double Z = 0.0;
    for (int j = 0; j < d; ++j) o[j] = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double s = dot(q, k + i * d, d) * scale;
        double a = exp(s - smax);
        Z += a;
        for (int j = 0; j < d; ++j) o[j] += a * v[i * d + j];
    }
    for (int j = 0; j < d; ++j) o[j] /= Z;
}

/* Dense attention over prompt rows followed by suffix rows (two buffers). */
void orc_dense_head_two(int d, const double *q,
                        int64_t n, const double *k, const double *v,
                        int64_t t, const double *ks, const double *vs,
                        double scale, double *o /* [d] */)
{
    double smax = -INFINITY;
    for (int64_t i = 0; i < n; ++i) { double s = dot(q, k + i * d, d) * scale; if (s > smax) smax = s; }
    for (int64_t i = 0; i < t; ++i) { double s = dot(q, ks + i * d, d) * scale; if (s > smax) smax = s; }
    double Z = 0.0;
    for (int j = 0; j < d; ++j) o[j] = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double a = exp(dot(q, k + i * d, d) * scale - smax);
        Z += a;
        for (int j = 0; j < d; ++j) o[j] += a * v[i * d + j];
    }
    for (int64_t i = 0; i < t; ++i) {
        double a = exp(dot(q, ks + i * d, d) * scale - smax);
        Z += a;
        for (int j = 0; j < d; ++j) o[j] += a * vs[i * d + j];
    }
    for (int j = 0; j < d; ++j) o[j] /= Z;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 4: contiguous parent partition                                  */
/* ------------------------------------------------------------------------- */

/* Parents are consecutive spans of P tokens; the last may be short. Writes
 * parent_start[0..n_parents] (0-based, half-open) and returns n_parents =
 * ceil(N / P). */
int32_t orc_contiguous_parents(int32_t N, int32_t P, int32_t *parent_start)
{
    int32_t n_parents = (N + P - 1) / P;
    for (int32_t u = 0; u < n_parents; ++u) parent_start[u] = u * P;
    parent_start[n_parents] = N;
    return n_parents;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 2: actual-key teams from a parent partition                     */
/* ------------------------------------------------------------------------- */

static double sqdist(const double *a, const double *b, int d)
{
    double s = 0.0;
    for (int j = 0; j < d; ++j) { double e = a[j] - b[j]; s += e * e; }
    return s;
}

/* keys: [N][d] prefill keys in token order. Parents are given as index lists:
 * parent u holds tokens parent_member[parent_start[u] .. parent_start[u+1]),
 * listed in increasing token index. R = maximum representatives per parent.
 * Outputs (teams in emission order: parent by parent, representative-selection
 * order inside a parent):
 *   team_start[M+1], team_member[N]  members of team g in increasing token index
 *   rep_row[M]                       token index of the representative of team g
 * Returns M. Ties: representative choices go to the smallest token index,
 * assignments to the earliest-selected representative ("Shared team
 * construction" paragraph). */
int32_t orc_build_teams(int32_t N, int d, const double *keys,
                        int32_t n_parents, const int32_t *parent_start, const int32_t *parent_member,
                        int32_t R,
                        int32_t *team_start, int32_t *team_member, int32_t *rep_row)
{
    (void)N;
    double *mu = (double *)malloc(sizeof(double) * (size_t)d);
    int32_t M = 0, rows_out = 0;
    team_start[0] = 0;
    for (int32_t p = 0; p < n_parents; ++p) {
        const int32_t *C = parent_member + parent_start[p];
        int32_t nC = parent_start[p + 1] - parent_start[p];
        int32_t r = R < nC ? R : nC;
        /* parent mean */
        for (int j = 0; j < d; ++j) mu[j] = 0.0;
        for (int32_t a = 0; a < nC; ++a)
            for (int j = 0; j < d; ++j) mu[j] += keys[(int64_t)C[a] * d + j];
        for (int j = 0; j < d; ++j) mu[j] /= (double)nC;
        /* first representative: the actual key nearest the mean */
        int32_t *L = (int32_t *)malloc(sizeof(int32_t) * (size_t)r);      /* positions in C */
        char *is_rep = (char *)calloc((size_t)nC, 1);
        double best = INFINITY; int32_t arg = 0;
        for (int32_t a = 0; a < nC; ++a) {
            double dist = sqdist(keys + (int64_t)C[a] * d, mu, d);
            if (dist < best) { best = dist; arg = a; }
        }
        L[0] = arg; is_rep[arg] = 1;
        /* farthest-first: maximise the distance to the nearest chosen representative */
        for (int32_t u = 1; u < r; ++u) {
            double far = -INFINITY; int32_t farg = -1;
            for (int32_t a = 0; a < nC; ++a) {
                if (is_rep[a]) continue;
                double nearest = INFINITY;
                for (int32_t w = 0; w < u; ++w) {
                    double dist = sqdist(keys + (int64_t)C[a] * d, keys + (int64_t)C[L[w]] * d, d);
                    if (dist < nearest) nearest = dist;
                }
                if (nearest > far) { far = nearest; farg = a; }
            }
            L[u] = farg; is_rep[farg] = 1;
        }
        /* nearest-representative assignment, then representative self-ownership */
        int32_t *b = (int32_t *)malloc(sizeof(int32_t) * (size_t)nC);
        for (int32_t a = 0; a < nC; ++a) {
            double nearest = INFINITY; int32_t owner = -1;
            for (int32_t u = 0; u < r; ++u) {
                double dist = sqdist(keys + (int64_t)C[a] * d, keys + (int64_t)C[L[u]] * d, d);
                if (dist < nearest) { nearest = dist; owner = u; }
            }
            b[a] = owner;
        }
        for (int32_t u = 0; u < r; ++u) b[L[u]] = u;
        /* emit the r teams of this parent */
        for (int32_t u = 0; u < r; ++u) {
            for (int32_t a = 0; a < nC; ++a)
                if (b[a] == u) team_member[rows_out++] = C[a];
            rep_row[M] = C[L[u]];
            ++M;
            team_start[M] = rows_out;
        }
        free(b); free(is_rep); free(L);
    }
    free(mu);
    return M;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1: SANTA++ attention for one query head                         */
/* ------------------------------------------------------------------------- */

typedef struct { double y; int32_t g; } orc_scored;

/* Descending perturbed score; equal scores (a continuum-probability-zero event
 * the paper does not order) go to the smaller team id. */
static int cmp_scored(const void *pa, const void *pb)
{
    const orc_scored *a = (const orc_scored *)pa, *b = (const orc_scored *)pb;
    if (a->y > b->y) return -1;
    if (a->y < b->y) return 1;
    return (a->g > b->g) - (a->g < b->g);
}

/*
 * Inputs
 *   q[d]; prompt rows k_cache/v_cache [N][d] in token order; team records as
 *   CSR (team_start[M+1], team_member[*] token indices) plus the frozen
 *   representative keys rep_key[M][d]; exact suffix ks/vs [t][d]; requested
 *   team count K >= 1; the M Gumbel draws (unused when K >= M); scale = 1/sqrt(d).
 * Outputs
 *   o[d]          estimated attention output U^ / Z^
 *   sel[Ke]       selected teams in descending perturbed score (Ke = min(K, M);
 *                 0..M-1 in order when K >= M)
 *   logc[Ke]      log of the conditional inclusion correction c_g (0 when K >= M)
 *   tau_out       the (K+1)-st largest perturbed score (NaN when K >= M)
 *   margin_out    Y_(K) - Y_(K+1), how far the draw is from a different set
 *   phi_out[M], y_out[M]   routing logits and perturbed scores (nullable)
 *   U_out[d], Z_out        the two unnormalised sums multiplied by e^{-shift}
 *                          (nullable); shift = *shift_io if use_shift != 0,
 *                          else the maximum corrected logit, written back
 * Returns Ke.
 */
int32_t orc_decode_head_given_gumbel(
    int d, const double *q,
    int64_t N, const double *k_cache, const double *v_cache,
    int32_t M, const int32_t *team_start, const int32_t *team_member, const double *rep_key,
    int64_t t, const double *ks, const double *vs,
    int32_t K, const double *gumbel, double scale,
    double *o, int32_t *sel, double *logc, double *tau_out, double *margin_out,
    double *phi_out, double *y_out, double *U_out, double *Z_out,
    int use_shift, double *shift_io)
{
    (void)N;
    int32_t Ke = K < M ? K : M;                         /* K <- min(K, M) */
    double tau = NAN, margin = INFINITY;
    double *c = (double *)malloc(sizeof(double) * (size_t)(Ke > 0 ? Ke : 1));
    if (Ke == M) {
        /* select every team with correction one; no draw is consumed */
        for (int32_t g = 0; g < M; ++g) { sel[g] = g; c[g] = 1.0; }
        if (phi_out || y_out)
            for (int32_t g = 0; g < M; ++g) {
                double n_g = (double)(team_start[g + 1] - team_start[g]);
                double phi = log(n_g) + dot(q, rep_key + (int64_t)g * d, d) * scale;
                if (phi_out) phi_out[g] = phi;
                if (y_out) y_out[g] = NAN;
            }
    } else {
        orc_scored *Y = (orc_scored *)malloc(sizeof(orc_scored) * (size_t)M);
        double *phi = (double *)malloc(sizeof(double) * (size_t)M);
        for (int32_t g = 0; g < M; ++g) {
            double n_g = (double)(team_start[g + 1] - team_start[g]);
            phi[g] = log(n_g) + dot(q, rep_key + (int64_t)g * d, d) * scale;   /* routing logit */
            Y[g].y = phi[g] + gumbel[g];                                       /* perturbed score */
            Y[g].g = g;
            if (phi_out) phi_out[g] = phi[g];
            if (y_out) y_out[g] = Y[g].y;
        }
        qsort(Y, (size_t)M, sizeof(orc_scored), cmp_scored);
        for (int32_t a = 0; a < Ke; ++a) sel[a] = Y[a].g;      /* the K largest */
        tau = Y[Ke].y;                                         /* the (K+1)-st largest */
        margin = Y[Ke - 1].y - Y[Ke].y;
        for (int32_t a = 0; a < Ke; ++a)
            c[a] = -expm1(-exp(phi[sel[a]] - tau));            /* 1 - exp[-exp(phi - tau)] */
        free(phi); free(Y);
    }
    for (int32_t a = 0; a < Ke; ++a) logc[a] = log(c[a]);

    /* exact logits of every member of every selected team and of the suffix;
     * one common shift so that the exponentials stay in range */
    double shift;
    if (use_shift) {
        shift = *shift_io;
    } else {
        shift = -INFINITY;
        for (int64_t i = 0; i < t; ++i) {
            double s = dot(q, ks + i * d, d) * scale;
            if (s > shift) shift = s;
        }
        for (int32_t a = 0; a < Ke; ++a) {
            int32_t g = sel[a];
            for (int32_t m = team_start[g]; m < team_start[g + 1]; ++m) {
                double s = dot(q, k_cache + (int64_t)team_member[m] * d, d) * scale - logc[a];
                if (s > shift) shift = s;
            }
        }
        if (shift_io) *shift_io = shift;
    }
    double Zhat = 0.0;
    double *Uhat = (double *)malloc(sizeof(double) * (size_t)d);
    for (int j = 0; j < d; ++j) Uhat[j] = 0.0;
    /* suffix rows: weight one */
    for (int64_t i = 0; i < t; ++i) {
        double a_i = exp(dot(q, ks + i * d, d) * scale - shift);
        Zhat += a_i;
        for (int j = 0; j < d; ++j) Uhat[j] += a_i * vs[i * d + j];
    }
    /* selected teams: team sums first, then divided by c_g */
    double *Ug = (double *)malloc(sizeof(double) * (size_t)d);
    for (int32_t a = 0; a < Ke; ++a) {
        int32_t g = sel[a];
        double Zg = 0.0;
        for (int j = 0; j < d; ++j) Ug[j] = 0.0;
        for (int32_t m = team_start[g]; m < team_start[g + 1]; ++m) {
            int64_t i = team_member[m];
            double a_i = exp(dot(q, k_cache + i * d, d) * scale - shift);
            Zg += a_i;
            for (int j = 0; j < d; ++j) Ug[j] += a_i * v_cache[i * d + j];
        }
        Zhat += Zg / c[a];
        for (int j = 0; j < d; ++j) Uhat[j] += Ug[j] / c[a];
    }
    for (int j = 0; j < d; ++j) o[j] = Uhat[j] / Zhat;
    if (U_out) for (int j = 0; j < d; ++j) U_out[j] = Uhat[j];
    if (Z_out) *Z_out = Zhat;
    if (tau_out) *tau_out = tau;
    if (margin_out) *margin_out = margin;
    free(Ug); free(Uhat); free(c);
    return Ke;
}

/* Algorithm 1 with the Gumbel draws taken from the Philox stream keyed by
 * (seed; step, head, stream). */
int32_t orc_decode_head(
    int d, const double *q,
    int64_t N, const double *k_cache, const double *v_cache,
    int32_t M, const int32_t *team_start, const int32_t *team_member, const double *rep_key,
    int64_t t, const double *ks, const double *vs,
    int32_t K, uint64_t seed, uint32_t step, uint32_t head, uint32_t stream, double scale,
    double *o, int32_t *sel, double *logc, double *tau_out, double *margin_out)
{
    double *gumbel = (double *)malloc(sizeof(double) * (size_t)(M > 0 ? M : 1));
    if (K < M) orc_gumbel_many(seed, step, head, stream, M, gumbel);
    int32_t Ke = orc_decode_head_given_gumbel(d, q, N, k_cache, v_cache, M, team_start, team_member,
                                              rep_key, t, ks, vs, K, gumbel, scale, o, sel, logc,
                                              tau_out, margin_out, NULL, NULL, NULL, NULL, 0, NULL);
    free(gumbel);
    return Ke;
}

/*
 * One decode step of one sequence under GQA: query head h uses KV head h / G
 * (G = n_q_heads / n_kv_heads), shares that head's team records with its
 * siblings, and samples on its own Philox counter. Buffers are per KV head,
 * concatenated: k_cache/v_cache [n_kv][N][d], team_start [n_kv][M_max+1] with
 * M[j] teams used, team_member [n_kv][N], rep_key [n_kv][M_max][d], suffix
 * [n_kv][t][d]. Outputs per query head: o [n_q][d], sel/logc [n_q][K],
 * tau/margin [n_q]. Heads are independent; OpenMP, when compiled in, runs
 * them on separate threads without changing any result.
 */
void orc_decode_step(
    int d, int32_t n_q, int32_t n_kv, const double *q /* [n_q][d] */,
    int64_t N, const double *k_cache, const double *v_cache,
    int32_t M_max, const int32_t *M, const int32_t *team_start, const int32_t *team_member,
    const double *rep_key,
    int64_t t, const double *ks, const double *vs,
    int32_t K, uint64_t seed, uint32_t step, uint32_t stream, double scale,
    double *o, int32_t *sel, double *logc, double *tau, double *margin, int32_t n_threads)
{
    int32_t G = n_q / n_kv;
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads > 0 ? n_threads : 1)
#endif
    for (int32_t h = 0; h < n_q; ++h) {
        int32_t j = h / G;
        orc_decode_head(d, q + (int64_t)h * d,
                        N, k_cache + (int64_t)j * N * d, v_cache + (int64_t)j * N * d,
                        M[j], team_start + (int64_t)j * (M_max + 1), team_member + (int64_t)j * N,
                        rep_key + (int64_t)j * M_max * d,
                        t, ks + (int64_t)j * t * d, vs + (int64_t)j * t * d,
                        K, seed, step, (uint32_t)h, stream, scale,
                        o + (int64_t)h * d, sel + (int64_t)h * K, logc + (int64_t)h * K,
                        tau + h, margin + h);
    }
}

/* Dense attention for every query head of one sequence (same buffer layout). */
void orc_dense_step(
    int d, int32_t n_q, int32_t n_kv, const double *q,
    int64_t N, const double *k_cache, const double *v_cache,
    int64_t t, const double *ks, const double *vs, double scale, double *o, int32_t n_threads)
{
    int32_t G = n_q / n_kv;
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads > 0 ? n_threads : 1)
#endif
    for (int32_t h = 0; h < n_q; ++h) {
        int32_t j = h / G;
        orc_dense_head_two(d, q + (int64_t)h * d,
                           N, k_cache + (int64_t)j * N * d, v_cache + (int64_t)j * N * d,
                           t, ks + (int64_t)j * t * d, vs + (int64_t)j * t * d, scale,
                           o + (int64_t)h * d);
    }
}

int32_t orc_has_openmp(void)
{
#ifdef _OPENMP
    return 1;
#else
    return 0;
#endif
}

/* ------------------------------------------------------------------------- */
/* Accounting                                                                */
/* ------------------------------------------------------------------------- */

/* Eq. (method-budget): K = min{M, S / (P / R)}; R must divide P and P/R must
 * divide S. Returns -1 when the divisibility rules fail. */
int32_t orc_team_budget(int32_t M, int32_t S, int32_t P, int32_t R)
{
    if (P <= 0 || R <= 0 || S <= 0) return -1;
    if (P % R != 0) return -1;
    int32_t per = P / R;
    if (S % per != 0) return -1;
    int32_t K = S / per;
    return K < M ? K : M;
}

/* Eq. (qwen-logical-access): for calls c with m_c representatives scanned,
 * u_c distinct selected prompt rows (union over the heads of a KV head), e_c
 * suffix rows and cache length N_c, KV% = 100 * sum[m + 2(u + e)] / sum[2 N].
 * Arrays have n_calls entries. */
double orc_logical_access_pct(int64_t n_calls, const int64_t *m, const int64_t *u,
                              const int64_t *e, const int64_t *Ncache)
{
    double num = 0.0, den = 0.0;
    for (int64_t c = 0; c < n_calls; ++c) {
        num += (double)m[c] + 2.0 * ((double)u[c] + (double)e[c]);
        den += 2.0 * (double)Ncache[c];
    }
    return 100.0 * num / den;
}

/* Number of distinct prompt rows read for one KV head: the union, over the
 * n_heads query heads that share it, of the members of their selected teams. */
int64_t orc_union_rows(int32_t M, const int32_t *team_start, int32_t n_heads, int32_t Ke,
                       const int32_t *sel /* [n_heads][Ke] */)
{
    char *hit = (char *)calloc((size_t)(M > 0 ? M : 1), 1);
    for (int32_t h = 0; h < n_heads; ++h)
        for (int32_t a = 0; a < Ke; ++a) hit[sel[(int64_t)h * Ke + a]] = 1;
    int64_t rows = 0;
    for (int32_t g = 0; g < M; ++g)
        if (hit[g]) rows += team_start[g + 1] - team_start[g];
    free(hit);
    return rows;
}

/* Bytes of keys and values a dense decode step streams for one layer:
 * n_kv heads x N rows x d elements x (K and V) x bytes per element. */
double orc_dense_kv_bytes(int64_t N, int32_t n_kv, int32_t d, int32_t bytes_per_el)
{
    return 2.0 * (double)n_kv * (double)N * (double)d * (double)bytes_per_el;
}

/* Eq. (diagnostic-kl): agreement of the routing proposal with dense attention over
 * the N prompt tokens, for one query head; no sampling is involved.
 *   p_i  = dense attention weight of token i among the prompt tokens (softmax of
 *          q.k_i * scale over i = 1..N),
 *   P(g) = softmax over teams of log n_g + q.l_g * scale (l_g the routing key),
 *   q_i  = P(g(i)) / n_g(i)  (a team's probability spread equally over its members),
 *   KL(p || q) = sum_i p_i log(p_i / q_i), natural logarithm (nats).
 * Tokens with p_i = 0 in floating point contribute 0 (the limit of x log x).
 * team_start[M+1], team_member[N] (members of team g are team_member[team_start[g] ..
 * team_start[g+1])), rep_key[M][d]. */
double orc_routing_kl(int d, const double *q, int64_t N, const double *k, int32_t M,
                      const int32_t *team_start, const int32_t *team_member,
                      const double *rep_key, double scale)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)N);
    double *phi = (double *)malloc(sizeof(double) * (size_t)M);
    double smax = -INFINITY, pmax = -INFINITY;
    for (int64_t i = 0; i < N; ++i) {
        s[i] = dot(q, k + i * d, d) * scale;
        if (s[i] > smax) smax = s[i];
    }
    for (int32_t g = 0; g < M; ++g) {
        int32_t n_g = team_start[g + 1] - team_start[g];
        phi[g] = log((double)n_g) + dot(q, rep_key + (int64_t)g * d, d) * scale;
        if (phi[g] > pmax) pmax = phi[g];
    }
    double Z = 0.0, Zr = 0.0;
    for (int64_t i = 0; i < N; ++i) Z += exp(s[i] - smax);
    for (int32_t g = 0; g < M; ++g) Zr += exp(phi[g] - pmax);
    double kl = 0.0;
    for (int32_t g = 0; g < M; ++g) {
        int32_t n_g = team_start[g + 1] - team_start[g];
        /* log q_i for the members of g */
        double log_q = (phi[g] - pmax) - log(Zr) - log((double)n_g);
        for (int32_t a = team_start[g]; a < team_start[g + 1]; ++a) {
            int64_t i = team_member[a];
            double log_p = (s[i] - smax) - log(Z);
            double p = exp(log_p);
            if (p > 0.0) kl += p * (log_p - log_q);
        }
    }
    free(s);
    free(phi);
    return kl;
}

/* A real number stored as a 16-bit routing key and read back: fp64 -> fp32 (round to nearest),
 * then fp32 -> the element type (round to nearest, ties to even). half = 0: bf16 (the upper 16
 * bits of the fp32 pattern). half = 1: IEEE binary16 (10 fraction bits, smallest normal 2^-14,
 * gradual underflow in steps of 2^-24, overflow to infinity from 65520). */
double orc_round_to_elem(double x, int half)
{
    float f = (float)x;
    if (!half) {
        uint32_t bits;
        memcpy(&bits, &f, sizeof bits);
        uint32_t rounded = (bits + 0x7FFFu + ((bits >> 16) & 1u)) & 0xFFFF0000u;
        float back;
        memcpy(&back, &rounded, sizeof back);
        return (double)back;
    }
    if (f != f || isinf(f) || f == 0.0f) return (double)f;
    double a = fabs((double)f);
    int e;
    (void)frexp(a, &e);                                   /* a = m * 2^e with m in [0.5, 1) */
    int ulp_exp = e - 1 < -14 ? -24 : e - 11;             /* spacing of binary16 around a */
    double v = ldexp(nearbyint(ldexp(a, -ulp_exp)), ulp_exp);   /* nearbyint: ties to even */
    if (v > 65504.0) v = INFINITY;
    return f < 0.0f ? -v : v;
}

/* Centroid-guided baseline (Section "How closely routing follows dense attention" and the
 * appendix on the KL variants): every group is routed by the arithmetic mean of its keys
 * instead of an actual key; the routing logit still adds log n_g, sampling, correction and
 * estimator are unchanged. The paper forms the groups by k-means (orc_group_mean_keys_parents
 * takes any partition); here the groups are the contiguous parents of Algorithm 4.
 * For parent u: mean_u = (sum over its tokens in index order of k_i) / |C_u| in fp64, then
 * stored as a 16-bit value like every other routing key (orc_round_to_elem).
 * out_mean[n_parents][d] receives those values widened back to fp64. Returns n_parents. */
int32_t orc_group_mean_keys(int32_t N, int d, const double *keys, int32_t P, int half, double *out_mean)
{
    int32_t n_parents = (N + P - 1) / P;
    for (int32_t u = 0; u < n_parents; ++u) {
        int32_t lo = u * P, hi = (u + 1) * P < N ? (u + 1) * P : N;
        for (int j = 0; j < d; ++j) {
            double sum = 0.0;
            for (int32_t i = lo; i < hi; ++i) sum += keys[(int64_t)i * d + j];
            out_mean[(int64_t)u * d + j] = orc_round_to_elem(sum / (double)(hi - lo), half);
        }
    }
    return n_parents;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 3: parents from fitted centres                                  */
/* ------------------------------------------------------------------------- */

/* First line of Algorithm 3: the number of centres requested from the fit,
 * M_parent = min(N, max(2, floor(N / P))), for N >= 2. */
int32_t orc_kmeans_parent_count(int32_t N, int32_t P)
{
    int32_t m = N / P;
    if (m < 2) m = 2;
    if (m > N) m = N;
    return m;
}

/* Last two lines of Algorithm 3. The centres mu_u are an input (the fit that
 * produces them is orc_minibatch_kmeans below). Every key joins its nearest centre in squared
 * Euclidean distance, ties going to the smaller centre index; parents without
 * a key are omitted, the others keep the order of their centres.
 *   keys[N][d], centres[n_centres][d]
 *   label[N]                          centre index of each token
 *   parent_start[n_parents + 1], parent_member[N]   index lists, tokens increasing
 * Returns the number of non-empty parents. */
int32_t orc_nearest_centre_parents(int32_t N, int d, const double *keys,
                                   int32_t n_centres, const double *centres,
                                   int32_t *label, int32_t *parent_start, int32_t *parent_member)
{
    for (int32_t i = 0; i < N; ++i) {
        double best = INFINITY; int32_t arg = 0;
        for (int32_t u = 0; u < n_centres; ++u) {
            double dist = sqdist(keys + (int64_t)i * d, centres + (int64_t)u * d, d);
            if (dist < best) { best = dist; arg = u; }
        }
        label[i] = arg;
    }
    int32_t n_parents = 0, filled = 0;
    parent_start[0] = 0;
    for (int32_t u = 0; u < n_centres; ++u) {
        int32_t before = filled;
        for (int32_t i = 0; i < N; ++i)
            if (label[i] == u) parent_member[filled++] = i;
        if (filled > before) parent_start[++n_parents] = filled;
    }
    return n_parents;
}

/* The centroid-guided baseline on an arbitrary parent partition (the paper forms its groups by
 * k-means): one group per parent, members in increasing token index, routing key = arithmetic
 * mean of the parent's keys (fp64 sum in token order, one division), stored as a 16-bit value
 * (orc_round_to_elem) and widened back into out_mean[n_parents][d]. */
void orc_group_mean_keys_parents(int d, const double *keys, int32_t n_parents, const int32_t *parent_start,
                                 const int32_t *parent_member, int half, double *out_mean)
{
    for (int32_t u = 0; u < n_parents; ++u) {
        int32_t lo = parent_start[u], hi = parent_start[u + 1];
        for (int j = 0; j < d; ++j) {
            double sum = 0.0;
            for (int32_t a = lo; a < hi; ++a) sum += keys[(int64_t)parent_member[a] * d + j];
            out_mean[(int64_t)u * d + j] = orc_round_to_elem(sum / (double)(hi - lo), half);
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Algorithm 3, the fit: minibatch k-means with greedy k-means++ start        */
/* ------------------------------------------------------------------------- */

/* The paper names the routine and its settings (squared-Euclidean centres on the raw keys, greedy
 * k-means++ initialisation, minibatches sampled with replacement, cumulative-count centre updates,
 * a no-improvement stopping rule, a reassignment ratio, tolerance zero, a seed) and leaves the
 * rest to "the implementation default". This is the reading taken here, step by step; every random
 * choice is a word of the Philox stream with counter (slot, tag, stream, step) and the seed as key,
 * so the fit is a pure function of its arguments.
 *
 *  1. Initialisation sample: n_init = min(N, max(3 * batch, 3 * k)) distinct keys, the head of a
 *     Fisher-Yates shuffle of 0..N-1 (tag 1: position i swaps with i + floor(word * (N - i) / 2^32)).
 *  2. Greedy k-means++ on the sample, L = 2 + floor(ln k) trials per centre (tag 2): the first
 *     centre is a uniform sample point; each later one is the best of L points drawn with
 *     probability proportional to the squared distance to the nearest centre chosen so far (inverse
 *     CDF over the sample in order), "best" meaning the smallest resulting potential
 *     sum_i min(closest_i, |x_i - candidate|^2), ties to the earlier trial.
 *     Sums over the sample (the potential of a trial, the running sums of the inverse CDF) are
 *     taken in blocks of 128 consecutive sample points: the points of a block are added in order,
 *     the block sums are added in order, and a running sum is (sum of the earlier blocks) + (sum
 *     inside its block so far). The paper leaves the order open; this one lets the blocks be
 *     summed side by side.
 *  3. At most max_iter * ceil(N / batch) minibatch steps. Step t draws `batch` indices uniformly
 *     with replacement (tag 3), assigns each to its nearest centre (ties to the smaller index),
 *     then moves every centre that received points to the mean of all points it has received so
 *     far: c <- (c * count + sum of the new points) / (count + n), count <- count + n.
 *  4. Reassignment, at steps with (t + 1) divisible by 10 + floor(smallest count): centres whose
 *     count is below ratio * (largest count), at most batch / 2 of them, in index order, jump onto
 *     distinct points of the current minibatch (head of a Fisher-Yates shuffle of its slots, tag 4)
 *     and take the smallest count among the centres that stay.
 *  5. Stopping: the per-point inertia of each minibatch (measured before its update) feeds an
 *     exponentially weighted average with alpha = min(1, 2 * batch / (N + 1)); the fit stops after
 *     `patience` consecutive steps without a new minimum of that average.
 * Returns the number of steps run; centres[k][d] are the fp64 centres. */
static uint32_t km_word(uint64_t seed, uint32_t slot, uint32_t tag, uint32_t stream, uint32_t step)
{
    uint32_t ctr[4] = {slot, tag, stream, step};
    uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return out[0];
}

static int32_t km_index(uint32_t word, int32_t n) { return (int32_t)(((uint64_t)word * (uint64_t)n) >> 32); }

/* Sum of x[0..n) in blocks of 128 (see step 2 above); cum, when given, receives the running sums. */
#define KM_SUM_BLOCK 128
static double km_blocked_sum(const double *x, int32_t n, double *cum)
{
    double off = 0.0;
    for (int32_t b0 = 0; b0 < n; b0 += KM_SUM_BLOCK) {
        int32_t e = b0 + KM_SUM_BLOCK < n ? b0 + KM_SUM_BLOCK : n;
        double w = 0.0;
        for (int32_t i = b0; i < e; ++i) {
            w += x[i];
            if (cum) cum[i] = off + w;
        }
        off += w;
    }
    return off;
}

int32_t orc_minibatch_kmeans(int32_t N, int d, const double *keys, int32_t k, int32_t batch, int32_t max_iter,
                             int32_t patience, double ratio, uint64_t seed, uint32_t stream, double *centres)
{
    /* 1. initialisation sample */
    int32_t n_init = 3 * batch > 3 * k ? 3 * batch : 3 * k;
    if (n_init > N) n_init = N;
    int32_t *perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    for (int32_t i = 0; i < N; ++i) perm[i] = i;
    for (int32_t i = 0; i < n_init; ++i) {
        int32_t r = i + km_index(km_word(seed, (uint32_t)i, 1u, stream, 0u), N - i);
        int32_t t = perm[i]; perm[i] = perm[r]; perm[r] = t;
    }
    /* 2. greedy k-means++ */
    int32_t L = 2 + (int32_t)floor(log((double)k));
    double *closest = (double *)malloc(sizeof(double) * (size_t)n_init);
    double *cand = (double *)malloc(sizeof(double) * (size_t)n_init * (size_t)L);
    int32_t *pick = (int32_t *)malloc(sizeof(int32_t) * (size_t)L);
    {
        int32_t first = km_index(km_word(seed, 0u, 2u, stream, 0u), n_init);
        memcpy(centres, keys + (int64_t)perm[first] * d, sizeof(double) * (size_t)d);
        for (int32_t i = 0; i < n_init; ++i) closest[i] = sqdist(keys + (int64_t)perm[i] * d, centres, d);
    }
    double *cum = (double *)malloc(sizeof(double) * (size_t)n_init);
    double *term = (double *)malloc(sizeof(double) * (size_t)n_init);
    for (int32_t c = 1; c < k; ++c) {
        double total = km_blocked_sum(closest, n_init, cum);
        for (int32_t l = 0; l < L; ++l) {
            double target = orc_uniform_open(km_word(seed, (uint32_t)l, 2u, stream, (uint32_t)c)) * total;
            int32_t at = n_init - 1;
            for (int32_t i = 0; i < n_init; ++i) {
                if (cum[i] > target) { at = i; break; }
            }
            pick[l] = at;
        }
        int32_t best = 0;
        double best_pot = INFINITY;
        for (int32_t l = 0; l < L; ++l) {
            const double *x = keys + (int64_t)perm[pick[l]] * d;
            for (int32_t i = 0; i < n_init; ++i) {
                double dist = sqdist(keys + (int64_t)perm[i] * d, x, d);
                cand[(int64_t)l * n_init + i] = dist;
                term[i] = dist < closest[i] ? dist : closest[i];
            }
            double pot = km_blocked_sum(term, n_init, NULL);
            if (pot < best_pot) { best_pot = pot; best = l; }
        }
        memcpy(centres + (int64_t)c * d, keys + (int64_t)perm[pick[best]] * d, sizeof(double) * (size_t)d);
        for (int32_t i = 0; i < n_init; ++i) {
            double dist = cand[(int64_t)best * n_init + i];
            if (dist < closest[i]) closest[i] = dist;
        }
    }
    free(term); free(cum); free(pick); free(cand); free(closest); free(perm);

    /* 3.-5. minibatch steps */
    double *count = (double *)calloc((size_t)k, sizeof(double));
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)batch);
    int32_t *label = (int32_t *)malloc(sizeof(int32_t) * (size_t)batch);
    int32_t *slots = (int32_t *)malloc(sizeof(int32_t) * (size_t)batch);
    double *sum = (double *)malloc(sizeof(double) * (size_t)d);
    int64_t t_max = (int64_t)max_iter * ((N + batch - 1) / batch);
    double alpha = 2.0 * (double)batch / ((double)N + 1.0);
    if (alpha > 1.0) alpha = 1.0;
    double ewa = 0.0, ewa_min = INFINITY;
    int32_t bad = 0, steps = 0;
    for (int64_t t = 0; t < t_max; ++t) {
        double inertia = 0.0;
        for (int32_t s = 0; s < batch; ++s) {
            idx[s] = km_index(km_word(seed, (uint32_t)s, 3u, stream, (uint32_t)t), N);
            double bestd = INFINITY; int32_t arg = 0;
            for (int32_t u = 0; u < k; ++u) {
                double dist = sqdist(keys + (int64_t)idx[s] * d, centres + (int64_t)u * d, d);
                if (dist < bestd) { bestd = dist; arg = u; }
            }
            label[s] = arg;
            inertia += bestd;
        }
        /* cumulative-count update */
        for (int32_t u = 0; u < k; ++u) {
            int32_t n = 0;
            for (int j = 0; j < d; ++j) sum[j] = 0.0;
            for (int32_t s = 0; s < batch; ++s) {
                if (label[s] != u) continue;
                ++n;
                for (int j = 0; j < d; ++j) sum[j] += keys[(int64_t)idx[s] * d + j];
            }
            if (n == 0) continue;
            double grown = count[u] + (double)n;
            for (int j = 0; j < d; ++j)
                centres[(int64_t)u * d + j] = (centres[(int64_t)u * d + j] * count[u] + sum[j]) / grown;
            count[u] = grown;
        }
        /* reassignment of starved centres */
        {
            double cmin = INFINITY, cmax = 0.0;
            for (int32_t u = 0; u < k; ++u) { if (count[u] < cmin) cmin = count[u]; if (count[u] > cmax) cmax = count[u]; }
            int64_t period = 10 + (int64_t)floor(cmin);
            if (ratio > 0.0 && (t + 1) % period == 0) {
                double thr = ratio * cmax;
                int32_t n_move = 0, cap = batch / 2;
                double keep_min = INFINITY;
                for (int32_t u = 0; u < k; ++u) {
                    if (count[u] < thr && n_move < cap) ++n_move;
                    else if (count[u] < keep_min) keep_min = count[u];
                }
                if (n_move > 0) {
                    for (int32_t s = 0; s < batch; ++s) slots[s] = s;
                    for (int32_t i = 0; i < n_move; ++i) {
                        int32_t r = i + km_index(km_word(seed, (uint32_t)i, 4u, stream, (uint32_t)t), batch - i);
                        int32_t tmp = slots[i]; slots[i] = slots[r]; slots[r] = tmp;
                    }
                    int32_t moved = 0;
                    for (int32_t u = 0; u < k && moved < n_move; ++u) {
                        if (!(count[u] < thr)) continue;
                        memcpy(centres + (int64_t)u * d, keys + (int64_t)idx[slots[moved]] * d, sizeof(double) * (size_t)d);
                        count[u] = keep_min;
                        ++moved;
                    }
                }
            }
        }
        /* stopping rule */
        ++steps;
        double per_point = inertia / (double)batch;
        ewa = t == 0 ? per_point : ewa * (1.0 - alpha) + per_point * alpha;
        if (ewa < ewa_min) { ewa_min = ewa; bad = 0; }
        else if (++bad >= patience) break;
    }
    free(sum); free(slots); free(label); free(idx); free(count);
    return steps;
}

/* Shared-row accounting for a shared-latent cache, Eq. (mla-logical-access): per decoding call c,
 * r[c] routing rows (one per representative), u[c] rows in the union over all heads of the
 * selected prompt members and the exact suffix, d[c] rows a dense call reads. One row stands for a
 * token's shared latent and rotary key; a row used in routing and in attention counts in both.
 * Counts are pooled over the calls before the division. Returns the percentage. */
double orc_mla_logical_access_pct(int64_t n_calls, const int64_t *r, const int64_t *u, const int64_t *d)
{
    double num = 0.0, den = 0.0;
    for (int64_t c = 0; c < n_calls; ++c) {
        num += (double)r[c] + (double)u[c];
        den += (double)d[c];
    }
    return 100.0 * num / den;
}
