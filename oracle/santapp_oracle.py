"""ctypes front end of the fp64 CPU oracle (oracle/santapp_oracle.c).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the tests, the smoke check and the
benchmark's cpu-baseline / reference arm import this module. It marshals numpy
arrays into the C functions and holds no arithmetic of the method itself.
"""
import ctypes
import os

import numpy as np

from . import build_oracle

_c = ctypes
_f64p = np.ctypeslib.ndpointer(dtype=np.float64, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(dtype=np.int32, flags="C_CONTIGUOUS")
_i64p = np.ctypeslib.ndpointer(dtype=np.int64, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(dtype=np.uint32, flags="C_CONTIGUOUS")

_lib = None


def lib():
    global _lib
    if _lib is None:
        path = build_oracle.build()
        L = ctypes.CDLL(path)
        L.orc_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
        L.orc_philox4x32_10.restype = None
        L.orc_team_word.argtypes = [_c.c_uint64, _c.c_uint32, _c.c_uint32, _c.c_uint32, _c.c_uint32]
        L.orc_team_word.restype = _c.c_uint32
        L.orc_uniform_open.argtypes = [_c.c_uint32]
        L.orc_uniform_open.restype = _c.c_double
        L.orc_gumbel.argtypes = [_c.c_uint32]
        L.orc_gumbel.restype = _c.c_double
        L.orc_gumbel_many.argtypes = [_c.c_uint64, _c.c_uint32, _c.c_uint32, _c.c_uint32, _c.c_int32, _f64p]
        L.orc_gumbel_many.restype = None
        L.orc_dense_head.argtypes = [_c.c_int, _f64p, _c.c_int64, _f64p, _f64p, _c.c_double, _f64p]
        L.orc_dense_head.restype = None
        L.orc_dense_head_two.argtypes = [_c.c_int, _f64p, _c.c_int64, _f64p, _f64p,
                                         _c.c_int64, _f64p, _f64p, _c.c_double, _f64p]
        L.orc_dense_head_two.restype = None
        L.orc_contiguous_parents.argtypes = [_c.c_int32, _c.c_int32, _i32p]
        L.orc_contiguous_parents.restype = _c.c_int32
        L.orc_build_teams.argtypes = [_c.c_int32, _c.c_int, _f64p, _c.c_int32, _i32p, _i32p, _c.c_int32,
                                      _i32p, _i32p, _i32p]
        L.orc_build_teams.restype = _c.c_int32
        vp = _c.c_void_p
        L.orc_decode_head_given_gumbel.argtypes = [
            _c.c_int, _f64p, _c.c_int64, _f64p, _f64p,
            _c.c_int32, _i32p, _i32p, _f64p,
            _c.c_int64, _f64p, _f64p,
            _c.c_int32, _f64p, _c.c_double,
            _f64p, _i32p, _f64p, vp, vp, vp, vp, vp, vp, _c.c_int, vp]
        L.orc_decode_head_given_gumbel.restype = _c.c_int32
        L.orc_decode_head.argtypes = [
            _c.c_int, _f64p, _c.c_int64, _f64p, _f64p,
            _c.c_int32, _i32p, _i32p, _f64p,
            _c.c_int64, _f64p, _f64p,
            _c.c_int32, _c.c_uint64, _c.c_uint32, _c.c_uint32, _c.c_uint32, _c.c_double,
            _f64p, _i32p, _f64p, vp, vp]
        L.orc_decode_head.restype = _c.c_int32
        L.orc_decode_step.argtypes = [
            _c.c_int, _c.c_int32, _c.c_int32, _f64p,
            _c.c_int64, _f64p, _f64p,
            _c.c_int32, _i32p, _i32p, _i32p, _f64p,
            _c.c_int64, _f64p, _f64p,
            _c.c_int32, _c.c_uint64, _c.c_uint32, _c.c_uint32, _c.c_double,
            _f64p, _i32p, _f64p, _f64p, _f64p, _c.c_int32]
        L.orc_decode_step.restype = None
        L.orc_dense_step.argtypes = [
            _c.c_int, _c.c_int32, _c.c_int32, _f64p,
            _c.c_int64, _f64p, _f64p, _c.c_int64, _f64p, _f64p, _c.c_double, _f64p, _c.c_int32]
        L.orc_dense_step.restype = None
        L.orc_has_openmp.restype = _c.c_int32
        L.orc_team_budget.argtypes = [_c.c_int32] * 4
        L.orc_team_budget.restype = _c.c_int32
        L.orc_logical_access_pct.argtypes = [_c.c_int64, _i64p, _i64p, _i64p, _i64p]
        L.orc_logical_access_pct.restype = _c.c_double
        L.orc_union_rows.argtypes = [_c.c_int32, _i32p, _c.c_int32, _c.c_int32, _i32p]
        L.orc_union_rows.restype = _c.c_int64
        L.orc_dense_kv_bytes.argtypes = [_c.c_int64, _c.c_int32, _c.c_int32, _c.c_int32]
        L.orc_dense_kv_bytes.restype = _c.c_double
        L.orc_routing_kl.argtypes = [_c.c_int, _f64p, _c.c_int64, _f64p, _c.c_int32, _i32p, _i32p, _f64p, _c.c_double]
        L.orc_routing_kl.restype = _c.c_double
        L.orc_group_mean_keys.argtypes = [_c.c_int32, _c.c_int, _f64p, _c.c_int32, _c.c_int, _f64p]
        L.orc_round_to_elem.argtypes = [_c.c_double, _c.c_int]
        L.orc_round_to_elem.restype = _c.c_double
        L.orc_group_mean_keys.restype = _c.c_int32
        L.orc_group_mean_keys_parents.argtypes = [_c.c_int, _f64p, _c.c_int32, _i32p, _i32p, _c.c_int, _f64p]
        L.orc_group_mean_keys_parents.restype = None
        L.orc_mla_logical_access_pct.argtypes = [_c.c_int64, _i64p, _i64p, _i64p]
        L.orc_mla_logical_access_pct.restype = _c.c_double
        L.orc_minibatch_kmeans.argtypes = [_c.c_int32, _c.c_int, _f64p, _c.c_int32, _c.c_int32, _c.c_int32, _c.c_int32,
                                           _c.c_double, _c.c_uint64, _c.c_uint32, _f64p]
        L.orc_minibatch_kmeans.restype = _c.c_int32
        L.orc_kmeans_parent_count.argtypes = [_c.c_int32, _c.c_int32]
        L.orc_kmeans_parent_count.restype = _c.c_int32
        L.orc_nearest_centre_parents.argtypes = [_c.c_int32, _c.c_int, _f64p, _c.c_int32, _f64p, _i32p, _i32p, _i32p]
        L.orc_nearest_centre_parents.restype = _c.c_int32
        _lib = L
    return _lib


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _empty_rows(d):
    return np.zeros((1, d), dtype=np.float64)


def philox4x32_10(ctr, key):
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(np.asarray(ctr, dtype=np.uint32), np.asarray(key, dtype=np.uint32), out)
    return out


def team_word(seed, step, head, stream, g):
    return int(lib().orc_team_word(seed, step, head, stream, g))


def uniform_open(x):
    return float(lib().orc_uniform_open(x))


def gumbel(x):
    return float(lib().orc_gumbel(x))


def gumbel_many(seed, step, head, stream, M):
    out = np.zeros(max(M, 1), dtype=np.float64)
    lib().orc_gumbel_many(seed, step, head, stream, M, out)
    return out[:M]


def dense_head(q, k, v, scale):
    q, k, v = _f64(q), _f64(k), _f64(v)
    d = q.shape[0]
    o = np.zeros(d, dtype=np.float64)
    lib().orc_dense_head(d, q, k.shape[0], k, v, scale, o)
    return o


def dense_head_two(q, k, v, ks, vs, scale):
    q, k, v = _f64(q), _f64(k), _f64(v)
    d = q.shape[0]
    t = 0 if ks is None else ks.shape[0]
    ks = _f64(ks) if t else _empty_rows(d)
    vs = _f64(vs) if t else _empty_rows(d)
    o = np.zeros(d, dtype=np.float64)
    lib().orc_dense_head_two(d, q, k.shape[0], k, v, t, ks, vs, scale, o)
    return o


def contiguous_parents(N, P):
    buf = np.zeros((N + P - 1) // P + 1, dtype=np.int32)
    n = lib().orc_contiguous_parents(N, P, buf)
    return buf[: n + 1].copy()


def build_teams(keys, parent_start, parent_member, R):
    """Algorithm 2. Returns (team_start[M+1], team_member[N], rep_row[M])."""
    keys = _f64(keys)
    N, d = keys.shape
    parent_start = _i32(parent_start)
    parent_member = _i32(parent_member)
    n_parents = parent_start.shape[0] - 1
    team_start = np.zeros(N + 1, dtype=np.int32)
    team_member = np.zeros(N, dtype=np.int32)
    rep_row = np.zeros(N, dtype=np.int32)
    M = lib().orc_build_teams(N, d, keys, n_parents, parent_start, parent_member, R,
                              team_start, team_member, rep_row)
    return team_start[: M + 1].copy(), team_member, rep_row[:M].copy()


def build_teams_contiguous(keys, P, R):
    N = keys.shape[0]
    ps = contiguous_parents(N, P)
    return build_teams(keys, ps, np.arange(N, dtype=np.int32), R)


class HeadResult:
    __slots__ = ("o", "sel", "logc", "tau", "margin", "phi", "y", "U", "Z", "shift")


def decode_head_given_gumbel(q, k_cache, v_cache, team_start, team_member, rep_key, ks, vs, K,
                             gumbel_draws, scale, shift=None, want_routing=False):
    """Algorithm 1 with the M Gumbel draws passed in."""
    q, k_cache, v_cache, rep_key = _f64(q), _f64(k_cache), _f64(v_cache), _f64(rep_key)
    team_start, team_member = _i32(team_start), _i32(team_member)
    d = q.shape[0]
    M = team_start.shape[0] - 1
    t = 0 if ks is None else ks.shape[0]
    ks = _f64(ks) if t else _empty_rows(d)
    vs = _f64(vs) if t else _empty_rows(d)
    Ke = min(K, M)
    g = _f64(gumbel_draws) if gumbel_draws is not None else np.zeros(max(M, 1))
    o = np.zeros(d)
    sel = np.zeros(max(Ke, 1), dtype=np.int32)
    logc = np.zeros(max(Ke, 1))
    tau, margin, Z, sh = (_c.c_double() for _ in range(4))
    U = np.zeros(d)
    phi = np.zeros(max(M, 1)) if want_routing else None
    y = np.zeros(max(M, 1)) if want_routing else None
    use_shift = 0
    if shift is not None:
        use_shift = 1
        sh.value = shift
    lib().orc_decode_head_given_gumbel(
        d, q, k_cache.shape[0], k_cache, v_cache, M, team_start, team_member, rep_key,
        t, ks, vs, K, g, scale, o, sel, logc,
        _c.addressof(tau), _c.addressof(margin),
        phi.ctypes.data if want_routing else None, y.ctypes.data if want_routing else None,
        U.ctypes.data, _c.addressof(Z), use_shift, _c.addressof(sh))
    r = HeadResult()
    r.o, r.sel, r.logc = o, sel[:Ke], logc[:Ke]
    r.tau, r.margin, r.U, r.Z, r.shift = tau.value, margin.value, U, Z.value, sh.value
    r.phi = phi[:M] if want_routing else None
    r.y = y[:M] if want_routing else None
    return r


def decode_head(q, k_cache, v_cache, team_start, team_member, rep_key, ks, vs, K,
                seed, step, head, stream, scale):
    """Algorithm 1 with draws from the Philox stream (seed; step, head, stream)."""
    q, k_cache, v_cache, rep_key = _f64(q), _f64(k_cache), _f64(v_cache), _f64(rep_key)
    team_start, team_member = _i32(team_start), _i32(team_member)
    d = q.shape[0]
    M = team_start.shape[0] - 1
    t = 0 if ks is None else ks.shape[0]
    ks = _f64(ks) if t else _empty_rows(d)
    vs = _f64(vs) if t else _empty_rows(d)
    Ke = min(K, M)
    o = np.zeros(d)
    sel = np.zeros(max(Ke, 1), dtype=np.int32)
    logc = np.zeros(max(Ke, 1))
    tau, margin = _c.c_double(), _c.c_double()
    lib().orc_decode_head(d, q, k_cache.shape[0], k_cache, v_cache, M, team_start, team_member,
                          rep_key, t, ks, vs, K, seed, step, head, stream, scale,
                          o, sel, logc, _c.addressof(tau), _c.addressof(margin))
    r = HeadResult()
    r.o, r.sel, r.logc, r.tau, r.margin = o, sel[:Ke], logc[:Ke], tau.value, margin.value
    r.phi = r.y = r.U = r.Z = r.shift = None
    return r


class StepResult:
    __slots__ = ("o", "sel", "logc", "tau", "margin")


def decode_step(q, k_cache, v_cache, M, team_start, team_member, rep_key, ks, vs, K,
                seed, step, stream, scale, n_threads=1):
    """One sequence, all query heads under GQA.

    q [n_q, d]; k_cache/v_cache [n_kv, N, d]; M [n_kv]; team_start [n_kv, M_max+1];
    team_member [n_kv, N]; rep_key [n_kv, M_max, d]; ks/vs [n_kv, t, d] or None.
    """
    q, k_cache, v_cache, rep_key = _f64(q), _f64(k_cache), _f64(v_cache), _f64(rep_key)
    team_start, team_member, M = _i32(team_start), _i32(team_member), _i32(M)
    n_q, d = q.shape
    n_kv, N, _ = k_cache.shape
    M_max = team_start.shape[1] - 1
    t = 0 if ks is None else ks.shape[1]
    ks = _f64(ks) if t else np.zeros((n_kv, 1, d))
    vs = _f64(vs) if t else np.zeros((n_kv, 1, d))
    o = np.zeros((n_q, d))
    sel = np.full((n_q, K), -1, dtype=np.int32)
    logc = np.zeros((n_q, K))
    tau = np.zeros(n_q)
    margin = np.zeros(n_q)
    lib().orc_decode_step(d, n_q, n_kv, q, N, k_cache, v_cache, M_max, M, team_start, team_member,
                          rep_key, t, ks, vs, K, seed, step, stream, scale,
                          o, sel, logc, tau, margin, n_threads)
    r = StepResult()
    r.o, r.sel, r.logc, r.tau, r.margin = o, sel, logc, tau, margin
    return r


def dense_step(q, k_cache, v_cache, ks, vs, scale, n_threads=1):
    q, k_cache, v_cache = _f64(q), _f64(k_cache), _f64(v_cache)
    n_q, d = q.shape
    n_kv, N, _ = k_cache.shape
    t = 0 if ks is None else ks.shape[1]
    ks = _f64(ks) if t else np.zeros((n_kv, 1, d))
    vs = _f64(vs) if t else np.zeros((n_kv, 1, d))
    o = np.zeros((n_q, d))
    lib().orc_dense_step(d, n_q, n_kv, q, N, k_cache, v_cache, t, ks, vs, scale, o, n_threads)
    return o


def has_openmp():
    return bool(lib().orc_has_openmp())


def team_budget(M, S, P, R):
    return int(lib().orc_team_budget(M, S, P, R))


def logical_access_pct(m, u, e, Ncache):
    a = [np.ascontiguousarray(x, dtype=np.int64).reshape(-1) for x in (m, u, e, Ncache)]
    return float(lib().orc_logical_access_pct(a[0].shape[0], *a))


def union_rows(team_start, sel):
    team_start = _i32(team_start)
    sel = _i32(sel)
    if sel.ndim == 1:
        sel = sel[None, :]
    return int(lib().orc_union_rows(team_start.shape[0] - 1, team_start, sel.shape[0], sel.shape[1], sel))


def dense_kv_bytes(N, n_kv, d, bytes_per_el):
    return float(lib().orc_dense_kv_bytes(N, n_kv, d, bytes_per_el))


def routing_kl(q, k, team_start, team_member, rep_key, scale):
    """KL(p || q) in nats between dense attention over the prompt and the routing proposal spread
    over team members (Eq. diagnostic-kl), for one query head."""
    q, k, rep_key = _f64(q), _f64(k), _f64(rep_key)
    team_start, team_member = _i32(team_start), _i32(team_member)
    return float(lib().orc_routing_kl(q.shape[0], q, k.shape[0], k, team_start.shape[0] - 1, team_start,
                                      team_member, rep_key, scale))


def round_to_elem(x, elem="bf16"):
    """fp64 -> fp32 -> the 16-bit element type (round to nearest even), as a float64 value."""
    return float(lib().orc_round_to_elem(float(x), 1 if elem == "fp16" else 0))


def group_mean_keys(keys, P, elem="bf16"):
    """Centroid-guided baseline on contiguous parents: (team_start, team_member, mean_key) with one
    group per parent, members in token order, and the parent's arithmetic-mean key rounded to a
    value of the 16-bit element type as its routing key."""
    keys = _f64(keys)
    N, d = keys.shape
    n_parents = (N + P - 1) // P
    mean = np.zeros((n_parents, d))
    got = lib().orc_group_mean_keys(N, d, keys, P, 1 if elem == "fp16" else 0, mean)
    assert got == n_parents
    return contiguous_parents(N, P), np.arange(N, dtype=np.int32), mean


def kmeans_parent_count(N, P):
    """First line of Algorithm 3: min(N, max(2, N // P))."""
    return int(lib().orc_kmeans_parent_count(N, P))


def nearest_centre_parents(keys, centres):
    """Last two lines of Algorithm 3 for given centres. Returns (label[N], parent_start, parent_member):
    nearest centre per token (ties to the smaller centre index) and the non-empty parents as index
    lists in centre order, tokens increasing."""
    keys, centres = _f64(keys), _f64(centres)
    N, d = keys.shape
    label = np.zeros(N, dtype=np.int32)
    parent_start = np.zeros(centres.shape[0] + 1, dtype=np.int32)
    parent_member = np.zeros(N, dtype=np.int32)
    n = lib().orc_nearest_centre_parents(N, d, keys, centres.shape[0], centres, label, parent_start, parent_member)
    return label, parent_start[: n + 1].copy(), parent_member


def group_mean_keys_parents(keys, parent_start, parent_member, elem="bf16"):
    """Centroid-guided groups on a given partition: (team_start, team_member, mean_key), one group
    per parent, members in token order, the mean key rounded to a value of the 16-bit element type."""
    keys = _f64(keys)
    parent_start, parent_member = _i32(parent_start), _i32(parent_member)
    n = parent_start.shape[0] - 1
    mean = np.zeros((n, keys.shape[1]))
    lib().orc_group_mean_keys_parents(keys.shape[1], keys, n, parent_start, parent_member,
                                      1 if elem == "fp16" else 0, mean)
    return parent_start.copy(), parent_member.copy(), mean


def minibatch_kmeans(keys, k, batch=4096, max_iter=100, patience=10, ratio=0.01, seed=0, stream=0):
    """The fit of Algorithm 3 with the paper's settings as defaults. Returns (centres[k, d] fp64, steps)."""
    keys = _f64(keys)
    N, d = keys.shape
    centres = np.zeros((k, d))
    steps = lib().orc_minibatch_kmeans(N, d, keys, k, batch, max_iter, patience, ratio, seed, stream, centres)
    return centres, int(steps)


def shared_latent_records(rows, d_latent, P, R):
    """Teams of a shared-latent cache (appendix "Token sparsity after latent compression"): rows
    [N, d_latent + d_rope] hold a content latent followed by a rotary key; contiguous parents
    (Algorithm 4) and Algorithm 2 run on the content latents alone, and a team's routing key is
    its representative's whole row. Returns (team_start, team_member, rep_rows)."""
    rows = _f64(rows)
    ts, tm, rep = build_teams_contiguous(np.ascontiguousarray(rows[:, :d_latent]), P, R)
    return ts, tm, np.ascontiguousarray(rows[rep])


def shared_latent_step(q, rows, d_latent, team_start, team_member, rep_rows, suffix_rows, K, seed, step, stream,
                       scale, n_threads=1):
    """Algorithm 1 for the n_q heads that share one row per token: a head's logit is its query
    against the whole row (latent and rotary part), its value the row's latent part. Argument
    marshalling only: one KV "head", keys = rows, values = rows with the rotary columns zeroed
    (they add exact zeros to every sum). Returns the StepResult with o [n_q, d_latent]."""
    rows, q = _f64(rows), _f64(q)
    vals = rows.copy()
    vals[:, d_latent:] = 0.0
    ks = vs = None
    if suffix_rows is not None and len(suffix_rows):
        ks = _f64(suffix_rows)[None]
        vs = ks.copy()
        vs[:, :, d_latent:] = 0.0
    M = np.array([len(team_start) - 1], dtype=np.int32)
    r = decode_step(q, rows[None], vals[None], M, _i32(team_start)[None], _i32(team_member)[None], _f64(rep_rows)[None],
                    ks, vs, K, seed, step, stream, scale, n_threads=n_threads)
    r.o = np.ascontiguousarray(r.o[:, :d_latent])
    return r


def mla_logical_access_pct(r, u, d):
    """Shared-row logical access of Eq. (mla-logical-access), pooled over the calls."""
    r, u, d = (np.ascontiguousarray(a, dtype=np.int64) for a in (r, u, d))
    return float(lib().orc_mla_logical_access_pct(r.shape[0], r, u, d))
