"""Pins for the oracle's shared-latent rows (appendix "Token sparsity after latent compression"):
16 heads share one row per token, a content latent of 512 numbers followed by a rotary key of 64;
a head's logit uses the whole row, its value is the latent part; teams come from the latents alone
and are shared by the heads, which draw independently; access is counted in shared rows over the
union of the heads' selections (Eq. mla-logical-access)."""
import math

import numpy as np
from scipy.special import softmax

from oracle import santapp_oracle as orc

D_LAT, D_ROPE, HEADS = 512, 64, 16


def _case(seed, N=320, t=3):
    rng = np.random.default_rng(seed)
    centres = rng.standard_normal((12, D_LAT))
    rows = np.concatenate([centres[rng.integers(0, 12, N)] + 0.3 * rng.standard_normal((N, D_LAT)),
                           rng.standard_normal((N, D_ROPE))], axis=1)
    suffix = np.concatenate([centres[rng.integers(0, 12, t)] + 0.3 * rng.standard_normal((t, D_LAT)),
                             rng.standard_normal((t, D_ROPE))], axis=1)
    q = 0.2 * rng.standard_normal((HEADS, D_LAT + D_ROPE)) + 0.1 * rows[rng.integers(0, N, HEADS)]
    return rows, suffix, q, 1.0 / math.sqrt(D_LAT + D_ROPE)


def test_every_team_selected_is_dense_attention_over_the_shared_rows():
    rows, suffix, q, scale = _case(1)
    ts, tm, rep = orc.shared_latent_records(rows, D_LAT, 16, 4)
    M = len(ts) - 1
    r = orc.shared_latent_step(q, rows, D_LAT, ts, tm, rep, suffix, M + 5, 0, 0, 0, scale)
    allrows = np.concatenate([rows, suffix])
    w = softmax(q @ allrows.T * scale, axis=1)                 # whole row in the logit
    assert np.allclose(r.o, w @ allrows[:, :D_LAT], rtol=0, atol=1e-12)   # latent part as the value
    assert r.o.shape == (HEADS, D_LAT) and np.all(np.isnan(r.tau))


def test_teams_come_from_the_latents_and_routing_keys_are_whole_rows():
    rows, suffix, q, scale = _case(2)
    ts, tm, rep = orc.shared_latent_records(rows, D_LAT, 16, 4)
    other = rows.copy()
    other[:, D_LAT:] = np.random.default_rng(9).standard_normal((rows.shape[0], D_ROPE))    # other rotary parts
    ts2, tm2, rep2 = orc.shared_latent_records(other, D_LAT, 16, 4)
    assert np.array_equal(ts, ts2) and np.array_equal(tm, tm2)          # the partition ignores them
    assert np.array_equal(rep[:, :D_LAT], rep2[:, :D_LAT]) and not np.array_equal(rep, rep2)
    # ... but the draw does not: the routing logit is q against the representative's whole row
    K = 8
    a = orc.shared_latent_step(q, rows, D_LAT, ts, tm, rep, suffix, K, 3, 1, 0, scale)
    b = orc.shared_latent_step(q, rows, D_LAT, ts, tm, rep2, suffix, K, 3, 1, 0, scale)
    assert not np.array_equal(a.sel, b.sel)
    h, g = 5, int(a.sel[5, 0])
    gum = orc.gumbel_many(3, 1, h, 0, len(ts) - 1)
    assert g in a.sel[h]
    y = np.array([math.log(ts[x + 1] - ts[x]) + float(q[h] @ rep[x]) * scale for x in range(len(ts) - 1)]) + gum
    assert np.array_equal(a.sel[h], np.argsort(-y, kind="stable")[:K])


def test_a_head_alone_equals_the_head_beside_its_fifteen_siblings_and_siblings_differ():
    rows, suffix, q, scale = _case(3)
    ts, tm, rep = orc.shared_latent_records(rows, D_LAT, 16, 4)
    K = 6
    r = orc.shared_latent_step(q, rows, D_LAT, ts, tm, rep, suffix, K, 11, 4, 2, scale)
    vals = rows.copy(); vals[:, D_LAT:] = 0
    vs = suffix.copy(); vs[:, D_LAT:] = 0
    for h in (0, 7, 15):
        alone = orc.decode_head(q[h], rows, vals, ts, tm, rep, suffix, vs, K, 11, 4, h, 2, scale)
        assert np.array_equal(alone.sel, r.sel[h]) and np.array_equal(alone.o[:D_LAT], r.o[h])
    assert len({tuple(s) for s in r.sel.tolist()}) > 1                  # independent draws per head


def test_shared_row_accounting_on_the_union_over_all_heads():
    rows, suffix, q, scale = _case(4, N=640, t=5)
    ts, tm, rep = orc.shared_latent_records(rows, D_LAT, 16, 4)
    M, N, t = len(ts) - 1, rows.shape[0], suffix.shape[0]
    assert M == N // 4
    for K in (2, 8, 32):
        r = orc.shared_latent_step(q, rows, D_LAT, ts, tm, rep, suffix, K, 5, 0, 0, scale)
        per_head = [orc.union_rows(ts, r.sel[h:h + 1]) for h in range(HEADS)]
        u = orc.union_rows(ts, r.sel)                                   # rows no head leaves out are read once
        teams = set(r.sel.ravel().tolist())
        assert u == sum(int(ts[g + 1] - ts[g]) for g in teams)
        assert max(per_head) <= u <= min(N, sum(per_head))
        pct = orc.mla_logical_access_pct([M], [u + t], [N + t])
        assert abs(pct - 100.0 * (M + u + t) / (N + t)) < 1e-12
    full = orc.mla_logical_access_pct([M], [N + t], [N + t])            # every team selected: routing comes on top
    assert abs(full - 100.0 * (1 + M / (N + t))) < 1e-12 and full > 100.0
