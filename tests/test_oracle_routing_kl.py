"""Pins for the oracle's routing-agreement diagnostic, Eq. (diagnostic-kl): KL(p || q) between
dense attention over the prompt (p) and the routing proposal spread over team members (q).

What fixes it without another implementation: with every key its own team the proposal IS dense
attention (routing key = the key, n_g = 1), so KL = 0; with a single team holding every key q is
uniform, so KL = log N - H(p); scaling invariances; and the defining sum re-evaluated with numpy
on the oracle's own team records.
"""
import math

import numpy as np

from oracle import santapp_oracle as orc


def _softmax(x):
    x = x - x.max()
    e = np.exp(x)
    return e / e.sum()


def _case(seed, N=96, d=16):
    rng = np.random.default_rng(seed)
    k = rng.normal(size=(N, d))
    q = rng.normal(size=d) * 1.5
    return q, k


def test_every_key_its_own_team_gives_zero():
    q, k = _case(0)
    N = k.shape[0]
    ts = np.arange(N + 1, dtype=np.int32)
    tm = np.arange(N, dtype=np.int32)
    assert abs(orc.routing_kl(q, k, ts, tm, k, 0.25)) < 1e-12
    # any order of the singleton teams gives the same proposal
    perm = np.random.default_rng(1).permutation(N).astype(np.int32)
    assert abs(orc.routing_kl(q, k, ts, perm, k[perm], 0.25)) < 1e-12


def test_one_team_holding_everything_is_log_n_minus_entropy():
    q, k = _case(2)
    N = k.shape[0]
    scale = 0.3
    p = _softmax(k @ q * scale)
    want = math.log(N) + float((p * np.log(p)).sum())
    ts = np.array([0, N], dtype=np.int32)
    tm = np.arange(N, dtype=np.int32)
    for rep in (k[5], np.zeros_like(k[0]), 100.0 * k[7]):              # the routing key cannot matter
        assert abs(orc.routing_kl(q, k, ts, tm, rep[None, :], scale) - want) < 1e-12


def test_matches_the_defining_sum_on_built_teams():
    q, k = _case(3, N=200, d=24)
    scale = 1.0 / math.sqrt(24)
    ts, tm, rep = orc.build_teams_contiguous(k, 40, 5)
    M = len(ts) - 1
    n = np.diff(ts).astype(np.float64)
    P = _softmax(np.log(n) + k[rep] @ q * scale)
    p = _softmax(k @ q * scale)
    qi = np.empty(k.shape[0])
    for g in range(M):
        qi[tm[ts[g]:ts[g + 1]]] = P[g] / n[g]
    assert abs(qi.sum() - 1.0) < 1e-12                                 # a distribution over the prompt tokens
    want = float((p * np.log(p / qi)).sum())
    got = orc.routing_kl(q, k, ts, tm, k[rep], scale)
    assert abs(got - want) < 1e-12
    assert got > 0.0                                                   # Gibbs: positive unless q = p


def test_invariances():
    q, k = _case(4, N=120, d=16)
    ts, tm, rep = orc.build_teams_contiguous(k, 30, 6)
    base = orc.routing_kl(q, k, ts, tm, k[rep], 0.2)
    # query scale and logit scale trade off exactly (powers of two keep the products exact)
    assert abs(orc.routing_kl(2.0 * q, k, ts, tm, k[rep], 0.1) - base) < 1e-12
    # the order of the members inside a team does not matter
    tm2 = tm.copy()
    for g in range(len(ts) - 1):
        tm2[ts[g]:ts[g + 1]] = tm2[ts[g]:ts[g + 1]][::-1]
    assert abs(orc.routing_kl(q, k, ts, tm2, k[rep], 0.2) - base) < 1e-12
    # shifting every key by a vector orthogonal to q changes neither p nor the proposal
    u = np.random.default_rng(9).normal(size=16)
    u -= q * (u @ q) / (q @ q)
    assert abs(orc.routing_kl(q, k + u, ts, tm, (k + u)[rep], 0.2) - base) < 1e-9
