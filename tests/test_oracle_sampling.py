"""Pins for the oracle's Algorithm 1: routing weight, Gumbel-top-K sampling,
conditional inclusion correction and the inverse-inclusion estimator.

Nothing here re-types the oracle's formulas as the expected value: the
expectations come from the laws the paper states (first-draw probabilities
proportional to the routing weights, the successive-sampling law, unbiasedness
of the two unnormalised sums, K = M equals dense attention) evaluated by exact
enumeration, quadrature or library softmax.
"""
import itertools
import math

import numpy as np
import pytest
from scipy.special import softmax

from oracle import santapp_oracle as orc


def _toy(M, sizes, d=4, t=2, seed=0, spread=1.0):
    """A tiny cache: M teams with the given sizes; returns everything Algorithm 1 needs."""
    rng = np.random.default_rng(seed)
    N = int(sum(sizes))
    k = rng.standard_normal((N, d)) * spread
    v = rng.standard_normal((N, d))
    perm = rng.permutation(N).astype(np.int32)              # teams are not contiguous in token order
    team_start = np.zeros(M + 1, dtype=np.int32)
    team_start[1:] = np.cumsum(sizes)
    team_member = perm
    rep_rows = np.array([team_member[team_start[g]] for g in range(M)])
    rep_key = k[rep_rows].copy()
    ks = rng.standard_normal((t, d)) * spread if t else None
    vs = rng.standard_normal((t, d)) if t else None
    q = rng.standard_normal(d) * spread
    return dict(q=q, k=k, v=v, team_start=team_start, team_member=team_member, rep_key=rep_key,
                ks=ks, vs=vs, N=N, d=d)


def _run(c, K, gumbel, shift=None, want_routing=False):
    return orc.decode_head_given_gumbel(c["q"], c["k"], c["v"], c["team_start"], c["team_member"],
                                        c["rep_key"], c["ks"], c["vs"], K, gumbel,
                                        1.0 / math.sqrt(c["d"]), shift=shift, want_routing=want_routing)


def _routing_weights(c):
    """Z~_g = n_g exp(q.l_g / sqrt d), straight from the sentence that defines it."""
    n = np.diff(c["team_start"]).astype(np.float64)
    return n * np.exp(c["rep_key"] @ c["q"] / math.sqrt(c["d"]))


def _dense_sums(c):
    kk = c["k"] if c["ks"] is None else np.vstack([c["k"], c["ks"]])
    vv = c["v"] if c["vs"] is None else np.vstack([c["v"], c["vs"]])
    a = np.exp(kk @ c["q"] / math.sqrt(c["d"]))
    return a.sum(), a @ vv


def test_routing_logit_is_log_size_plus_scaled_rep_score():
    c = _toy(5, [1, 2, 3, 4, 5])
    r = _run(c, 2, np.zeros(5), want_routing=True)
    assert np.allclose(np.exp(r.phi), _routing_weights(c), rtol=1e-13)
    assert np.allclose(r.y, r.phi)                       # zero noise: Y = phi


def test_zero_noise_selects_largest_routing_weights_and_tau_is_next():
    c = _toy(6, [3, 1, 4, 1, 5, 9], seed=3)
    w = _routing_weights(c)
    order = np.argsort(-w)
    for K in (1, 2, 3, 5):
        r = _run(c, K, np.zeros(6))
        assert list(r.sel) == list(order[:K])
        assert r.tau == pytest.approx(math.log(w[order[K]]), rel=1e-13)
        assert r.margin == pytest.approx(math.log(w[order[K - 1]] / w[order[K]]), abs=1e-12)


def test_noise_is_added_not_subtracted():
    c = _toy(4, [2, 2, 2, 2], seed=5)
    g = np.array([0.0, 0.0, 50.0, 0.0])
    assert list(_run(c, 1, g).sel) == [2]


def test_ties_go_to_smaller_team_id():
    c = _toy(4, [2, 2, 2, 2], seed=5)
    c["rep_key"][:] = c["rep_key"][0]                    # identical routing logits
    r = _run(c, 2, np.zeros(4))
    assert list(r.sel) == [0, 1]


def test_first_draw_law_chi_square():
    """K = 1: Pr(argmax Y = g) = Z~_g / sum Z~ over 1e5 keyed draws."""
    c = _toy(8, [1, 2, 3, 4, 5, 6, 7, 8], seed=11, spread=1.5)
    p = _routing_weights(c)
    p /= p.sum()
    n = 100_000
    counts = np.zeros(8)
    for step in range(n):
        g = orc.gumbel_many(99, step, 0, 0, 8)
        counts[_run(c, 1, g).sel[0]] += 1
    chi2 = np.sum((counts - n * p) ** 2 / (n * p))
    assert chi2 < 29.9                                   # chi^2_7 at 1e-4


def test_every_key_its_own_team_first_draw_is_exact_softmax():
    """SANTA limit: singleton teams make the routing logit the exact logit, so the
    first-draw law is the attention distribution itself."""
    rng = np.random.default_rng(2)
    M, d = 10, 8
    k = rng.standard_normal((M, d)) * 2
    v = rng.standard_normal((M, d))
    q = rng.standard_normal(d)
    ts, tm, rep = orc.build_teams_contiguous(k, P=5, R=5)         # R = P: every key becomes a team
    assert np.all(np.diff(ts) == 1)
    rep_key = k[rep]
    scale = 1.0 / math.sqrt(d)
    r = orc.decode_head_given_gumbel(q, k, v, ts, tm, rep_key, None, None, 1, np.zeros(M), scale,
                                     want_routing=True)
    p = softmax(k[tm] @ q * scale)                       # library softmax over the teams' keys
    assert np.allclose(softmax(r.phi), p, rtol=1e-12)
    n = 60_000
    counts = np.zeros(M)
    for step in range(n):
        g = orc.gumbel_many(5, step, 1, 2, M)
        counts[orc.decode_head_given_gumbel(q, k, v, ts, tm, rep_key, None, None, 1, g, scale).sel[0]] += 1
    keep = n * p > 5
    chi2 = np.sum((counts[keep] - n * p[keep]) ** 2 / (n * p[keep]))
    assert chi2 < 35.0


def _exact_inclusion(w, K):
    """Marginal inclusion probabilities under the successive-sampling law: each
    draw picks among the remaining teams in proportion to Z~_g."""
    M = len(w)
    pi = np.zeros(M)
    for prefix in itertools.permutations(range(M), K):
        rest = w.sum()
        pr = 1.0
        for g in prefix:
            pr *= w[g] / rest
            rest -= w[g]
        for g in prefix:
            pi[g] += pr
    return pi


@pytest.mark.parametrize("M,K,sizes", [(5, 2, [1, 2, 3, 4, 5]), (6, 3, [2, 1, 7, 1, 3, 2])])
def test_inclusion_probabilities_enumeration_vs_frequency_vs_rao_blackwell(M, K, sizes):
    """Three-way agreement: exact pi_g by enumeration; empirical inclusion
    frequency over 1e5 draws; mean of the conditional probability rho_g(T_-g)
    with T_-g found by brute force. Also E[1{g in S} / c_g] = 1 with the
    oracle's own c_g, and for a selected team T_-g equals tau exactly."""
    c = _toy(M, sizes, seed=21 + M, spread=1.2)
    w = _routing_weights(c)
    pi = _exact_inclusion(w, K)
    assert pi.sum() == pytest.approx(K, rel=1e-12)
    n = 100_000
    freq = np.zeros(M)
    rb = np.zeros(M)
    inv = np.zeros(M)
    inv2 = np.zeros(M)
    for step in range(n):
        g = orc.gumbel_many(2024, step, 4, 1, M)
        r = _run(c, K, g, want_routing=True)
        freq[r.sel] += 1
        for a, team in enumerate(r.sel):
            x = math.exp(-r.logc[a])
            inv[team] += x
            inv2[team] += x * x
        # leave-one-out thresholds by brute force
        for team in range(M):
            others = np.delete(r.y, team)
            T = np.sort(others)[::-1][K - 1]
            rb[team] += -math.expm1(-math.exp(r.phi[team] - T))
            if team in r.sel:
                assert T == r.tau
    freq /= n
    rb /= n
    se = np.sqrt(pi * (1 - pi) / n)
    assert np.all(np.abs(freq - pi) < 4.5 * se)
    assert np.all(np.abs(rb - pi) < 4.5 * se)            # Rao-Blackwell has smaller variance still
    mean_inv = inv / n
    se_inv = np.sqrt(np.maximum(inv2 / n - mean_inv ** 2, 1e-12) / n)
    assert np.all(np.abs(mean_inv - 1.0) < 4.5 * se_inv)


def test_unbiased_sums_monte_carlo_and_biased_ratio():
    """E[Z^] = Z and E[U^] = U (suffix included with weight one, no 1/K factor),
    while the ratio is visibly biased at K = 1."""
    c = _toy(6, [1, 3, 2, 6, 1, 4], d=4, t=3, seed=8, spread=1.6)
    Z, U = _dense_sums(c)
    o_dense = U / Z
    for K in (1, 3):
        n = 100_000
        zs = np.zeros(n)
        us = np.zeros((n, 4))
        os_ = np.zeros((n, 4))
        for step in range(n):
            g = orc.gumbel_many(77, step, 2, 0, 6)
            r = _run(c, K, g, shift=0.0)
            zs[step], us[step], os_[step] = r.Z, r.U, r.o
        assert abs(zs.mean() - Z) < 4.5 * zs.std() / math.sqrt(n)
        assert np.all(np.abs(us.mean(0) - U) < 4.5 * us.std(0) / math.sqrt(n))
        assert 4.5 * zs.std() / math.sqrt(n) / Z < (0.15 if K == 1 else 0.03)   # the test has power
        if K == 1:
            bias = np.abs(os_.mean(0) - o_dense) / (os_.std(0) / math.sqrt(n))
            assert bias.max() > 6.0                      # the normalised ratio is biased


@pytest.mark.parametrize("M,K,n_grid", [(2, 1, 128), (3, 1, 24), (3, 2, 20)])
def test_unbiased_sums_by_midpoint_quadrature(M, K, n_grid):
    """Deterministic check: integrate Z^ and U^ over the uniforms u in (0,1)^M on
    midpoint grids (G = -log(-log u)) of n and 2n points per axis. The integrand
    jumps where the selected set changes, so the rule converges like 1/n; one
    Richardson step (2 I_2n - I_n) removes that term. The integrals must equal
    the dense sums Z and U."""
    c = _toy(M, [2, 1, 3][:M], d=3, t=1, seed=30 + M, spread=1.0)
    Z, U = _dense_sums(c)

    def integrate(n):
        u = (np.arange(n) + 0.5) / n
        gum = -np.log(-np.log(u))
        zacc, uacc = 0.0, np.zeros(3)
        for idx in itertools.product(range(n), repeat=M):
            r = _run(c, K, gum[list(idx)], shift=0.0)
            zacc += r.Z
            uacc += r.U
        return zacc / n ** M, uacc / n ** M

    z1, u1 = integrate(n_grid)
    z2, u2 = integrate(2 * n_grid)
    assert 2 * z2 - z1 == pytest.approx(Z, rel=1e-2)
    assert np.allclose(2 * u2 - u1, U, rtol=0, atol=1e-2 * np.abs(U).max())
    assert abs(z2 - Z) < abs(z1 - Z)                     # and the plain rule converges


def test_k_at_least_m_is_dense_attention_without_draws():
    c = _toy(7, [2, 5, 1, 1, 3, 8, 4], d=6, t=4, seed=13, spread=2.0)
    kk = np.vstack([c["k"], c["ks"]])
    vv = np.vstack([c["v"], c["vs"]])
    expect = softmax(kk @ c["q"] / math.sqrt(6)) @ vv    # library softmax, textbook attention
    for K in (7, 8, 100):
        r = _run(c, K, np.full(7, np.nan))               # draws must not be consumed
        assert list(r.sel) == list(range(7))
        assert np.all(r.logc == 0.0)
        assert np.allclose(r.o, expect, rtol=1e-12, atol=1e-14)
    assert np.allclose(orc.dense_head_two(c["q"], c["k"], c["v"], c["ks"], c["vs"], 1 / math.sqrt(6)),
                       expect, rtol=1e-12, atol=1e-14)
    assert np.allclose(orc.dense_head(c["q"], kk, vv, 1 / math.sqrt(6)), expect, rtol=1e-12, atol=1e-14)


def test_dominant_team_gives_near_dense_output():
    """K < M but one team carries almost all the mass: its correction tends to
    one and the estimate tends to dense attention."""
    c = _toy(5, [3, 2, 2, 2, 2], d=4, t=0, seed=17, spread=0.3)
    first = c["team_member"][0:3]
    c["k"][first] = c["q"] * 600.0                       # huge logits for team 0
    c["rep_key"][0] = c["k"][first[0]]
    Z, U = _dense_sums(c)
    r = _run(c, 1, orc.gumbel_many(1, 0, 0, 0, 5))
    assert list(r.sel) == [0]
    assert r.logc[0] == pytest.approx(0.0, abs=1e-8)
    assert np.allclose(r.o, U / Z, atol=1e-7)


def test_estimator_matches_definition_given_selection():
    """Given the oracle's own S and c_g, recompute U^/Z^ from the defining sums
    with numpy (team sums divided by c_g, suffix with weight one)."""
    c = _toy(9, [4, 1, 2, 7, 3, 1, 1, 5, 2], d=5, t=3, seed=40, spread=1.5)
    g = orc.gumbel_many(3, 14, 15, 9, 9)
    r = _run(c, 4, g)
    scale = 1 / math.sqrt(5)
    Zh = np.exp(c["ks"] @ c["q"] * scale).sum()
    Uh = np.exp(c["ks"] @ c["q"] * scale) @ c["vs"]
    for a, team in enumerate(r.sel):
        rows = c["team_member"][c["team_start"][team]:c["team_start"][team + 1]]
        e = np.exp(c["k"][rows] @ c["q"] * scale)
        Zh += e.sum() / math.exp(r.logc[a])
        Uh += (e @ c["v"][rows]) / math.exp(r.logc[a])
    assert np.allclose(r.o, Uh / Zh, rtol=1e-12)


def test_decode_head_uses_the_keyed_stream():
    c = _toy(12, [2] * 12, d=4, t=1, seed=50)
    scale = 0.5
    a = orc.decode_head(c["q"], c["k"], c["v"], c["team_start"], c["team_member"], c["rep_key"],
                        c["ks"], c["vs"], 3, 42, 7, 5, 2, scale)
    g = orc.gumbel_many(42, 7, 5, 2, 12)
    b = _run(c, 3, g)
    assert list(a.sel) == list(b.sel) and np.array_equal(a.o, b.o) and a.tau == b.tau


def test_gqa_heads_are_independent_and_share_team_records():
    """A head's result is the same computed alone or beside its siblings; heads
    of one KV head draw different teams from the same records."""
    rng = np.random.default_rng(60)
    n_q, n_kv, d, N, t = 6, 2, 8, 48, 3
    k = rng.standard_normal((n_kv, N, d))
    v = rng.standard_normal((n_kv, N, d))
    ks = rng.standard_normal((n_kv, t, d))
    vs = rng.standard_normal((n_kv, t, d))
    q = rng.standard_normal((n_q, d))
    recs = [orc.build_teams_contiguous(k[j], P=16, R=4) for j in range(n_kv)]
    M = np.array([len(r[0]) - 1 for r in recs], dtype=np.int32)
    M_max = int(M.max())
    ts = np.zeros((n_kv, M_max + 1), dtype=np.int32)
    tm = np.zeros((n_kv, N), dtype=np.int32)
    rk = np.zeros((n_kv, M_max, d))
    for j, (s, m, rep) in enumerate(recs):
        ts[j, :len(s)] = s
        tm[j] = m
        rk[j, :len(rep)] = k[j][rep]
    scale = 1 / math.sqrt(d)
    step = orc.decode_step(q, k, v, M, ts, tm, rk, ks, vs, 3, 9, 4, 11, scale, n_threads=2)
    sels = set()
    for h in range(n_q):
        j = h // 3
        one = orc.decode_head(q[h], k[j], v[j], recs[j][0], recs[j][1], k[j][recs[j][2]], ks[j], vs[j],
                              3, 9, 4, h, 11, scale)
        assert np.array_equal(one.o, step.o[h])
        assert list(one.sel) == list(step.sel[h])
        sels.add(tuple(one.sel))
    assert len(sels) > 1
    dense = orc.dense_step(q, k, v, ks, vs, scale, n_threads=2)
    for h in range(n_q):
        kk = np.vstack([k[h // 3], ks[h // 3]])
        vv = np.vstack([v[h // 3], vs[h // 3]])
        assert np.allclose(dense[h], softmax(kk @ q[h] * scale) @ vv, rtol=1e-12)
