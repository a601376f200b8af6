"""Pins for the oracle's accounting helpers against figures printed in the paper
(tests/golden/paper_accounting.txt carries the values and their citations)."""
import os

import numpy as np

from oracle import santapp_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_accounting.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, value, _ = [x.strip() for x in line.split("|", 2)]
            out[name] = float(value)
    return out


def test_dense_kv_stream_per_token():
    g = _golden()
    mib = orc.dense_kv_bytes(32768, 4, 128, 2) / 2 ** 20
    assert mib == g["dense_kv_mib_per_layer_token_32k_bf16"]
    assert mib == g["packed_kv_mib_32k_fp16"]


def test_budget_rule():
    g = _golden()
    assert orc.team_budget(10 ** 6, 128, 16, 4) == g["teams_for_S128_P16_R4"]
    assert orc.team_budget(10 ** 6, int(g["S_for_K31_P16_R4"]), 16, 4) == 31
    assert orc.team_budget(20, 128, 16, 4) == 20          # K = min{M, S/(P/R)}
    assert orc.team_budget(100, 128, 16, 5) == -1         # R must divide P
    assert orc.team_budget(100, 126, 16, 4) == -1         # P/R must divide S


def test_logical_access_counter():
    g = _golden()
    N = 32768
    # SANTA: numerator per call is N (+ sampled value rows); the scan alone is 50 %.
    # In the counter's terms that is m = N representatives and nothing else.
    assert orc.logical_access_pct([N], [0], [0], [N]) == g["santa_full_key_scan_access_pct"]
    # Contiguous P=16, R=4 at 32K: routing scans N/4 representatives (12.5 %); the
    # printed totals of 15.0-15.7 % then correspond to a union of ~0.8-1.05 K rows
    # per KV head, i.e. about 7 heads x 32 teams x 4 rows.
    lo = orc.logical_access_pct([N // 4], [820], [0], [N])
    hi = orc.logical_access_pct([N // 4], [1049], [0], [N])
    assert abs(lo - g["contiguous_S128_access_pct_low"]) < 0.01
    assert abs(hi - g["contiguous_S128_access_pct_high"]) < 0.01
    # counts add across calls before division (sum of numerators over sum of denominators)
    a = orc.logical_access_pct([10, 30], [1, 2], [3, 4], [100, 300])
    assert a == 100.0 * ((10 + 2 * 4) + (30 + 2 * 6)) / (2 * 400)


def test_union_rows_counts_each_team_once():
    ts = np.array([0, 3, 4, 9, 10], dtype=np.int32)
    sel = np.array([[0, 2], [2, 3], [0, 3]], dtype=np.int32)
    assert orc.union_rows(ts, sel) == 3 + 5 + 1
    assert orc.union_rows(ts, sel[:1]) == 8


def test_shared_row_counter_of_a_shared_latent_cache():
    """Eq. (mla-logical-access): routing rows and the union over heads are both charged against the
    dense shared-row count, pooled over calls. The paper prints the two terms and their total for
    S = 512 and the attention term and the total for S = 1024; the counter must be additive in
    exactly that way."""
    g = _golden()
    d = 100000                                                       # any dense row count: percentages scale
    r = round(g["mla_S512_routing_pct"] * d / 100)
    u = round(g["mla_S512_attention_pct"] * d / 100)
    assert abs(orc.mla_logical_access_pct([r], [u], [d]) - g["mla_S512_total_pct"]) < 0.005
    assert abs(orc.mla_logical_access_pct([r], [0], [d]) - g["mla_S512_routing_pct"]) < 0.005
    # S = 1024: the printed total minus the printed attention term leaves a routing term within 0.1 of
    # S = 512's (the routing scan does not depend on the budget, only the trajectory's length does)
    routing_1024 = g["mla_S1024_total_pct"] - g["mla_S1024_attention_pct"]
    assert abs(routing_1024 - g["mla_S512_routing_pct"]) < 0.1
    u2 = round(g["mla_S1024_attention_pct"] * d / 100)
    r2 = round(routing_1024 * d / 100)
    assert abs(orc.mla_logical_access_pct([r2], [u2], [d]) - g["mla_S1024_total_pct"]) < 0.005
    # above 100 % is possible: a row read in both passes is charged twice
    assert orc.mla_logical_access_pct([50], [100], [100]) == 150.0
    # pooled before the division, not a mean of ratios
    assert orc.mla_logical_access_pct([10, 0], [10, 0], [100, 300]) == 5.0
    # one counted row per token: no factor 2 for keys and values, unlike the GQA counter
    assert orc.mla_logical_access_pct([0], [7], [14]) == 50.0
    assert orc.logical_access_pct([0], [7], [0], [14]) == 50.0
