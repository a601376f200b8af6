"""Shared-latent rows on the GPU against the oracle's composition of Algorithm 1 (appendix "Token
sparsity after latent compression"): records bit for bit, sampled teams as sets in order, log c,
tau, outputs within the tolerances of the main path, the union's row count, and the dense call."""
import numpy as np
import pytest
import torch

from oracle import santapp_oracle as orc
from paper_2609_35629_b200 import binding as sp
from paper_2609_35629_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu

SPARSE_TOL = 2e-3       # |out - oracle| <= tol * max |value|, as for the K/V path
DENSE_TOL = 1e-3
D = synth.LATENT_DIM


class LatentLayer:
    def __init__(self, spec, data=None):
        self.spec = spec
        self.data = data if data is not None else synth.make_latent_layer(spec)
        self.geom = sp.LatentGeometry(spec.n_seqs, spec.n_heads, spec.parent_size, spec.reps_per_parent)
        self.rows = sp.bf16_bits_to_cuda(self.data.rows)
        self.suffix = sp.bf16_bits_to_cuda(self.data.suffix)
        self.teams = sp.santapp_latent_build_teams(self.geom, spec.prompt_len, self.rows)
        torch.cuda.synchronize()
        t = self.teams
        self.csr = t.team_row_start.cpu().numpy()
        self.row_token = t.row_token.cpu().numpy()
        self.rep_bits = t.rep_rows.view(torch.int16).cpu().numpy().view(np.uint16)
        self.packed_bits = t.rows_packed.view(torch.int16).cpu().numpy().view(np.uint16)
        self.seq_team_off = t.seq_team_off.cpu().numpy()
        self.off = self.data.seq_row_off

    def records(self, b):
        t0, t1 = int(self.seq_team_off[b]), int(self.seq_team_off[b + 1])
        ts = self.csr[t0 + b: t1 + b + 1]
        tm = self.row_token[self.off[b]: self.off[b + 1]]
        rep = synth.to_f64(self.rep_bits[t0:t1])
        return ts, tm, rep


def check_records(layer):
    spec = layer.spec
    for b in range(spec.n_seqs):
        rows_b = layer.data.rows[layer.off[b]: layer.off[b + 1]]
        ts, tm, rep = orc.shared_latent_records(synth.to_f64(rows_b), D, spec.parent_size, spec.reps_per_parent)
        g_ts, g_tm, g_rep = layer.records(b)
        assert np.array_equal(g_ts, ts), f"team offsets differ (seq {b})"
        assert np.array_equal(g_tm, tm), f"member order differs (seq {b})"
        assert np.array_equal(g_rep, rep), f"representative rows differ (seq {b})"
        assert np.array_equal(layer.packed_bits[layer.off[b]: layer.off[b + 1]], rows_b[tm]), "packed rows are not the members' rows"
    amax = layer.teams.rep_abs_max.cpu().numpy()
    for b in range(spec.n_seqs):
        assert amax[b] == np.abs(layer.records(b)[2]).max()


def gpu_step(layer, q_bits, sl, K, seed, step, dense=False, stream_base=0):
    q = sp.bf16_bits_to_cuda(q_bits)
    sl_dev = torch.from_numpy(np.asarray(sl, dtype=np.int32)).cuda()
    if dense:
        out = sp.santapp_latent_dense_decode_attn(layer.geom, layer.teams, q, layer.suffix, sl_dev, synth.LATENT_SCALE)
        torch.cuda.synchronize()
        return out.cpu().numpy(), None
    dbg = sp.LatentDebugBuffers(layer.geom, K, "cuda")
    out = sp.santapp_latent_decode_attn(layer.geom, layer.teams, q, layer.suffix, sl_dev, K, seed, step, synth.LATENT_SCALE,
                                        stream_base=stream_base, debug=dbg)
    torch.cuda.synchronize()
    return out.cpu().numpy(), dbg


def check_step(layer, step, K=None, seed=1234, suffix_len=None, seqs=None, stream_base=0):
    spec = layer.spec
    K = spec.n_sample if K is None else K
    q_bits = synth.make_latent_queries(spec, layer.data, step)
    sl = spec.suffix_len(step) if suffix_len is None else np.asarray(suffix_len, dtype=np.int32)
    out, dbg = gpu_step(layer, q_bits, sl, K, seed, step, stream_base=stream_base)
    assert int(dbg.status.item()) == 0
    sel, logc, tau = dbg.sel_idx.cpu().numpy(), dbg.sel_logc.cpu().numpy(), dbg.tau.cpu().numpy()
    union = dbg.union_rows.cpu().numpy()
    worst = 0.0
    for b in (range(spec.n_seqs) if seqs is None else seqs):
        rows_b = synth.to_f64(layer.data.rows[layer.off[b]: layer.off[b + 1]])
        ts, tm, rep = layer.records(b)
        t = int(sl[b])
        suf = synth.to_f64(layer.data.suffix[b, :t]) if t else None
        r = orc.shared_latent_step(synth.to_f64(q_bits[b]), rows_b, D, ts, tm, rep, suf, K, seed, step, stream_base + b,
                                   synth.LATENT_SCALE, n_threads=4)
        M = len(ts) - 1
        Ke = min(K, M)
        if Ke < M:
            assert np.all(r.margin > 1e-9), "seeded workload too close to a selection boundary"
            assert np.allclose(tau[b], r.tau, rtol=0, atol=1e-9)
        else:
            assert np.all(np.isnan(tau[b]))
        for h in range(spec.n_heads):
            pu.assert_same_sample(sel[b, h, :Ke], logc[b, h, :Ke], r.sel[h, :Ke], r.logc[h, :Ke], f"(seq {b}, head {h}, step {step})")
        assert np.all(sel[b, :, Ke:] == -1)
        assert union[b, 0] == orc.union_rows(ts, r.sel[:, :Ke])
        vmax = np.abs(rows_b[:, :D]).max()
        err = np.abs(out[b] - r.o).max()
        worst = max(worst, err / vmax)
        assert err <= SPARSE_TOL * vmax, f"max |delta| {err} > {SPARSE_TOL} * {vmax} (seq {b})"
    return worst, union


def check_dense(layer, step, suffix_len=None, seqs=None):
    spec = layer.spec
    q_bits = synth.make_latent_queries(spec, layer.data, step)
    sl = spec.suffix_len(step) if suffix_len is None else np.asarray(suffix_len, dtype=np.int32)
    out, _ = gpu_step(layer, q_bits, sl, 0, 0, step, dense=True)
    for b in (range(spec.n_seqs) if seqs is None else seqs):
        rows_b = synth.to_f64(layer.data.rows[layer.off[b]: layer.off[b + 1]])
        t = int(sl[b])
        allrows = np.concatenate([rows_b, synth.to_f64(layer.data.suffix[b, :t])]) if t else rows_b
        vals = allrows.copy()
        vals[:, D:] = 0.0
        ref = orc.dense_step(synth.to_f64(q_bits[b]), allrows[None], vals[None], None, None, synth.LATENT_SCALE, n_threads=4)[:, :D]
        vmax = np.abs(rows_b[:, :D]).max()
        err = np.abs(out[b] - ref).max()
        assert err <= DENSE_TOL * vmax, f"dense max |delta| {err} > {DENSE_TOL} * {vmax} (seq {b})"


@pytest.fixture(scope="module")
def small():
    return LatentLayer(synth.LatentSpec("small", [1500, 777, 2048], n_sample=24, suffix_cap=12, suffix_len0=[0, 3, 12]))


def test_records_ragged_sequences_with_short_tails(small):
    check_records(small)


def test_records_other_parent_shapes():
    for P, R in ((32, 8), (8, 8), (16, 1), (5, 5)):
        check_records(LatentLayer(synth.LatentSpec(f"p{P}r{R}", [333, 64], parent_size=P, reps_per_parent=R, n_sample=4)))


def test_records_identical_rows_tie_rules():
    spec = synth.LatentSpec("ties", [200, 45], n_sample=4)
    data = synth.make_latent_layer(spec)
    data.rows[:] = data.rows[0]
    check_records(LatentLayer(spec, data))


def test_records_ignore_the_rotary_columns():
    spec = synth.LatentSpec("rope", [400], n_sample=4)
    a = synth.make_latent_layer(spec)
    b = synth.make_latent_layer(spec)
    b.rows[:, D:] = synth.round_bits(np.random.default_rng(5).standard_normal((400, 64), dtype=np.float32) * 50)
    la, lb = LatentLayer(spec, a), LatentLayer(spec, b)
    assert np.array_equal(la.csr, lb.csr) and np.array_equal(la.row_token, lb.row_token)


@pytest.mark.parametrize("step", [0, 3, 11])
def test_step_small_ragged_batch(small, step):
    check_step(small, step)


def test_step_dense_small(small):
    check_dense(small, 0)
    check_dense(small, 9)


def test_step_every_team_when_budget_reaches_team_count():
    layer = LatentLayer(synth.LatentSpec("allteams", [96, 700], n_sample=24, suffix_cap=4, suffix_len0=[2, 0]))
    worst, union = check_step(layer, 0)          # sequence 0 has 24 teams: all read, nothing drawn
    assert union[0, 0] == 96


def test_step_fewer_heads_and_odd_sizes():
    for H, lens in ((5, [1, 17, 1000]), (1, [513]), (9, [31, 33])):
        layer = LatentLayer(synth.LatentSpec(f"h{H}", lens, n_heads=H, n_sample=7, suffix_cap=3, suffix_len0=[1] * len(lens)))
        check_step(layer, 2)
        check_dense(layer, 2)


def test_step_many_short_sequences_blocks_span_several():
    """200 sequences of 5 to 300 rows: every block's range covers several sequences, most shares are
    shorter than a tile or than the copy ring, sequences with fewer teams than the budget sit beside
    sequences that sample."""
    rng = np.random.default_rng(3)
    lens = [int(x) for x in rng.integers(5, 300, size=200)]
    layer = LatentLayer(synth.LatentSpec("short", lens, n_sample=9, suffix_cap=6, suffix_len0=[int(x) for x in rng.integers(0, 7, size=200)],
                                         suffix_growth=0))
    check_step(layer, 0)
    check_dense(layer, 0)


def test_step_paper_point_8k_all_budgets():
    """8K context, P = 16, R = 4, 16 heads; the study's budgets S = 128, 256, 512, 1024 rows are
    K = 32, 64, 128, 256 teams."""
    layer = LatentLayer(synth.LatentSpec("8k", [8192, 8192], suffix_cap=16, suffix_len0=[0, 5]))
    check_records(layer)
    for K in (32, 64, 128, 256):
        worst, union = check_step(layer, 1, K=K)
        # shared-row accounting on the kernel's own counts (Eq. mla-logical-access)
        sl = layer.spec.suffix_len(1)
        M = [len(layer.records(b)[0]) - 1 for b in range(2)]
        pct = orc.mla_logical_access_pct(np.array(M), union[:, 0] + sl, np.array(layer.spec.prompt_len) + sl)
        assert 0.0 < pct < 125.0
    check_dense(layer, 1)


def test_step_full_bench_batch_sampled_sequences():
    """The bench's launch configuration (32 sequences of 8K, K = 128): three sequences against the oracle."""
    spec = synth.spec_latent_8k()
    layer = LatentLayer(spec)
    check_step(layer, 0, seqs=[0, 13, 31])
    check_dense(layer, 0, seqs=[0, 31])


def test_step_ragged_batch_with_several_tiles_per_scoring_warp():
    """72 sequences of 3000 to 5500 rows: more 128-team blocks of the scorer than fit on the GPU at
    once, so every scoring warp takes three tiles in a row, the last of them ragged or empty; four
    sequences (the shortest and the longest among them) against the oracle."""
    rng = np.random.default_rng(5)
    lens = [int(x) for x in rng.integers(3000, 5500, size=72)]
    lens[7], lens[40] = 3000, 5499
    layer = LatentLayer(synth.LatentSpec("ragged72", lens, n_sample=48, suffix_cap=4,
                                         suffix_len0=[int(x) for x in rng.integers(0, 5, size=72)], suffix_growth=0))
    check_step(layer, 0, seqs=[0, 7, 40, 71])


def test_two_hundred_steps_of_the_sampler():
    """Many draws on one layer (a different seed every step, K = 96 of 512 and 375 teams): now and
    then two candidates' scores agree in the upper half of their integer keys, which sends a head
    through the exact ranking pass; every sample must still be the oracle's."""
    layer = LatentLayer(synth.LatentSpec("soak", [2048, 1500], n_sample=96, suffix_cap=12, suffix_len0=[0, 3]))
    for step in range(200):
        check_step(layer, step, seed=step * 7 + 1)


def test_tcgen05_variant_of_the_attention_kernel(small, monkeypatch):
    """The tensor-memory variant (chosen by the environment) against the oracle: sparse with a ragged
    tail and a suffix, dense, and a sequence of the full batch shape; its bounded waits must not expire."""
    monkeypatch.setenv("SANTAPP_LATENT_ATTEND", "tcgen05")
    check_step(small, 3)
    check_dense(small, 9)
    layer = LatentLayer(synth.LatentSpec("8k", [8192, 5000], suffix_cap=16, suffix_len0=[0, 5]))
    check_step(layer, 1, K=128)
    check_dense(layer, 1)
    for H, lens in ((5, [1, 17, 1000]), (9, [31, 33])):
        odd = LatentLayer(synth.LatentSpec(f"h{H}", lens, n_heads=H, n_sample=7, suffix_cap=3, suffix_len0=[1] * len(lens)))
        check_step(odd, 2)
        check_dense(odd, 2)
    rng = np.random.default_rng(4)
    lens = [int(x) for x in rng.integers(5, 300, size=200)]
    short = LatentLayer(synth.LatentSpec("short", lens, n_sample=9, suffix_cap=6, suffix_len0=[3] * 200, suffix_growth=0))
    check_step(short, 0)
    check_dense(short, 0)


def test_same_seed_same_bits_and_step_changes_the_sample(small):
    q_bits = synth.make_latent_queries(small.spec, small.data, 0)
    sl = small.spec.suffix_len(0)
    a, da = gpu_step(small, q_bits, sl, 24, 7, 5)
    b, db = gpu_step(small, q_bits, sl, 24, 7, 5)
    c, dc = gpu_step(small, q_bits, sl, 24, 7, 6)
    assert np.array_equal(a, b) and torch.equal(da.sel_idx, db.sel_idx)
    assert not torch.equal(da.sel_idx, dc.sel_idx)


def test_bad_arguments_are_refused_on_the_host(small):
    q = sp.bf16_bits_to_cuda(synth.make_latent_queries(small.spec, small.data, 0))
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_latent_decode_attn(small.geom, small.teams, q, None, None, 257, 0, 0, synth.LATENT_SCALE, workspace=ws)
    assert e.value.status == sp.SANTAPP_ERR_UNSUPPORTED
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_latent_decode_attn(small.geom, small.teams, q, None, None, 8, 0, 0, 0.0)
    assert e.value.status == sp.SANTAPP_ERR_INVALID_ARG
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_latent_decode_attn(small.geom, small.teams, q, None, None, 8, 0, 0, synth.LATENT_SCALE, workspace=ws[:4096])
    assert e.value.status == sp.SANTAPP_ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_latent_sizes(sp.LatentGeometry(1, 17), [10])
    assert e.value.status == sp.SANTAPP_ERR_UNSUPPORTED
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_latent_sizes(sp.LatentGeometry(1, 16, 64, 4), [10])
    assert e.value.status == sp.SANTAPP_ERR_UNSUPPORTED
