"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle
on the same seeded inputs.

Bars (from the benchmark spec): sampled team indices bit-exact for the same
seed; sparse outputs within 2e-3 * max|V|; dense outputs within 1e-3 * max|V|;
team records identical (the builder evaluates distances in fp64 in the oracle's
order, so even near-ties must fall the same way).
"""
import math

import numpy as np
import pytest
import torch

from oracle import santapp_oracle as orc
from paper_2609_35629_b200 import binding as sp
from paper_2609_35629_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu

SPARSE_TOL = 2e-3
DENSE_TOL = 1e-3

_cache = {}


def layer_for(name, spec_fn, **kw):
    key = (name, tuple(sorted(kw.items())))
    if key not in _cache:
        spec = spec_fn(**kw)
        data = synth.make_layer(spec, layer=0, keep_centres=(spec.query_kind == "concentrated"))
        _cache[key] = pu.GpuLayer(spec, data)
    return _cache[key]


def check_team_records(layer, seqs=None, kv_heads=None):
    spec = layer.spec
    for b in (range(spec.n_seqs) if seqs is None else seqs):
        r0, r1 = int(layer.seq_row_off[b]), int(layer.seq_row_off[b + 1])
        for j in (range(spec.n_kv_heads) if kv_heads is None else kv_heads):
            keys = synth.to_f64(layer.data.k_prompt[j, r0:r1], spec.elem)
            ts_o, tm_o, rep_o = orc.build_teams_contiguous(keys, spec.parent_size, spec.reps_per_parent)
            ts_g, tm_g, rep_g = layer.records(b, j)
            assert np.array_equal(ts_g, ts_o)
            assert np.array_equal(tm_g, tm_o)
            assert np.array_equal(rep_g, keys[rep_o])                 # frozen representative keys
            # packed rows are the member rows, K and V alike
            assert np.array_equal(layer.k_packed_bits[j, r0:r1], layer.data.k_prompt[j, r0:r1][tm_g])
            assert np.array_equal(layer.v_packed_bits[j, r0:r1], layer.data.v_prompt[j, r0:r1][tm_g])


def check_sparse_step(layer, step, K, seed=1234, stream_base=0, suffix_len=None, seqs=None):
    spec = layer.spec
    q_bits = synth.make_queries(spec, layer.data, step)
    sl = spec.suffix_len(step) if suffix_len is None else np.asarray(suffix_len, dtype=np.int32)
    out, dbg = pu.gpu_step(layer, q_bits, sl, K, seed, step, stream_base)
    ref = pu.oracle_step(layer, q_bits, sl, K, seed, step, stream_base, seqs=seqs)
    assert int(dbg.status.item()) == 0
    sel = dbg.sel_idx.cpu().numpy()
    logc = dbg.sel_logc.cpu().numpy()
    tau = dbg.tau.cpu().numpy()
    union = dbg.union_rows.cpu().numpy()
    vmax = pu.max_abs_v(layer)
    worst = 0.0
    G = spec.group
    for b, r in ref.items():
        for j in range(spec.n_kv_heads):
            ts, _, _ = layer.records(b, j)
            M = len(ts) - 1                                           # teams of this (sequence, KV head)
            Ke = min(K, M)
            hs = slice(j * G, (j + 1) * G)
            if Ke < M:
                assert np.all(r.margin[hs] > 1e-9), "seeded workload too close to a selection boundary"
            for h in range(j * G, (j + 1) * G):
                pu.assert_same_sample(sel[b, h, :Ke], logc[b, h, :Ke], r.sel[h, :Ke], r.logc[h, :Ke], f"(seq {b}, head {h}, step {step})")
            assert np.all(sel[b, hs, Ke:] == -1)
            if Ke < M:
                assert np.allclose(tau[b, hs], r.tau[hs], rtol=0, atol=1e-9)
            else:
                assert np.all(np.isnan(tau[b, hs]))
            assert union[b, j] == orc.union_rows(ts, r.sel[hs, :Ke])
        err = np.abs(out[b] - r.o).max()
        worst = max(worst, err)
        assert err <= SPARSE_TOL * vmax, f"max |delta| {err} > {SPARSE_TOL} * {vmax}"
    return worst


def check_dense_step(layer, step, suffix_len=None, seqs=None):
    spec = layer.spec
    q_bits = synth.make_queries(spec, layer.data, step)
    sl = spec.suffix_len(step) if suffix_len is None else np.asarray(suffix_len, dtype=np.int32)
    out, _ = pu.gpu_step(layer, q_bits, sl, 0, 0, step, dense=True)
    ref = pu.oracle_step(layer, q_bits, sl, 0, 0, step, dense=True, seqs=seqs)
    vmax = pu.max_abs_v(layer)
    for b, o in ref.items():
        err = np.abs(out[b] - o).max()
        assert err <= DENSE_TOL * vmax, f"dense max |delta| {err} > {DENSE_TOL} * {vmax}"


# ---------------------------------------------------------------------------------------------

def test_team_records_small_gqa_ragged_with_short_tail():
    layer = layer_for("small", synth.spec_small_gqa)
    check_team_records(layer)


def test_team_records_tiny_config():
    layer = layer_for("tiny", synth.spec_tiny)
    check_team_records(layer)


def test_team_records_duplicate_keys_and_singletons():
    """Exact ties everywhere (all keys equal) and R = P (every key its own team)."""
    spec = synth.spec_small_gqa(prompt=(300, 77), parent_size=64, reps=64)
    data = synth.make_layer(spec)
    layer = pu.GpuLayer(spec, data)
    check_team_records(layer)
    assert np.all(np.diff(layer.records(0, 0)[0]) == 1)
    spec2 = synth.spec_small_gqa(prompt=(200, 130), parent_size=64, reps=8)
    data2 = synth.make_layer(spec2)
    data2.k_prompt[:] = data2.k_prompt[0, 0]                        # every key identical
    layer2 = pu.GpuLayer(spec2, data2)
    check_team_records(layer2)


def test_decode_small_gqa_steps():
    layer = layer_for("small", synth.spec_small_gqa)
    for step in range(3):
        check_sparse_step(layer, step, K=8)


@pytest.mark.parametrize("K", [1, 2, 31, 33])
def test_decode_small_gqa_budgets(K):
    layer = layer_for("small", synth.spec_small_gqa)
    check_sparse_step(layer, 1, K=K)


def test_decode_k_at_least_m_equals_dense():
    layer = layer_for("small", synth.spec_small_gqa)
    spec = layer.spec
    M_max = int(layer.teams.sizes.max_teams_per_seq)
    step = 2
    q_bits = synth.make_queries(spec, layer.data, step)
    sl = spec.suffix_len(step)
    check_sparse_step(layer, step, K=M_max)                          # all sequences: shortcut
    out_s, _ = pu.gpu_step(layer, q_bits, sl, M_max, 5, step)
    out_d, _ = pu.gpu_step(layer, q_bits, sl, 0, 0, step, dense=True)
    assert np.abs(out_s - out_d).max() <= 1e-5 * pu.max_abs_v(layer)
    # mixed: K between the two sequences' team counts -> one sampled, one dense
    Ms = np.diff(layer.seq_team_off)
    if Ms.min() < Ms.max():
        check_sparse_step(layer, step, K=int(Ms.min()))


def test_stream_base_and_64_bit_seed():
    """The sequence stream is stream_base + sequence index, and both halves of the seed key the draw."""
    layer = layer_for("small", synth.spec_small_gqa)
    check_sparse_step(layer, 1, K=8, seed=(0xDEADBEEF << 32) | 0x12345678, stream_base=7)
    spec = layer.spec
    q_bits = synth.make_queries(spec, layer.data, 1)
    sl = spec.suffix_len(1)
    _, d0 = pu.gpu_step(layer, q_bits, sl, 8, 5, 1, stream_base=0)
    _, d1 = pu.gpu_step(layer, q_bits, sl, 8, 5, 1, stream_base=1)
    _, d2 = pu.gpu_step(layer, q_bits, sl, 8, 5 | (1 << 40), 1, stream_base=0)
    s0, s1, s2 = (d.sel_idx.cpu().numpy() for d in (d0, d1, d2))
    assert not np.array_equal(s0, s1) and not np.array_equal(s0, s2)


def test_scale_override():
    """An explicit logit scale replaces 1 / sqrt(d) in routing and in attention alike."""
    layer = layer_for("small", synth.spec_small_gqa)
    spec = layer.spec
    q_bits = synth.make_queries(spec, layer.data, 0)
    sl = spec.suffix_len(0)
    scale = 0.05
    q = sp.bf16_bits_to_cuda(q_bits)
    dbg = sp.DebugBuffers(layer.geom, 8, "cuda")
    out = sp.santapp_decode_attn(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix,
                                 torch.from_numpy(sl).cuda(), 8, 3, 0, scale=scale, debug=dbg).cpu().numpy()
    dense = sp.santapp_dense_decode_attn(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix,
                                         torch.from_numpy(sl).cuda(), scale=scale).cpu().numpy()
    vmax = pu.max_abs_v(layer)
    for b in range(spec.n_seqs):
        oi = layer.oracle_inputs(b)
        t = int(sl[b])
        ks = synth.bf16_to_f64(layer.data.k_suffix[b, :, :t]) if t else None
        vs = synth.bf16_to_f64(layer.data.v_suffix[b, :, :t]) if t else None
        qf = synth.bf16_to_f64(q_bits[b])
        # float32(0.05) is what the library receives
        r = orc.decode_step(qf, oi["k"], oi["v"], oi["M"], oi["ts"], oi["tm"], oi["rk"], ks, vs, 8, 3, 0, b,
                            float(np.float32(scale)))
        assert np.array_equal(dbg.sel_idx.cpu().numpy()[b], r.sel)
        assert np.abs(out[b] - r.o).max() <= SPARSE_TOL * vmax
        o_d = orc.dense_step(qf, oi["k"], oi["v"], ks, vs, float(np.float32(scale)))
        assert np.abs(dense[b] - o_d).max() <= DENSE_TOL * vmax


@pytest.mark.parametrize("P,R", [(512, 64), (32, 2), (64, 64), (100, 10)])
def test_team_records_other_parent_shapes(P, R):
    spec = synth.spec_small_gqa(prompt=(1300, 700), parent_size=P, reps=R)
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    check_team_records(layer, kv_heads=[0, 3])
    check_sparse_step(layer, 0, K=4)


def test_decode_one_team_left_out():
    """K = M - 1, the smallest sampled case: tau is the single excluded team's score."""
    layer = layer_for("small", synth.spec_small_gqa)
    Ms = np.diff(layer.seq_team_off)
    check_sparse_step(layer, 0, K=int(Ms.min()) - 1)
    check_sparse_step(layer, 1, K=int(Ms.max()) - 1)                 # the shorter sequence takes every team


def test_decode_large_logits():
    """Queries scaled up sixteen-fold: logits in the hundreds, softmax weights and corrections at
    the ends of their ranges; the log-sum-exp bookkeeping must hold."""
    layer = layer_for("small", synth.spec_small_gqa)
    spec = layer.spec
    q_bits = synth.make_queries(spec, layer.data, 2)
    big = synth.f32_to_bf16_bits(16.0 * synth.bf16_to_f32(q_bits))
    _check_with_queries(layer, big, K=8, step=2)


def test_decode_suffix_edge_cases():
    layer = layer_for("small", synth.spec_small_gqa)
    check_sparse_step(layer, 0, K=8, suffix_len=[0, 0])
    check_sparse_step(layer, 0, K=8, suffix_len=[layer.spec.suffix_cap, 1])
    check_dense_step(layer, 0, suffix_len=[0, 0])
    check_dense_step(layer, 0, suffix_len=[layer.spec.suffix_cap, 1])


def test_decode_every_key_its_own_team():
    spec = synth.spec_small_gqa(prompt=(256, 128), parent_size=32, reps=32, n_sample=16)
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    check_sparse_step(layer, 0, K=16)


def test_decode_single_team_sequence():
    """M = 1 for a sequence: K >= M, so the single team is always read."""
    spec = synth.spec_small_gqa(prompt=(64, 700), parent_size=64, reps=1, n_sample=4)
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    check_sparse_step(layer, 0, K=4)
    check_dense_step(layer, 0)


def test_dense_small_gqa():
    layer = layer_for("small", synth.spec_small_gqa)
    for step in range(2):
        check_dense_step(layer, step)


def test_tiny_config_all_queries():
    """Config 1: 1 head, 4096 keys + 16 suffix rows, 256 teams, 16 sampled, 32 queries."""
    layer = layer_for("tiny", synth.spec_tiny)
    for step in range(32):
        check_sparse_step(layer, step, K=16, seed=0)
    check_dense_step(layer, 0)


def test_same_seed_same_bits_and_seed_changes_sample():
    layer = layer_for("small", synth.spec_small_gqa)
    spec = layer.spec
    q_bits = synth.make_queries(spec, layer.data, 0)
    sl = spec.suffix_len(0)
    a, da = pu.gpu_step(layer, q_bits, sl, 8, 99, 0)
    b, db = pu.gpu_step(layer, q_bits, sl, 8, 99, 0)
    assert np.array_equal(da.sel_idx.cpu().numpy(), db.sel_idx.cpu().numpy())
    assert np.abs(a - b).max() <= 1e-6 * pu.max_abs_v(layer)         # merge order may differ by rounding
    c, dc = pu.gpu_step(layer, q_bits, sl, 8, 100, 0)
    assert not np.array_equal(da.sel_idx.cpu().numpy(), dc.sel_idx.cpu().numpy())
    d, dd = pu.gpu_step(layer, q_bits, sl, 8, 99, 1)
    assert not np.array_equal(da.sel_idx.cpu().numpy(), dd.sel_idx.cpu().numpy())


def test_ragged_batch_medium():
    """Ragged CSR-of-CSR metadata: 6 sequences of different lengths, 31 sampled teams."""
    spec = synth.spec_ragged(n_steps=2, n_seqs=6, lo=1024, hi=6144)
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    check_team_records(layer, seqs=[0, 5], kv_heads=[1])
    check_sparse_step(layer, 0, K=31)
    check_dense_step(layer, 1)


def test_qwen_32k_full_size_batch1():
    """Config 2 at full size (28 heads over 4 KV heads, 32K prompt, 2048 teams per KV head,
    32 sampled teams): every head against the oracle, several steps; team records of one KV
    head against the oracle's Algorithm 2."""
    layer = layer_for("qwen_b1", synth.spec_qwen_b1)
    check_team_records(layer, kv_heads=[2])
    for step in (0, 7, 255):
        check_sparse_step(layer, step, K=32)
    check_sparse_step(layer, 3, K=32, suffix_len=[0])
    check_sparse_step(layer, 4, K=31)
    check_sparse_step(layer, 5, K=128)
    check_dense_step(layer, 9)


def test_keys_in_runs_variant():
    """Cluster ids in geometric runs (positional locality): smaller, more even teams than with
    independent draws; same method, same bars."""
    import dataclasses
    spec = dataclasses.replace(synth.spec_small_gqa(prompt=(2048, 1500)), key_layout="runs")
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    check_team_records(layer, kv_heads=[0])
    for step in range(2):
        check_sparse_step(layer, step, K=8)
    check_dense_step(layer, 0)


def test_centroid_guided_groups():
    """Groups routed by their mean key (one group per contiguous parent): records equal to the
    oracle's, bit for bit, and a decode step on them matches the oracle like any other."""
    import dataclasses
    spec = dataclasses.replace(synth.spec_small_gqa(prompt=(2048, 1100)), parent_size=16, reps_per_parent=1,
                               n_sample=24)
    data = synth.make_layer(spec)
    layer = pu.GpuLayer(spec, data, builder=sp.santapp_build_groups_mean)
    for b in range(spec.n_seqs):
        r0, r1 = int(layer.seq_row_off[b]), int(layer.seq_row_off[b + 1])
        for j in range(spec.n_kv_heads):
            ts_o, tm_o, mean_o = orc.group_mean_keys(synth.bf16_to_f64(data.k_prompt[j, r0:r1]), spec.parent_size)
            ts_g, tm_g, rep_g = layer.records(b, j)
            assert np.array_equal(ts_g, ts_o) and np.array_equal(tm_g, tm_o)
            assert np.array_equal(rep_g, mean_o)
            assert np.array_equal(layer.k_packed_bits[j, r0:r1], data.k_prompt[j, r0:r1])
            assert np.array_equal(layer.v_packed_bits[j, r0:r1], data.v_prompt[j, r0:r1])
    for step in range(2):
        check_sparse_step(layer, step, K=24)
    check_dense_step(layer, 0)
    # the builder insists on one group per parent
    bad = sp.Geometry(spec.n_seqs, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, 16, 4)
    with pytest.raises(sp.SantappError):
        sp.santapp_build_groups_mean(bad, spec.prompt_len, layer.k_prompt, layer.v_prompt)


def test_paper_operating_point_32k():
    """Parents of 16 keys with 4 representatives at 32K (8192 teams of about 4 rows per KV head),
    31 sampled teams, no suffix: routing reads an eighth of the dense bytes, gathers are tiny."""
    layer = layer_for("paper_point", synth.spec_paper_point)
    check_team_records(layer, kv_heads=[1])
    for step in (0, 9):
        check_sparse_step(layer, step, K=31)
    check_dense_step(layer, 2)


def test_paper_operating_point_128k():
    """The same operating point at 131072 tokens: 32768 teams per KV head."""
    spec = synth.spec_paper_point(prompt=131072)
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    check_sparse_step(layer, 0, K=31)
    check_dense_step(layer, 1)


def test_qwen_32k_batch8_concentrated_sampled_sequences():
    """Config 3 shape (8 sequences, 64 sampled teams, concentrated queries): the GPU runs the
    whole batch, the oracle checks two of the sequences."""
    layer = layer_for("qwen_b8", synth.spec_qwen_b8, n_steps=2)
    check_sparse_step(layer, 0, K=64, seqs=[0, 5])
    check_dense_step(layer, 1, seqs=[3])


def _query_from_rows(layer, rows, gain):
    """Queries that point at given prompt rows: q[b, h] = gain * k[row], rounded to bf16."""
    spec = layer.spec
    q = np.zeros((spec.n_seqs, spec.n_q_heads, spec.head_dim), dtype=np.uint16)
    for b in range(spec.n_seqs):
        r0 = int(layer.seq_row_off[b])
        for h in range(spec.n_q_heads):
            k = synth.bf16_to_f32(layer.data.k_prompt[h // spec.group, r0 + rows[b]])
            q[b, h] = synth.f32_to_bf16_bits(gain * k)
    return q


def _check_with_queries(layer, q_bits, K, step=0, seed=77):
    spec = layer.spec
    sl = spec.suffix_len(step)
    out, dbg = pu.gpu_step(layer, q_bits, sl, K, seed, step, 0)
    ref = pu.oracle_step(layer, q_bits, sl, K, seed, step, 0)
    sel = dbg.sel_idx.cpu().numpy()
    vmax = pu.max_abs_v(layer)
    for b, r in ref.items():
        assert np.all(r.margin > 1e-9)
        assert np.array_equal(sel[b, :, :K], r.sel[:, :K]), f"sampled teams differ (seq {b})"
        assert np.allclose(dbg.sel_logc.cpu().numpy()[b, :, :K], r.logc[:, :K], rtol=0, atol=1e-5)
        assert np.abs(out[b] - r.o).max() <= SPARSE_TOL * vmax


@pytest.mark.parametrize("boost", [3.0, 16.0])
def test_decode_outlier_score_far_above_the_rest(boost):
    """One team's routing score towers over the others (its representative's key is scaled up and
    the queries point at it): the bound on the (K+1)-st score has to look far below the top
    (moderate boost) or give up and re-evaluate every team (large boost)."""
    spec = synth.spec_small_gqa(n_seqs=2, prompt=(2048, 1536), parent_size=128, reps=16, n_sample=8)
    data = synth.make_layer(spec)
    rows = [37, 900]
    for b in range(spec.n_seqs):
        r = int(data.seq_row_off[b]) + rows[b]
        k = synth.bf16_to_f32(data.k_prompt[:, r])
        data.k_prompt[:, r] = synth.f32_to_bf16_bits(boost * k)
    layer = pu.GpuLayer(spec, data)
    _check_with_queries(layer, _query_from_rows(layer, rows, 2.0), K=8)


def test_decode_identical_keys_large_norm_every_team_is_a_candidate():
    """All keys equal and large: the fp32 scores of all teams agree to within the guard, so every
    one of the 1024 teams is re-evaluated exactly (more than fit in one pass), and the ranking is
    decided by log n_g and the Gumbel terms alone."""
    spec = synth.spec_small_gqa(n_seqs=1, prompt=(8192,), parent_size=128, reps=16, n_sample=8, suffix0=(3,))
    data = synth.make_layer(spec)
    k0 = synth.bf16_to_f32(data.k_prompt[0, 0]) * 24.0
    data.k_prompt[:] = synth.f32_to_bf16_bits(k0)
    layer = pu.GpuLayer(spec, data)
    _check_with_queries(layer, _query_from_rows(layer, [5], 2.0), K=8)
    _check_with_queries(layer, _query_from_rows(layer, [5], 2.0), K=40, step=1)


def test_decode_many_short_sequences():
    """24 sequences (672 query heads, 96 pairs): plans in global memory, equal row ranges, and the
    sampler's smaller blocks."""
    spec = synth.spec_small_gqa(n_seqs=24, prompt=tuple(384 + 64 * (i % 5) for i in range(24)), parent_size=64,
                                reps=8, n_sample=8, suffix0=tuple(i % 4 for i in range(24)))
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    check_sparse_step(layer, 0, K=8)
    check_sparse_step(layer, 1, K=40)
    check_dense_step(layer, 0)


@pytest.mark.parametrize("n_q,n_kv", [(32, 4), (8, 2), (6, 6), (3, 1)])
def test_decode_other_group_sizes(n_q, n_kv):
    """GQA groups of 8, 4, 1 and 3 query heads per KV head (the tensor-core tile holds up to 8)."""
    import dataclasses
    spec = dataclasses.replace(synth.spec_small_gqa(prompt=(1100, 640)), n_q_heads=n_q, n_kv_heads=n_kv)
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    check_sparse_step(layer, 0, K=8)
    check_sparse_step(layer, 1, K=33)
    check_dense_step(layer, 0)


def test_non_finite_query_raises_status_bits_and_leaves_the_library_usable():
    """A NaN query makes every routing score of its head incomparable: the call must finish, say so
    in the status word (bit 1: sample completed arbitrarily; bit 0: non-finite output), hand on only
    valid team ids, and the next clean call must be unaffected."""
    layer = layer_for("small", synth.spec_small_gqa)
    spec = layer.spec
    q_bits = synth.make_queries(spec, layer.data, 0).copy()
    q_bits[0, 3, :] = 0x7FC0                                          # bf16 NaN in every dim of one head
    sl = spec.suffix_len(0)
    out, dbg = pu.gpu_step(layer, q_bits, sl, 8, 5, 0)
    status = int(dbg.status.item())
    assert status & 2 and status & 1
    sel = dbg.sel_idx.cpu().numpy()
    Ms = np.diff(layer.seq_team_off)
    for b in range(spec.n_seqs):
        assert sel[b].min() >= 0 and sel[b].max() < Ms[b]
    assert np.isnan(out[0, 3]).all()
    assert np.isfinite(out[1]).all()                                  # other sequences are untouched
    check_sparse_step(layer, 0, K=8)                                  # and a clean call still matches the oracle


def test_ragged_batch_full_size_sampled_sequences():
    """Config 4 at full size (32 sequences of 8K to 64K tokens, suffixes up to 1024 rows, 31 sampled
    teams): the GPU runs the whole batch, the oracle checks the shortest, the longest and one more."""
    layer = layer_for("ragged_full", synth.spec_ragged)
    lens = np.asarray(layer.spec.prompt_len)
    seqs = sorted({int(lens.argmin()), int(lens.argmax()), 17})
    check_sparse_step(layer, 0, K=31, seqs=seqs)
    check_sparse_step(layer, 127, K=31, seqs=seqs[:1])
    check_dense_step(layer, 3, seqs=seqs[-1:])
    _cache.pop(("ragged_full", ()), None)                              # 2 GB of device memory


def test_long_context_128k_sampled_sequence():
    """Config 5 shape (4 sequences of 131072 tokens, 8192 teams per KV head): budgets 16 and 128,
    one sequence against the oracle."""
    layer = layer_for("long", synth.spec_long)
    check_sparse_step(layer, 0, K=16, seqs=[2])
    check_sparse_step(layer, 1, K=128, seqs=[0])
    check_dense_step(layer, 0, seqs=[3])
    _cache.pop(("long", ()), None)


def test_decode_more_pairs_than_one_window():
    """160 short sequences = 640 (sequence, KV head) pairs, more than the attention kernel stages at
    a time; the oracle checks the first, the last and two in between."""
    n = 160
    spec = synth.spec_small_gqa(n_seqs=n, prompt=tuple(192 + 64 * (i % 3) for i in range(n)), parent_size=64, reps=8,
                                n_sample=8, suffix0=tuple(i % 3 for i in range(n)))
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    seqs = [0, 53, 106, n - 1]
    check_sparse_step(layer, 0, K=8, seqs=seqs)
    check_dense_step(layer, 1, seqs=seqs)


def test_device_side_step_offset_equals_explicit_step():
    """step = 3 with a device-side offset of 4 draws the same sample as step = 7."""
    layer = layer_for("small", synth.spec_small_gqa)
    spec = layer.spec
    q = sp.bf16_bits_to_cuda(synth.make_queries(spec, layer.data, 0))
    sl = torch.from_numpy(spec.suffix_len(0)).cuda()
    d1 = sp.DebugBuffers(layer.geom, 8, "cuda")
    d2 = sp.DebugBuffers(layer.geom, 8, "cuda")
    off = torch.tensor([4], dtype=torch.int32, device="cuda")
    o1 = sp.santapp_decode_attn(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix, sl, 8, 11, 7, debug=d1)
    o2 = sp.santapp_decode_attn(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix, sl, 8, 11, 3, debug=d2,
                                step_dev=off)
    torch.cuda.synchronize()
    assert torch.equal(d1.sel_idx, d2.sel_idx)
    assert torch.allclose(o1, o2, rtol=0, atol=1e-6)


def test_stage_mask_reruns_one_stage_on_the_same_workspace():
    layer = layer_for("small", synth.spec_small_gqa)
    spec = layer.spec
    q = sp.bf16_bits_to_cuda(synth.make_queries(spec, layer.data, 1))
    sl = torch.from_numpy(spec.suffix_len(1)).cuda()
    ws = torch.empty(sp.santapp_decode_workspace_bytes(layer.geom, layer.teams, 8), dtype=torch.uint8, device="cuda")
    args = (layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix, sl, 8, 5, 1)
    full = sp.santapp_decode_attn(*args, workspace=ws).clone()
    assert sp.santapp_last_launch_count() == 4          # scoring, sampling + read plans, attention, merge
    try:
        # each stage alone, in pipeline order, reusing what the full call left in the workspace;
        # only the last stage writes the output
        for mask in (sp.STAGE_ATTEND | sp.STAGE_MERGE, sp.STAGE_ROUTE, sp.STAGE_SELECT, sp.STAGE_ATTEND, sp.STAGE_MERGE):
            sp.santapp_set_stage_mask(mask)
            again = sp.santapp_decode_attn(*args, workspace=ws)
            assert sp.santapp_last_launch_count() <= 3
            torch.cuda.synchronize()
            if mask & sp.STAGE_MERGE:
                assert torch.allclose(full, again, rtol=0, atol=1e-6)
    finally:
        sp.santapp_set_stage_mask(sp.STAGE_ALL)


def test_guard_words_around_the_workspaces_survive_every_call():
    """The decode, dense and build workspaces sit between guard words (a known pattern in the 4 KB
    before and after each): a kernel writing outside the sizes the library asked for would change
    them. One small batch with the plan inside the attention kernel, one ragged batch with plans in
    global memory."""
    def guarded(n_bytes):
        pad = 4096
        buf = torch.full((n_bytes + 2 * pad + 256,), 0xA5, dtype=torch.uint8, device="cuda")
        off = (-buf.data_ptr()) % 256                     # the workspace itself 256-byte aligned
        return buf, buf[off + pad: off + pad + n_bytes], (off, pad, n_bytes)

    def intact(buf, where):
        off, pad, n = where
        head, tail = buf[:off + pad], buf[off + pad + n:]
        return bool((head == 0xA5).all()) and bool((tail == 0xA5).all())

    cases = [synth.spec_small_gqa(seed=21),
             synth.spec_small_gqa(seed=22, n_seqs=24, prompt=tuple(200 + 97 * (i % 7) for i in range(24)), parent_size=64,
                                  reps=8, n_sample=8, suffix0=tuple(i % 5 for i in range(24)))]
    for spec in cases:
        layer = pu.GpuLayer(spec, synth.make_layer(spec))
        q_bits = synth.make_queries(spec, layer.data, 1)
        q = sp.bf16_bits_to_cuda(q_bits)
        sl_np = spec.suffix_len(1)
        sl = torch.from_numpy(sl_np).cuda()
        K = spec.n_sample
        buf, ws, where = guarded(sp.santapp_decode_workspace_bytes(layer.geom, layer.teams, K))
        dbg = sp.DebugBuffers(layer.geom, K, "cuda")
        out = sp.santapp_decode_attn(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix, sl, K, 77, 1, debug=dbg,
                                     workspace=ws)
        torch.cuda.synchronize()
        assert intact(buf, where), "decode wrote outside its workspace"
        ref = pu.oracle_step(layer, q_bits, sl_np, K, 77, 1)
        vmax = pu.max_abs_v(layer)
        for b, r in ref.items():
            assert np.array_equal(dbg.sel_idx.cpu().numpy()[b][:, :r.sel.shape[1]], r.sel)
            assert np.abs(out[b].cpu().numpy() - r.o).max() <= SPARSE_TOL * vmax
        buf, ws, where = guarded(sp.santapp_dense_workspace_bytes(layer.geom, layer.teams))
        dense = sp.santapp_dense_decode_attn(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix, sl, workspace=ws)
        torch.cuda.synchronize()
        assert intact(buf, where), "dense decode wrote outside its workspace"
        dref = pu.oracle_step(layer, q_bits, sl_np, 0, 0, 1, dense=True)
        for b, o in dref.items():
            assert np.abs(dense[b].cpu().numpy() - o).max() <= DENSE_TOL * vmax
        # the team builder's workspace, through the C ABI with a guarded buffer
        sizes = sp.santapp_build_teams_sizes(layer.geom, spec.prompt_len)
        buf, ws, where = guarded(max(sizes.build_workspace_bytes, 256))
        teams = sp.Teams(layer.geom, sizes, "cuda")
        import ctypes
        g = layer.geom.c()
        arr = (ctypes.c_int32 * spec.n_seqs)(*[int(x) for x in spec.prompt_len])
        rc = sp.load_library().santapp_build_teams(ctypes.byref(g), arr, ctypes.c_void_p(layer.k_prompt.data_ptr()),
                                                   ctypes.c_void_p(layer.v_prompt.data_ptr()), ctypes.byref(teams.c),
                                                   ctypes.c_void_p(ws.data_ptr()), ws.numel(), None)
        torch.cuda.synchronize()
        assert rc == 0 and intact(buf, where), "team build wrote outside its workspace"
        assert torch.equal(teams.team_row_start, layer.teams.team_row_start)
        assert torch.equal(teams.k_packed.view(torch.int16), layer.teams.k_packed.view(torch.int16))
