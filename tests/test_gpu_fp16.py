"""GPU parity with IEEE fp16 inputs (the element type of the paper's own kernel runs): the same
checks as for bf16 on team records, sampled teams and outputs, plus a case with softmax weights far below the fp16 range."""
import numpy as np
import pytest

from oracle import santapp_oracle as orc
from paper_2609_35629_b200 import binding as sp
from paper_2609_35629_b200 import synth

import parity_util as pu
from test_gpu_parity import DENSE_TOL, check_dense_step, check_sparse_step, check_team_records
from test_gpu_parents import _check_records, _labels_gpu, _layer_from_labels

pytestmark = pytest.mark.gpu


def _fp16(spec):
    spec.elem = "fp16"
    return spec


def test_fp16_small_gqa_records_and_steps():
    spec = _fp16(synth.spec_small_gqa())
    layer = pu.GpuLayer(spec, synth.make_layer(spec, layer=0))
    assert layer.teams.k_packed.dtype.itemsize == 2 and str(layer.teams.k_packed.dtype) == "torch.float16"
    check_team_records(layer)
    for step in range(spec.n_steps):
        check_sparse_step(layer, step, spec.n_sample)
    for K in (1, 31, 33):
        check_sparse_step(layer, 0, K)
    check_dense_step(layer, 1)


def test_fp16_results_differ_from_bf16_reading_of_the_same_bits():
    """Guard against a silent bf16 path: the same bit patterns read as bf16 give other team records."""
    spec = _fp16(synth.spec_small_gqa())
    data = synth.make_layer(spec, layer=0)
    layer = pu.GpuLayer(spec, data)
    spec_b = synth.spec_small_gqa()
    layer_b = pu.GpuLayer(spec_b, data)                       # same bits, declared bf16
    assert not np.array_equal(layer.row_token, layer_b.row_token)


def test_fp16_paper_operating_point_32k():
    """The paper's operating point in its own element type: P = 16, R = 4, K = 31, 32K, batch 1."""
    spec = _fp16(synth.spec_paper_point())
    layer = pu.GpuLayer(spec, synth.make_layer(spec, layer=0))
    check_team_records(layer, kv_heads=[3])
    for step in (0, 255):
        check_sparse_step(layer, step, K=31)
    check_dense_step(layer, 2)


def test_fp16_qwen_32k_and_ragged_dynamic_split():
    spec = _fp16(synth.spec_qwen_b1())
    layer = pu.GpuLayer(spec, synth.make_layer(spec, layer=0))
    check_sparse_step(layer, 1, K=32)
    spec = _fp16(synth.spec_ragged(n_seqs=12, lo=2048, hi=6144))
    layer = pu.GpuLayer(spec, synth.make_layer(spec, layer=0, keep_centres=True))
    check_team_records(layer, seqs=[0], kv_heads=[0])
    check_sparse_step(layer, 0, spec.n_sample)
    check_dense_step(layer, 0)


def test_fp16_centre_parents():
    spec = _fp16(synth.spec_small_gqa(prompt=(1536, 1000)))
    spec.reps_per_parent, spec.parent_size, spec.n_clusters = 4, 64, 24
    data = synth.make_layer(spec, layer=0, keep_centres=True)
    n_centres = [24, 9]
    cen = np.ascontiguousarray(np.concatenate([data.centres[:, :n] for n in n_centres], axis=1))
    labels = _labels_gpu(spec, data, n_centres, cen)
    row0 = c0 = 0
    for b, n in enumerate(n_centres):
        N = spec.prompt_len[b]
        for j in range(spec.n_kv_heads):
            keys = synth.to_f64(data.k_prompt[j, row0:row0 + N], "fp16")
            want, _, _ = orc.nearest_centre_parents(keys, cen[j, c0:c0 + n].astype(np.float64))
            assert np.array_equal(labels[j, row0:row0 + N], want)
        row0 += N
        c0 += n
    layer = _layer_from_labels(spec, data, labels, n_centres)
    _check_records(layer, labels, n_centres)
    check_sparse_step(layer, 0, spec.n_sample)


def test_fp16_weights_far_below_the_fp16_range_still_count():
    """One key scores 17.5 nats above 262143 others: relative to the global maximum each of those
    has a softmax weight of 2.5e-8, below anything fp16 can hold, yet together they hold 0.65 % of
    the mass. Weights are formed against the running maximum of each warp's own rows and merged in
    fp32, so the dense output must still match the oracle."""
    N = 262144
    spec = _fp16(synth.spec_small_gqa(n_seqs=1, prompt=(N,), suffix0=(0,)))
    data = synth.make_layer(spec, layer=0)
    rng = np.random.default_rng(7)
    d = spec.head_dim
    k = (0.02 * rng.standard_normal((spec.n_kv_heads, N, d))).astype(np.float32)
    k[:, 100, :] = 0.0
    k[:, 100, 0] = 6.0
    data.k_prompt[:] = synth.round_bits(k, "fp16")
    layer = pu.GpuLayer(spec, data)
    q = np.zeros((1, spec.n_q_heads, d), dtype=np.float32)
    q[..., 0] = 17.5 * np.sqrt(d) / 6.0                          # score of row 100: 17.5 nats, others near 0
    q_bits = synth.round_bits(q, "fp16")
    out, _ = pu.gpu_step(layer, q_bits, [0], 0, 0, 0, dense=True)
    ref = pu.oracle_step(layer, q_bits, [0], 0, 0, 0, dense=True)[0]
    vmax = pu.max_abs_v(layer)
    v100 = synth.to_f64(data.v_prompt[0, 100], "fp16")
    assert np.abs(ref[0] - v100).max() > 2 * DENSE_TOL * vmax       # the small weights matter at this tolerance
    assert np.abs(out[0] - ref).max() <= DENSE_TOL * vmax


def test_fp16_centroid_groups_contiguous_and_on_labels():
    """The centroid-guided baseline with fp16 inputs: the mean key is rounded to fp16, records equal the
    oracle's, and a decode step on them matches."""
    import dataclasses
    import torch
    spec = dataclasses.replace(synth.spec_small_gqa(prompt=(1024, 700)), parent_size=16, reps_per_parent=1,
                               n_sample=12, elem="fp16")
    data = synth.make_layer(spec)
    layer = pu.GpuLayer(spec, data, builder=sp.santapp_build_groups_mean)
    for b in range(spec.n_seqs):
        r0, r1 = int(layer.seq_row_off[b]), int(layer.seq_row_off[b + 1])
        for j in range(spec.n_kv_heads):
            keys = synth.to_f64(data.k_prompt[j, r0:r1], "fp16")
            ts_o, tm_o, mean_o = orc.group_mean_keys(keys, spec.parent_size, elem="fp16")
            ts_g, tm_g, rep_g = layer.records(b, j)
            assert np.array_equal(ts_g, ts_o) and np.array_equal(tm_g, tm_o) and np.array_equal(rep_g, mean_o)
    check_sparse_step(layer, 0, K=12)
    # the same on a random partition per KV head
    rng = np.random.default_rng(3)
    n_parents = [50, 33]
    labels = np.concatenate([rng.integers(0, p, size=(spec.n_kv_heads, n)) for p, n in zip(n_parents, spec.prompt_len)],
                            axis=1).astype(np.int32)
    lab_dev = torch.from_numpy(labels).cuda()
    layer2 = pu.GpuLayer(spec, data, builder=lambda g, n, k, v: sp.santapp_build_groups_mean_parents(g, n, n_parents, k, v, lab_dev))
    for b in range(spec.n_seqs):
        r0, r1 = int(layer2.seq_row_off[b]), int(layer2.seq_row_off[b + 1])
        for j in range(spec.n_kv_heads):
            keys = synth.to_f64(data.k_prompt[j, r0:r1], "fp16")
            lab = labels[j, r0:r1]
            kept = np.unique(lab)
            ps = np.concatenate([[0], np.cumsum([np.count_nonzero(lab == u) for u in kept])]).astype(np.int32)
            pm = np.concatenate([np.flatnonzero(lab == u) for u in kept]).astype(np.int32)
            ts_o, tm_o, mean_o = orc.group_mean_keys_parents(keys, ps, pm, elem="fp16")
            ts_g, tm_g, rep_g = layer2.records(b, j)
            assert np.array_equal(ts_g, ts_o) and np.array_equal(tm_g, tm_o) and np.array_equal(rep_g, mean_o)
    check_sparse_step(layer2, 1, K=12)
