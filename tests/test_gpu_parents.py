"""GPU parity for parents that are not contiguous spans: the nearest-centre assignment that closes
Algorithm 3, Algorithm 2 on parents of any size with empty parents omitted, and a decode step over
records whose team count differs between the KV heads of a sequence. Integer results (labels, CSR
offsets, member order, representative rows, sampled teams) must match the fp64 oracle exactly.
"""
import numpy as np
import pytest
import torch

from oracle import santapp_oracle as orc
from paper_2609_35629_b200 import binding as sp
from paper_2609_35629_b200 import synth

import parity_util as pu
from test_gpu_parity import check_dense_step, check_sparse_step

pytestmark = pytest.mark.gpu


def _spec(prompt=(1536, 1000), n_sample=8, R=4, n_clusters=24):
    spec = synth.spec_small_gqa(n_seqs=len(prompt), prompt=prompt, n_sample=n_sample)
    spec.reps_per_parent = R
    spec.parent_size = 64
    spec.n_clusters = n_clusters
    return spec


def _centres_for(spec, data, n_centres):
    """fp32 centres per KV head and sequence: the generating centres of the synthetic keys, with
    traps: a repeated centre (an exact tie), a centre far from every key (an empty parent) and a
    centre that coincides with one key (a parent of very few tokens)."""
    rng = np.random.default_rng(99)
    out = np.zeros((spec.n_kv_heads, sum(n_centres), spec.head_dim), dtype=np.float32)
    off = 0
    row0 = 0
    for b, n in enumerate(n_centres):
        for j in range(spec.n_kv_heads):
            c = data.centres[j, rng.permutation(spec.n_clusters)[:n]].copy()
            if n >= 4:
                c[n - 1] = c[0]                                        # tie: never wins
                c[n - 2] = 100.0                                       # attracts nothing
                key = synth.bf16_to_f32(data.k_prompt[j, row0 + 7])
                c[n - 3] = key                                         # sits on token 7
            out[j, off:off + n] = c
        off += n
        row0 += spec.prompt_len[b]
    return out


def _labels_gpu(spec, data, n_centres, centres):
    geom = pu.geometry(spec)
    k = sp.bf16_bits_to_cuda(data.k_prompt)
    lab = sp.santapp_assign_parents(geom, spec.prompt_len, n_centres, k, torch.from_numpy(centres).cuda())
    torch.cuda.synchronize()
    return lab.cpu().numpy()


def test_assignment_matches_the_oracle_with_ties_and_empty_centres():
    spec = _spec()
    data = synth.make_layer(spec, layer=0, keep_centres=True)
    n_centres = [24, 9]
    centres = _centres_for(spec, data, n_centres)
    lab = _labels_gpu(spec, data, n_centres, centres)
    row0 = c0 = 0
    for b, n in enumerate(n_centres):
        N = spec.prompt_len[b]
        for j in range(spec.n_kv_heads):
            keys = synth.bf16_to_f64(data.k_prompt[j, row0:row0 + N])
            want, ps, _ = orc.nearest_centre_parents(keys, centres[j, c0:c0 + n].astype(np.float64))
            assert np.array_equal(lab[j, row0:row0 + N], want)
            assert not np.any(want == n - 1) and not np.any(want == n - 2)     # the traps stayed empty
            assert ps.shape[0] - 1 < n
        row0 += N
        c0 += n


def _check_records(layer, labels, n_parents):
    spec = layer.spec
    for b in range(spec.n_seqs):
        r0, r1 = int(layer.seq_row_off[b]), int(layer.seq_row_off[b + 1])
        N = r1 - r0
        slots = int(layer.seq_team_off[b + 1] - layer.seq_team_off[b])
        assert slots == min(N, n_parents[b] * spec.reps_per_parent)
        for j in range(spec.n_kv_heads):
            keys = synth.to_f64(layer.data.k_prompt[j, r0:r1], spec.elem)
            lab = np.clip(labels[j, r0:r1], 0, n_parents[b] - 1)
            kept = np.unique(lab)
            ps = np.concatenate([[0], np.cumsum([np.count_nonzero(lab == u) for u in kept])]).astype(np.int32)
            pm = np.concatenate([np.flatnonzero(lab == u) for u in kept]).astype(np.int32)
            ts_o, tm_o, rep_o = orc.build_teams(keys, ps, pm, spec.reps_per_parent)
            ts_g, tm_g, rep_g = layer.records(b, j)
            assert len(ts_g) == len(ts_o), "team count"
            assert np.array_equal(ts_g, ts_o)
            assert np.array_equal(tm_g, tm_o)
            assert np.array_equal(rep_g, keys[rep_o])
            assert np.array_equal(layer.k_packed_bits[j, r0:r1], layer.data.k_prompt[j, r0:r1][tm_g])
            assert np.array_equal(layer.v_packed_bits[j, r0:r1], layer.data.v_prompt[j, r0:r1][tm_g])
            # slots behind the last team are empty teams
            t0 = int(layer.seq_team_off[b])
            M = len(ts_o) - 1
            tail = layer.team_row_start[j, t0 + b + M: t0 + b + slots + 1]
            assert np.all(tail == N)
            assert not layer.rep_bits[j, t0 + M: t0 + slots].any()


def _layer_from_labels(spec, data, labels, n_parents):
    lab_dev = torch.from_numpy(np.ascontiguousarray(labels, dtype=np.int32)).cuda()

    def builder(geom, prompt_len, k, v):
        return sp.santapp_build_teams_parents(geom, prompt_len, n_parents, k, v, lab_dev)
    return pu.GpuLayer(spec, data, builder=builder)


def test_records_from_centre_parents_match_algorithm_2_of_the_oracle():
    spec = _spec()
    data = synth.make_layer(spec, layer=0, keep_centres=True)
    n_centres = [24, 9]
    labels = _labels_gpu(spec, data, n_centres, _centres_for(spec, data, n_centres))
    layer = _layer_from_labels(spec, data, labels, n_centres)
    _check_records(layer, labels, n_centres)
    for step in range(2):
        check_sparse_step(layer, step, spec.n_sample)
    check_dense_step(layer, 0)


def test_records_from_arbitrary_labels_large_and_single_token_parents():
    """Labels that no clustering would produce: one parent of 1200 tokens (more than any contiguous
    parent may hold), single-token parents, empty labels, labels outside the range (clamped), and
    a different partition for each KV head."""
    spec = _spec(prompt=(1536, 700), n_sample=6, R=8)
    data = synth.make_layer(spec, layer=0, keep_centres=True)
    rng = np.random.default_rng(4)
    n_parents = [40, 12]
    labels = np.zeros((spec.n_kv_heads, spec.rows_total), dtype=np.int32)
    for j in range(spec.n_kv_heads):
        a = rng.integers(2, 36, size=1536)
        a[rng.permutation(1536)[:1200]] = 1                            # the big parent, scattered
        a[5], a[900] = 37, 38                                          # singletons
        a[6] = -3                                                      # clamped to 0
        a[7] = 1000                                                    # clamped to 39
        bseq = rng.integers(0, 12 - j, size=700)                       # head j never uses its last labels
        labels[j] = np.concatenate([a, bseq])
    layer = _layer_from_labels(spec, data, labels, n_parents)
    _check_records(layer, labels, n_parents)
    check_sparse_step(layer, 0, spec.n_sample)
    check_dense_step(layer, 0)


def test_pair_with_fewer_teams_than_the_budget_reads_every_team():
    """One KV head of a sequence ends up with at most K teams while the others have more: that pair
    reads all its teams uncorrected (K = min(K, M) in Algorithm 1), the others sample."""
    spec = _spec(prompt=(600, 512), n_sample=8, R=4)
    data = synth.make_layer(spec, layer=0, keep_centres=True)
    rng = np.random.default_rng(8)
    n_parents = [16, 16]
    labels = np.zeros((spec.n_kv_heads, spec.rows_total), dtype=np.int32)
    for j in range(spec.n_kv_heads):
        labels[j, :600] = rng.integers(0, 16, size=600)
        labels[j, 600:] = rng.integers(0, 16, size=512)
    labels[1, :600] = rng.integers(3, 5, size=600)                     # two parents: 8 teams = K
    labels[2, 600:] = 9                                                # one parent: 4 teams < K
    layer = _layer_from_labels(spec, data, labels, n_parents)
    _check_records(layer, labels, n_parents)
    assert int(layer.team_count[1, 0]) == 8 and int(layer.team_count[2, 1]) == 4
    assert int(layer.team_count[0, 0]) == 64
    for step in range(2):
        check_sparse_step(layer, step, spec.n_sample)


def test_contiguous_builder_reports_every_slot_as_a_team():
    spec = synth.spec_small_gqa()
    layer = pu.GpuLayer(spec, synth.make_layer(spec, layer=0))
    want = np.diff(layer.seq_team_off).astype(np.int32)
    assert np.array_equal(layer.team_count, np.tile(want, (spec.n_kv_heads, 1)))


def _centre_layer(spec):
    """The configuration `bench.py --parents centres` times: as many of the generating centres as the
    first line of Algorithm 3 asks for, assignment and records built on the GPU."""
    data = synth.make_layer(spec, layer=0, keep_centres=True)
    n_cen = [min(sp.santapp_kmeans_parent_count(n, spec.parent_size), spec.n_clusters) for n in spec.prompt_len]
    cen = np.ascontiguousarray(np.concatenate([data.centres[:, :n] for n in n_cen], axis=1))
    labels = _labels_gpu(spec, data, n_cen, cen)
    return _layer_from_labels(spec, data, labels, n_cen), labels, n_cen, cen


def test_centre_parents_32k_full_size():
    """Config 2's shape with parents from centres instead of contiguous spans: labels and records of
    one KV head against the oracle, then decode steps of every head."""
    spec = synth.spec_qwen_b1()
    layer, labels, n_cen, cen = _centre_layer(spec)
    j = 1
    keys = synth.bf16_to_f64(layer.data.k_prompt[j])
    want, ps, pm = orc.nearest_centre_parents(keys, cen[j].astype(np.float64))
    assert np.array_equal(labels[j], want)
    ts_o, tm_o, rep_o = orc.build_teams(keys, ps, pm, spec.reps_per_parent)
    ts_g, tm_g, rep_g = layer.records(0, j)
    assert np.array_equal(ts_g, ts_o) and np.array_equal(tm_g, tm_o) and np.array_equal(rep_g, keys[rep_o])
    sizes = np.diff(ps)
    assert sizes.max() > spec.parent_size                      # parents larger than any contiguous one
    for step in (0, 255):
        check_sparse_step(layer, step, K=32)
    check_dense_step(layer, 3)


def test_centre_parents_paper_point_32k():
    """The paper's operating point (P = 16, R = 4, K = 31) on centre parents: 2048 parents of uneven
    size, a different team count for every KV head."""
    spec = synth.spec_paper_point()
    layer, _, _, _ = _centre_layer(spec)
    assert len({int(c) for c in layer.team_count[:, 0]}) > 1
    check_sparse_step(layer, 0, K=31)


def test_centroid_groups_on_centre_parents():
    """The paper's centroid-guided baseline on a clustering's groups (nominal group size 16): one
    group per non-empty parent routed by its mean key; records equal to the oracle's, decode as usual."""
    spec = _spec(prompt=(2048, 1100), n_sample=12, R=1, n_clusters=128)
    spec.parent_size = 16
    data = synth.make_layer(spec, layer=0, keep_centres=True)
    n_centres = [sp.santapp_kmeans_parent_count(n, spec.parent_size) for n in spec.prompt_len]     # 128, 68
    cen = np.ascontiguousarray(np.concatenate([data.centres[:, :n] for n in n_centres], axis=1))
    labels = _labels_gpu(spec, data, n_centres, cen)
    lab_dev = torch.from_numpy(labels).cuda()

    def builder(geom, prompt_len, k, v):
        return sp.santapp_build_groups_mean_parents(geom, prompt_len, n_centres, k, v, lab_dev)
    layer = pu.GpuLayer(spec, data, builder=builder)
    for b in range(spec.n_seqs):
        r0, r1 = int(layer.seq_row_off[b]), int(layer.seq_row_off[b + 1])
        for j in range(spec.n_kv_heads):
            keys = synth.bf16_to_f64(data.k_prompt[j, r0:r1])
            _, ps, pm = orc.nearest_centre_parents(keys, cen[j, sum(n_centres[:b]):sum(n_centres[:b + 1])].astype(np.float64))
            ts_o, tm_o, mean_o = orc.group_mean_keys_parents(keys, ps, pm)
            ts_g, tm_g, rep_g = layer.records(b, j)
            assert np.array_equal(ts_g, ts_o) and np.array_equal(tm_g, tm_o) and np.array_equal(rep_g, mean_o)
            assert np.array_equal(layer.k_packed_bits[j, r0:r1], data.k_prompt[j, r0:r1][tm_g])
    for step in range(2):
        check_sparse_step(layer, step, spec.n_sample)
    bad = pu.geometry(_spec(prompt=(2048, 1100), R=4))
    with pytest.raises(sp.SantappError):
        sp.santapp_build_groups_mean_parents(bad, spec.prompt_len, n_centres, layer.k_prompt, layer.v_prompt, lab_dev)


def test_null_team_count_means_every_slot_is_a_team():
    """Records of the contiguous builder fill every slot, so the decode must give the same bits with
    team_count left NULL (callers that built their records before the field existed)."""
    spec = synth.spec_small_gqa()
    layer = pu.GpuLayer(spec, synth.make_layer(spec, layer=0))
    q_bits = synth.make_queries(spec, layer.data, 0)
    sl = spec.suffix_len(0)
    out_a, dbg_a = pu.gpu_step(layer, q_bits, sl, spec.n_sample, 5, 0)
    saved = layer.teams.c.team_count
    layer.teams.c.team_count = None
    try:
        out_b, dbg_b = pu.gpu_step(layer, q_bits, sl, spec.n_sample, 5, 0)
        dense_b, _ = pu.gpu_step(layer, q_bits, sl, 0, 0, 0, dense=True)
    finally:
        layer.teams.c.team_count = saved
    dense_a, _ = pu.gpu_step(layer, q_bits, sl, 0, 0, 0, dense=True)
    assert np.array_equal(out_a, out_b) and np.array_equal(dense_a, dense_b)
    assert torch.equal(dbg_a.sel_idx, dbg_b.sel_idx)
