"""GPU parity for the minibatch k-means fit of Algorithm 3: the CUDA fit and the fp64 oracle take
the same random words and the same fp64 arithmetic in the same order, so centres (rounded to fp32)
and step counts must be equal, not merely close."""
import numpy as np
import pytest
import torch

from oracle import santapp_oracle as orc
from paper_2609_35629_b200 import binding as sp
from paper_2609_35629_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu


def _fit_both(spec, n_centres, **opts):
    data = synth.make_layer(spec, layer=0, keep_centres=True)
    geom = pu.geometry(spec)
    k = sp.bf16_bits_to_cuda(data.k_prompt, dtype=geom.torch_dtype)
    centres, steps = sp.santapp_kmeans_fit(geom, spec.prompt_len, n_centres, k, **opts)
    torch.cuda.synchronize()
    centres, steps = centres.cpu().numpy(), steps.cpu().numpy()
    base = opts.get("stream_base", 0)
    o = {kk: v for kk, v in opts.items() if kk not in ("stream_base", "no_host_poll")}
    o = {"batch": o.pop("batch_size", 4096), "ratio": o.pop("reassignment_ratio", 0.01), **o}
    row0 = c0 = 0
    for b, kc in enumerate(n_centres):
        N = spec.prompt_len[b]
        for j in range(spec.n_kv_heads):
            keys = synth.to_f64(data.k_prompt[j, row0:row0 + N], spec.elem)
            want, want_steps = orc.minibatch_kmeans(keys, kc, stream=base + b * spec.n_kv_heads + j, **o)
            assert int(steps[j, b]) == want_steps, f"steps of pair ({b}, {j})"
            assert np.array_equal(centres[j, c0:c0 + kc], want.astype(np.float32)), f"centres of pair ({b}, {j})"
        row0 += N
        c0 += kc
    return data, centres, steps


def test_fit_matches_the_oracle_on_two_ragged_sequences():
    spec = synth.spec_small_gqa(prompt=(1536, 1000))
    spec.n_clusters = 24
    n_centres = [24, 9]
    _, _, steps = _fit_both(spec, n_centres, batch_size=256, seed=3, stream_base=11)
    assert steps.min() >= 10


def test_fit_with_reassignment_every_period_and_short_patience():
    """A high ratio moves centres at every period, a patience of 2 stops early, k is not a multiple of
    the centres a block updates, and the sample is the whole sequence."""
    spec = synth.spec_small_gqa(prompt=(700,), n_seqs=1, suffix0=(0,))
    _fit_both(spec, [13], batch_size=512, reassignment_ratio=0.9, patience=2, max_iter=30, seed=1 << 40)
    _fit_both(spec, [13], batch_size=64, reassignment_ratio=0.0, patience=10 ** 6, max_iter=2)


def test_fit_without_host_polling_gives_the_same_centres():
    """With no_host_poll the call never waits for the stream: every step up to the limit is enqueued
    and the steps of a fit that has already stopped do nothing, so centres and step counts stay
    those of the oracle (two sequences whose fits stop at different steps)."""
    spec = synth.spec_small_gqa(prompt=(1536, 1000))
    spec.n_clusters = 24
    _, _, steps = _fit_both(spec, [24, 9], batch_size=256, seed=3, stream_base=11, max_iter=20, no_host_poll=True)
    assert len(set(steps.ravel().tolist())) > 1
    assert steps.max() < 20 * 6                                 # the fits stopped before the limit


def test_fit_without_host_polling_can_be_captured_in_a_cuda_graph():
    """With no_host_poll the call only enqueues work: captured in a CUDA graph on a side stream and
    replayed twice, it leaves the centres and step counts of the plain call (which the test above
    compares with the oracle)."""
    spec = synth.spec_small_gqa(prompt=(1536, 1000))
    spec.n_clusters = 24
    data = synth.make_layer(spec, layer=0, keep_centres=True)
    geom = pu.geometry(spec)
    k = sp.bf16_bits_to_cuda(data.k_prompt, dtype=geom.torch_dtype)
    opts = dict(batch_size=256, seed=3, stream_base=11, max_iter=20, no_host_poll=True)
    want_c, want_s = sp.santapp_kmeans_fit(geom, spec.prompt_len, [24, 9], k, **opts)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        got_c, got_s = sp.santapp_kmeans_fit(geom, spec.prompt_len, [24, 9], k, **opts)
    for _ in range(2):
        got_c.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(got_c, want_c) and torch.equal(got_s, want_s)


def test_fit_on_a_sequence_too_long_for_the_shared_memory_shuffle():
    """52000 keys beside 900: the long sequence's index list does not fit in shared memory, so its
    initialisation sample is shuffled in global memory, the short one's in shared memory."""
    spec = synth.spec_small_gqa(prompt=(52000, 900), suffix0=(0, 0))
    spec.n_clusters = 16
    _fit_both(spec, [11, 6], batch_size=192, seed=5, max_iter=3, patience=4)


def test_fit_of_150_short_sequences_takes_its_tables_in_two_chunks():
    """More sequences than one kernel-argument chunk of the per-sequence tables holds (128)."""
    rng = np.random.default_rng(9)
    lens = tuple(int(x) for x in rng.integers(30, 70, size=150))
    spec = synth.spec_small_gqa(n_seqs=150, prompt=lens, suffix0=(0,) * 150)
    spec.n_clusters = 4
    _fit_both(spec, [2 + (i % 3) for i in range(150)], batch_size=16, seed=2, max_iter=2, patience=3)


def test_fit_fp16_inputs():
    spec = synth.spec_small_gqa(prompt=(900,), n_seqs=1, suffix0=(0,))
    spec.elem = "fp16"
    _fit_both(spec, [7], batch_size=128)


def test_fit_then_parents_then_decode():
    """Algorithm 3 end to end on the GPU (count, fit, assignment, omission of empty parents), then
    Algorithm 2 and a decode step on the result, each against the oracle."""
    from test_gpu_parents import _check_records, _layer_from_labels
    from test_gpu_parity import check_sparse_step
    spec = synth.spec_small_gqa(prompt=(2048, 1200))
    spec.parent_size, spec.reps_per_parent, spec.n_clusters = 64, 4, 32
    n_centres = [sp.santapp_kmeans_parent_count(n, spec.parent_size) for n in spec.prompt_len]
    assert n_centres == [32, 18]
    data, centres, _ = _fit_both(spec, n_centres, batch_size=512)
    geom = pu.geometry(spec)
    k = sp.bf16_bits_to_cuda(data.k_prompt)
    labels = sp.santapp_assign_parents(geom, spec.prompt_len, n_centres, k, torch.from_numpy(centres).cuda())
    torch.cuda.synchronize()
    labels = labels.cpu().numpy()
    keys = synth.bf16_to_f64(data.k_prompt[2, :2048])
    want, _, _ = orc.nearest_centre_parents(keys, centres[2, :32].astype(np.float64))
    assert np.array_equal(labels[2, :2048], want)
    layer = _layer_from_labels(spec, data, labels, n_centres)
    _check_records(layer, labels, n_centres)
    check_sparse_step(layer, 0, spec.n_sample)


def _one_pair_at_full_size(spec, j, **opts):
    """Fit every pair on the GPU, check one KV head against the oracle (the oracle takes seconds per pair)."""
    data = synth.make_layer(spec, layer=0)
    geom = pu.geometry(spec)
    n_centres = [sp.santapp_kmeans_parent_count(n, spec.parent_size) for n in spec.prompt_len]
    k = sp.bf16_bits_to_cuda(data.k_prompt)
    centres, steps = sp.santapp_kmeans_fit(geom, spec.prompt_len, n_centres, k, **opts)
    torch.cuda.synchronize()
    keys = synth.bf16_to_f64(data.k_prompt[j, :spec.prompt_len[0]])
    want, want_steps = orc.minibatch_kmeans(keys, n_centres[0], stream=j)
    assert int(steps[j, 0]) == want_steps
    assert np.array_equal(centres[j, :n_centres[0]].cpu().numpy(), want.astype(np.float32))
    return n_centres


def test_fit_config_2_full_size_paper_settings():
    """32K keys per KV head, 64 centres, the paper's settings (minibatch 4096, 100 iterations,
    patience 10, ratio 0.01, seed 0): the configuration `bench.py --parents kmeans` prepares."""
    assert _one_pair_at_full_size(synth.spec_qwen_b1(), j=1) == [64]


def test_fit_many_centres_paper_parent_size():
    """Parents of nominal size 16 (the paper's operating point) on 8K keys: 512 centres, 8 trials per
    centre, the initialisation sample is the whole sequence."""
    assert _one_pair_at_full_size(synth.spec_paper_point(prompt=8192), j=3) == [512]


@pytest.mark.parametrize("case", range(16))
def test_fit_random_small_configurations(case):
    rng = np.random.default_rng(500 + case)
    n_seqs = int(rng.integers(1, 4))
    prompt = tuple(int(rng.integers(2, 1500)) for _ in range(n_seqs))
    spec = synth.spec_small_gqa(n_seqs=n_seqs, prompt=prompt, suffix0=(0,) * n_seqs)
    spec.n_clusters = int(rng.integers(2, 30))
    spec.seed = case
    spec.elem = "fp16" if case % 2 else "bf16"
    n_centres = [int(rng.integers(1, min(n, 40) + 1)) for n in prompt]
    _fit_both(spec, n_centres, batch_size=int(rng.choice([16, 100, 512, 4096])), max_iter=int(rng.choice([1, 3, 100])),
              patience=int(rng.choice([1, 3, 10])), reassignment_ratio=float(rng.choice([0.0, 0.01, 0.5])),
              seed=int(rng.integers(1 << 62)), stream_base=int(rng.integers(1 << 30)))
