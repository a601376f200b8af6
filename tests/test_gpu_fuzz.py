"""Seeded random configurations through the whole path (records, one sparse step, one dense step)
against the oracle: shapes nobody would pick by hand (prompts of a few rows, budgets above and
below the team count, every group size, both element types, contiguous and label-given parents)."""
import numpy as np
import pytest
import torch

from paper_2609_35629_b200 import binding as sp
from paper_2609_35629_b200 import synth

import parity_util as pu
from test_gpu_parity import check_dense_step, check_sparse_step, check_team_records
from test_gpu_parents import _check_records, _layer_from_labels

pytestmark = pytest.mark.gpu

_GROUPS = [(1, 1), (2, 1), (3, 1), (4, 2), (6, 6), (8, 2), (10, 2), (12, 4), (14, 2), (28, 4), (16, 2), (32, 4)]
_PARENTS = [(1, 1), (2, 1), (4, 4), (8, 2), (16, 4), (32, 32), (64, 8), (100, 10), (128, 8), (512, 32), (512, 1)]


def _random_spec(rng):
    n_q, n_kv = _GROUPS[rng.integers(len(_GROUPS))]
    P, R = _PARENTS[rng.integers(len(_PARENTS))]
    n_seqs = int(rng.integers(1, 5))
    kind = rng.integers(3)
    if kind == 0:
        prompt = [int(rng.integers(1, 40)) for _ in range(n_seqs)]            # a few rows
    elif kind == 1:
        prompt = [int(rng.integers(40, 700)) for _ in range(n_seqs)]
    else:
        prompt = [int(rng.integers(700, 3000)) for _ in range(n_seqs)]
    cap = int(rng.choice([0, 1, 7, 32]))
    spec = synth.WorkloadSpec("fuzz", n_seqs, n_q, n_kv, prompt, int(rng.integers(2, 40)), P, R,
                              int(rng.choice([1, 2, 5, 16, 31, 64, 128])), 3, max(cap, 1),
                              [int(rng.integers(0, cap + 1)) for _ in range(n_seqs)], int(rng.integers(0, 2)),
                              seed=int(rng.integers(1 << 30)))
    spec.elem = "fp16" if rng.integers(2) else "bf16"
    spec.key_layout = "runs" if rng.integers(2) else "iid"
    return spec


@pytest.mark.parametrize("case", range(150))
def test_random_configuration(case):
    rng = np.random.default_rng(1000 + case)
    spec = _random_spec(rng)
    G = spec.n_q_heads // spec.n_kv_heads
    K = spec.n_sample
    data = synth.make_layer(spec, layer=0)
    by_labels = case % 3 == 2
    if by_labels:
        n_parents = [int(rng.integers(1, max(2, n // max(spec.parent_size // 2, 1) + 2))) for n in spec.prompt_len]
        labels = np.concatenate([rng.integers(0, p, size=(spec.n_kv_heads, n)) for p, n in zip(n_parents, spec.prompt_len)],
                                axis=1).astype(np.int32)
        slots = max(min(n, p * spec.reps_per_parent) for p, n in zip(n_parents, spec.prompt_len))
    else:
        slots = max(sum(min(spec.reps_per_parent, min(spec.parent_size, n - s))
                        for s in range(0, n, spec.parent_size)) for n in spec.prompt_len)
    if G * min(K, slots) > 1024:                                   # outside the library's limits
        K = spec.n_sample = max(1, 1024 // G)
    layer = _layer_from_labels(spec, data, labels, n_parents) if by_labels else pu.GpuLayer(spec, data)
    if by_labels:
        _check_records(layer, labels, n_parents)
    else:
        check_team_records(layer)
    step = int(rng.integers(0, 3))
    check_sparse_step(layer, step, K, seed=int(rng.integers(1 << 62)), stream_base=int(rng.integers(1 << 20)))
    check_dense_step(layer, step)


@pytest.mark.parametrize("case", range(40))
def test_random_batches_of_many_short_sequences(case):
    """Many (sequence, KV head) pairs per call: the read plans live in global memory and the rows of
    all pairs are cut into equal ranges, one per CTA, so CTAs cross pair boundaries all the time."""
    rng = np.random.default_rng(7000 + case)
    n_q, n_kv = _GROUPS[rng.integers(len(_GROUPS))]
    P, R = _PARENTS[rng.integers(len(_PARENTS))]
    n_seqs = int(rng.integers(8, 49))
    hi = int(rng.choice([6, 60, 400, 1500]))
    prompt = [int(rng.integers(1, hi + 1)) for _ in range(n_seqs)]
    cap = int(rng.choice([0, 3, 16]))
    spec = synth.WorkloadSpec("fuzz_many", n_seqs, n_q, n_kv, prompt, int(rng.integers(2, 20)), P, R,
                              int(rng.choice([1, 3, 8, 31, 64])), 2, max(cap, 1),
                              [int(rng.integers(0, cap + 1)) for _ in range(n_seqs)], 1, seed=int(rng.integers(1 << 30)))
    spec.elem = "fp16" if case % 2 else "bf16"
    G = n_q // n_kv
    slots = max(sum(min(R, min(P, n - s)) for s in range(0, n, P)) for n in prompt)
    K = spec.n_sample
    if G * min(K, slots) > 1024:
        K = spec.n_sample = max(1, 1024 // G)
    layer = pu.GpuLayer(spec, synth.make_layer(spec, layer=0))
    check_team_records(layer, seqs=[0, n_seqs - 1])
    check_sparse_step(layer, 1, K, seed=int(rng.integers(1 << 62)))
    check_dense_step(layer, 0)
