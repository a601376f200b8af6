"""The workspace-free dense entry point against the regular one.

santapp_dense_decode_attn_noalloc is for callers that cannot get device memory at the point of
the call (all of it already belongs to someone else's pool, or allocation calls are forbidden
or too disruptive where they run), so its scratch is a fixed array inside the library. This
test calls it through the C ABI twice in a row, on two different inputs, and checks each
result against santapp_dense_decode_attn on the same inputs and against the fp64 oracle, within
the dense tolerance of the parity tests. Two calls matter because the second one finds the array
as the first left it. One case has few (sequence, KV head) pairs (the plan is set up inside the
attention kernel), the other many (plan tables and row prefixes live in the array). The file
sorts last so that a failure here cannot hide any other test's result.
"""
import numpy as np
import pytest
import torch

from paper_2609_35629_b200 import binding as sp
from paper_2609_35629_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu

DENSE_TOL = 1e-3


def _two_calls_in_a_row(spec, suffixes):
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    vmax = pu.max_abs_v(layer)
    out = torch.empty((spec.n_seqs, spec.n_q_heads, spec.head_dim), dtype=torch.float32, device="cuda")
    for step, suffix in enumerate(suffixes):
        q_bits = synth.make_queries(spec, layer.data, step)
        q = sp.bf16_bits_to_cuda(q_bits)
        sl = torch.tensor(suffix, dtype=torch.int32, device="cuda")
        expect = sp.santapp_dense_decode_attn(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix, sl)
        torch.cuda.synchronize()
        got = sp.santapp_dense_decode_attn_noalloc(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix, sl,
                                                   out=out)
        torch.cuda.synchronize()
        assert got.data_ptr() == out.data_ptr()
        err = float((got - expect).abs().max())
        assert np.isfinite(err) and err <= DENSE_TOL * vmax, f"step {step}: max |delta| {err}"
        ref = pu.oracle_step(layer, q_bits, suffix, 0, 0, step, dense=True)
        for b, o in ref.items():
            err = float(np.abs(got[b].cpu().numpy() - o).max())
            assert err <= DENSE_TOL * vmax, f"step {step}, sequence {b}: max |delta| against the oracle {err}"


def test_noalloc_dense_matches_regular_dense_on_two_calls_in_a_row():
    spec = synth.spec_small_gqa(seed=3)
    _two_calls_in_a_row(spec, ([5, 0], [spec.suffix_cap, 7]))


def test_noalloc_dense_with_plans_in_the_array_on_two_calls_in_a_row():
    """Six sequences of different lengths are 24 pairs: more than the attention kernel sets up by
    itself, so the plan tables, the pairs' row prefix and the partials all live in the array,
    and the second call finds what the first left there."""
    spec = synth.spec_small_gqa(seed=4, n_seqs=6, prompt=(700, 300, 1536, 64, 1000, 420), parent_size=64, reps=8,
                                suffix0=(3, 0, 9, 1, 0, 30))
    assert sp.santapp_dense_workspace_bytes(pu.geometry(spec), pu.GpuLayer(spec, synth.make_layer(spec)).teams) \
        <= sp.SANTAPP_STATIC_SCRATCH_BYTES
    _two_calls_in_a_row(spec, ([3, 0, 9, 1, 0, 30], [0, 32, 1, 2, 17, 5]))


def test_noalloc_rejects_problems_beyond_the_built_in_scratch():
    """A batch whose workspace need exceeds the array is refused on the host with its own
    status and a message that names both sizes, before anything is launched."""
    spec = synth.spec_small_gqa(seed=3)
    layer = pu.GpuLayer(spec, synth.make_layer(spec))
    big = sp.Geometry(115, 28, 4, 128, spec.parent_size, spec.reps_per_parent)      # 460 pairs
    assert sp.santapp_dense_workspace_bytes(big, layer.teams) > sp.SANTAPP_STATIC_SCRATCH_BYTES
    q = torch.zeros((115, 28, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sp.SantappError) as e:
        sp.santapp_dense_decode_attn_noalloc(big, layer.teams, q, None, None, None)
    assert e.value.status == sp.SANTAPP_ERR_STATIC_SCRATCH
    assert "needs" in str(e.value)
