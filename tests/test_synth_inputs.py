"""The seeded input generators (no method arithmetic): determinism, the two key layouts, the bf16
helpers and the suffix schedule."""
import dataclasses

import numpy as np

from paper_2609_35629_b200 import synth


def test_layers_are_reproducible_and_seeded():
    spec = synth.spec_small_gqa()
    a, b = synth.make_layer(spec, layer=1), synth.make_layer(spec, layer=1)
    assert np.array_equal(a.k_prompt, b.k_prompt) and np.array_equal(a.v_suffix, b.v_suffix)
    c = synth.make_layer(spec, layer=2)
    assert not np.array_equal(a.k_prompt, c.k_prompt)
    d = synth.make_layer(synth.spec_small_gqa(seed=1), layer=1)
    assert not np.array_equal(a.k_prompt, d.k_prompt)
    q0, q1 = synth.make_queries(spec, a, 0), synth.make_queries(spec, a, 1)
    assert np.array_equal(q0, synth.make_queries(spec, a, 0)) and not np.array_equal(q0, q1)


def test_bf16_helpers_round_to_nearest_even_and_widen_exactly():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0, 3.0e38], dtype=np.float32)
    bits = synth.f32_to_bf16_bits(x)
    back = synth.bf16_to_f32(bits)
    assert back[0] == 1.0 and back[1] == 1.0                       # tie to even (down)
    assert back[2] == np.float32(1.0 + 2.0 ** -6)                  # tie to even (up)
    assert back[3] == -2.5 and back[4] == 0.0
    assert np.array_equal(synth.bf16_to_f64(bits), back.astype(np.float64))
    assert np.array_equal(synth.f32_to_bf16_bits(back), bits)      # idempotent


def _run_lengths(which):
    edges = np.flatnonzero(np.diff(which) != 0)
    return np.diff(np.concatenate([[-1], edges, [len(which) - 1]]))


def test_key_layouts():
    """"iid": every row draws its cluster independently; "runs": geometric runs of one cluster
    with mean length rows / clusters. Recover the cluster of each row by nearest centre."""
    base = synth.spec_small_gqa(n_seqs=1, prompt=(4096,), suffix0=(0,))
    for layout, lo, hi in (("iid", 1.0, 1.1), ("runs", 0.6 * 4096 / 32, 1.6 * 4096 / 32)):
        spec = dataclasses.replace(base, key_layout=layout)
        data = synth.make_layer(spec, keep_centres=True)
        k = synth.bf16_to_f32(data.k_prompt[0])[4:]                # skip the scaled sink rows
        c = data.centres[0]
        d2 = (k * k).sum(1)[:, None] - 2.0 * k @ c.T + (c * c).sum(1)[None, :]
        which = d2.argmin(1)
        mean_run = _run_lengths(which).mean()
        assert lo <= mean_run <= hi, (layout, mean_run)
    # the default layout is the independent one, and its data do not depend on the new field
    assert base.key_layout == "iid"


def test_suffix_schedule():
    spec = synth.spec_qwen_b1()
    assert spec.suffix_len(0)[0] == 1 and spec.suffix_len(10)[0] == 11
    assert spec.suffix_len(10_000)[0] == spec.suffix_cap            # clamps at the capacity
    assert synth.spec_paper_point().suffix_len(5)[0] == 0


def test_fp16_rounding_and_widening_are_exact_inverses_on_representable_values():
    import numpy as np
    from paper_2609_35629_b200 import synth
    rng = np.random.default_rng(0)
    x = rng.standard_normal(1000).astype(np.float32) * 3
    bits = synth.round_bits(x, "fp16")
    assert bits.dtype == np.uint16
    back = synth.to_f64(bits, "fp16")
    assert np.array_equal(back, x.astype(np.float16).astype(np.float64))        # numpy's round-to-nearest-even
    assert np.array_equal(synth.round_bits(back.astype(np.float32), "fp16"), bits)
    assert np.max(np.abs(back - x)) <= 2.0 ** -11 * np.max(np.abs(x)) + 1e-12      # 11 significant bits
    # bf16 stays the default and differs
    assert np.array_equal(synth.round_bits(x), synth.f32_to_bf16_bits(x))
    assert not np.array_equal(synth.round_bits(x), bits)


def test_spec_element_type_reaches_every_tensor():
    import numpy as np
    from paper_2609_35629_b200 import synth
    a = synth.spec_small_gqa()
    b = synth.spec_small_gqa()
    b.elem = "fp16"
    da, db = synth.make_layer(a), synth.make_layer(b)
    for name in ("k_prompt", "v_prompt", "k_suffix", "v_suffix"):
        xa, xb = synth.to_f64(getattr(da, name), "bf16"), synth.to_f64(getattr(db, name), "fp16")
        assert not np.array_equal(getattr(da, name), getattr(db, name))
        assert np.max(np.abs(xa - xb)) < 0.05                                   # same draws, other rounding
    qa, qb = synth.make_queries(a, da, 0), synth.make_queries(b, db, 0)
    assert qa.shape == qb.shape and not np.array_equal(qa, qb)


def test_shared_latent_inputs_are_seeded_and_shaped():
    spec = synth.LatentSpec("t", [100, 37], suffix_cap=5, suffix_len0=[0, 4])
    a, b = synth.make_latent_layer(spec), synth.make_latent_layer(spec)
    assert a.rows.shape == (137, synth.LATENT_ROW) and a.rows.dtype == np.uint16
    assert a.suffix.shape == (2, 5, synth.LATENT_ROW)
    assert np.array_equal(a.rows, b.rows) and np.array_equal(a.suffix, b.suffix)
    assert not np.array_equal(a.rows, synth.make_latent_layer(spec, layer=1).rows)
    q0, q1 = synth.make_latent_queries(spec, a, 0), synth.make_latent_queries(spec, a, 1)
    assert q0.shape == (2, 16, synth.LATENT_ROW) and not np.array_equal(q0, q1)
    assert np.array_equal(q0, synth.make_latent_queries(spec, b, 0))
    assert list(spec.suffix_len(3)) == [3, 5]
    # the scale is handed to the C ABI as a float: it must survive that conversion unchanged
    assert float(np.float32(synth.LATENT_SCALE)) == synth.LATENT_SCALE
    # sinks: the first four rows are four times larger
    x = synth.to_f32(a.rows)
    assert np.abs(x[:4]).mean() > 3.0 * np.abs(x[4:100]).mean()
