"""Pins for the oracle's centroid-guided grouping (one group per contiguous parent, routed by the
arithmetic mean of its keys, stored as a bf16 value)."""
import numpy as np

from oracle import santapp_oracle as orc
from paper_2609_35629_b200 import synth


def test_hand_worked_parents():
    k = np.arange(24, dtype=np.float64).reshape(6, 4)                # rows 0..5, parents of 4: {0..3}, {4, 5}
    ts, tm, mean = orc.group_mean_keys(k, 4)
    assert ts.tolist() == [0, 4, 6] and tm.tolist() == list(range(6))
    assert np.array_equal(mean, np.array([[6., 7., 8., 9.], [18., 19., 20., 21.]]))


def test_groups_of_one_key_are_the_keys():
    """P = 1: the mean of a single bf16 key is the key itself, so the variant coincides with
    every-key-its-own-team routing (the SANTA limit) and its routing KL is zero."""
    rng = np.random.default_rng(0)
    k = synth.bf16_to_f64(synth.f32_to_bf16_bits(rng.normal(size=(50, 16)).astype(np.float32)))
    ts, tm, mean = orc.group_mean_keys(k, 1)
    assert np.array_equal(mean, k) and ts.tolist() == list(range(51))
    q = rng.normal(size=16)
    assert abs(orc.routing_kl(q, k, ts, tm, mean, 0.25)) < 1e-12


def test_mean_is_rounded_to_a_bf16_value_to_nearest():
    rng = np.random.default_rng(1)
    k = synth.bf16_to_f64(synth.f32_to_bf16_bits(rng.normal(size=(37, 8)).astype(np.float32)))
    P = 10
    ts, tm, mean = orc.group_mean_keys(k, P)
    assert ts.tolist() == [0, 10, 20, 30, 37]
    for u in range(4):
        exact = k[ts[u]:ts[u + 1]].mean(axis=0)
        # a bf16 value: its float32 bit pattern has a zero low half
        bits = mean[u].astype(np.float32).view(np.uint32)
        assert np.all(bits & 0xFFFF == 0) and np.array_equal(mean[u].astype(np.float32).astype(np.float64), mean[u])
        # nearest: within half a unit in the last place (8 significant bits) of the exact mean
        assert np.all(np.abs(mean[u] - exact) <= 2.0 ** -8 * np.abs(exact) + 1e-300)
        # and equal to the independent rounding helper of the input generators
        want = synth.bf16_to_f64(synth.f32_to_bf16_bits(exact.astype(np.float32)))
        assert np.array_equal(mean[u], want)


def test_decode_with_mean_keys_keeps_the_dense_limit():
    """Algorithm 1 does not care what the routing key is: with K >= M it still returns dense attention."""
    rng = np.random.default_rng(2)
    k = synth.bf16_to_f64(synth.f32_to_bf16_bits(rng.normal(size=(64, 16)).astype(np.float32)))
    v = rng.normal(size=(64, 16))
    q = rng.normal(size=16)
    ts, tm, mean = orc.group_mean_keys(k, 8)
    r = orc.decode_head_given_gumbel(q, k, v, ts, tm, mean, None, None, 8, None, 0.25)
    assert np.allclose(r.o, orc.dense_head(q, k, v, 0.25), rtol=0, atol=1e-12)


def test_arbitrary_partition_reduces_to_the_contiguous_one():
    """On the contiguous partition the general routine must give the contiguous routine's keys."""
    rng = np.random.default_rng(3)
    k = synth.bf16_to_f64(synth.f32_to_bf16_bits(rng.normal(size=(45, 8)).astype(np.float32)))
    ts, tm, mean = orc.group_mean_keys(k, 7)
    ts2, tm2, mean2 = orc.group_mean_keys_parents(k, ts, tm)
    assert np.array_equal(ts, ts2) and np.array_equal(tm, tm2) and np.array_equal(mean, mean2)


def test_arbitrary_partition_hand_worked_and_rounded():
    k = np.array([[1.0, 10.0], [2.0, 20.0], [4.0, 40.0], [8.0, 80.0], [16.0, 160.0]])
    ps = np.array([0, 2, 5], dtype=np.int32)
    pm = np.array([4, 0, 1, 2, 3], dtype=np.int32)                 # parents {4, 0} and {1, 2, 3}
    _, _, mean = orc.group_mean_keys_parents(k, ps, pm)
    # (16 + 1) / 2 = 8.5 and (160 + 10) / 2 = 85 are bf16 values; (2 + 4 + 8) / 3 = 4.666..., (20 + 40 + 80) / 3 = 46.66...
    assert np.array_equal(mean[0], [8.5, 85.0])
    want = synth.bf16_to_f64(synth.f32_to_bf16_bits(np.array([14.0 / 3.0, 140.0 / 3.0], dtype=np.float32)))
    assert np.array_equal(mean[1], want)
    assert mean[1, 0] == 4.65625 and mean[1, 1] == 46.75           # nearest bf16 values, by hand


def test_rounding_to_fp16_matches_the_library_conversion():
    """fp64 -> fp32 -> binary16 against numpy's conversions on random values of every magnitude,
    exact ties, subnormals, the overflow threshold, signed zeros and infinities."""
    rng = np.random.default_rng(9)
    xs = np.concatenate([
        rng.standard_normal(4000) * np.exp(rng.uniform(-20, 12, size=4000)),
        np.array([0.0, -0.0, 1.0, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 2.0 ** -14, 2.0 ** -24, 2.0 ** -25,
                  1.5 * 2.0 ** -25, 2.0 ** -26, 65504.0, 65519.99, 65520.0, 70000.0, -65520.0, np.inf, -np.inf,
                  6.1e-5, 5.97e-8, 3.0e-8, 2.98e-8]),
    ])
    with np.errstate(over="ignore"):
        want = xs.astype(np.float32).astype(np.float16).astype(np.float64)
    got = np.array([orc.round_to_elem(x, "fp16") for x in xs])
    assert np.array_equal(got, want)
    assert np.array_equal(np.signbit(got), np.signbit(want))
    # and bf16 against the generators' helper
    want_b = synth.bf16_to_f64(synth.f32_to_bf16_bits(xs[np.isfinite(xs)].astype(np.float32)))
    got_b = np.array([orc.round_to_elem(x, "bf16") for x in xs[np.isfinite(xs)]])
    assert np.array_equal(got_b, want_b)


def test_fp16_mean_keys():
    rng = np.random.default_rng(10)
    k = synth.to_f64(synth.round_bits(rng.normal(size=(30, 8)).astype(np.float32), "fp16"), "fp16")
    ts, _, mean = orc.group_mean_keys(k, 7, elem="fp16")
    for u in range(len(ts) - 1):
        exact = k[ts[u]:ts[u + 1]].mean(axis=0)
        assert np.array_equal(mean[u], exact.astype(np.float32).astype(np.float16).astype(np.float64))
    _, _, mean2 = orc.group_mean_keys_parents(k, ts, np.arange(30, dtype=np.int32), elem="fp16")
    assert np.array_equal(mean, mean2)
