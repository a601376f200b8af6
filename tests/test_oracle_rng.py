"""Pins for the oracle's random stream (Philox4x32-10 -> open uniform -> Gumbel).

The paper asks only for independent Gumbel(0,1) draws with CDF exp(-exp(-x))
("Conditional inclusion correction" paragraph of the algorithm appendix); the
counter-based generator is this build's reading. Pins: an independent library
implementation of the same generator (cuRAND's host generator, which needs no
GPU), avalanche behaviour on the counter words the library cannot reach, and
the Gumbel law itself.
"""
import ctypes
import math

import numpy as np
import pytest

from oracle import santapp_oracle as orc


def _curand():
    for name in ("libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so.10", "libcurand.so"):
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    return None


def _curand_words(lib, seed, n_words, offset_words):
    gen = ctypes.c_void_p()
    CURAND_RNG_PSEUDO_PHILOX4_32_10 = 161
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), CURAND_RNG_PSEUDO_PHILOX4_32_10) == 0
    try:
        assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
        assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(offset_words)) == 0
        out = np.zeros(n_words, dtype=np.uint32)
        assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(n_words)) == 0
    finally:
        lib.curandDestroyGenerator(gen)
    return out


@pytest.mark.parametrize("seed", [0, 1, 0x123456789ABCDEF0, 0xFFFFFFFFFFFFFFFF])
@pytest.mark.parametrize("block0", [0, 1, 4095, 65533, 0xFFFFFFFE, (1 << 32) + 7, (5 << 40) + 0xFFFA])
def test_philox_words_match_curand_host_generator(seed, block0):
    """cuRAND's host Philox4_32_10 generator emits, as its i-th group of four
    words, the block for counter (i div 65536, 0, i mod 65536, 0) under key =
    (seed low, seed high): 65536 interleaved subsequences. The oracle's own
    implementation must give the same integers."""
    lib = _curand()
    if lib is None:
        pytest.skip("libcurand not loadable")
    n_blocks = 8
    words = _curand_words(lib, seed, 4 * n_blocks, 4 * block0)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for i in range(n_blocks):
        blk = block0 + i
        mine = orc.philox4x32_10([blk >> 16, 0, blk & 0xFFFF, 0], key)
        assert [int(x) for x in mine] == [int(x) for x in words[4 * i:4 * i + 4]]


def _popcount(x):
    return bin(int(x)).count("1")


@pytest.mark.parametrize("word", [0, 1, 2, 3])
def test_philox_avalanche_on_every_counter_word(word):
    """A block cipher-like bijection: flipping any single counter bit must flip
    about half of the 128 output bits. Catches a counter word that is ignored
    or wired to the wrong lane (the library pin above only varies words 0 and 2)."""
    rng = np.random.default_rng(7)
    flips = []
    for _ in range(200):
        ctr = [int(v) for v in rng.integers(0, 1 << 32, size=4)]
        key = [int(v) for v in rng.integers(0, 1 << 32, size=2)]
        bit = int(rng.integers(0, 32))
        a = orc.philox4x32_10(ctr, key)
        ctr2 = list(ctr)
        ctr2[word] ^= 1 << bit
        b = orc.philox4x32_10(ctr2, key)
        flips.append(sum(_popcount(x ^ y) for x, y in zip(a, b)))
    mean = np.mean(flips)
    assert 60.0 < mean < 68.0          # 64 +- 4.5 * sqrt(32 / 200)
    assert min(flips) > 30


def test_philox_is_injective_on_consecutive_counters():
    key = [3, 4]
    seen = set()
    for c0 in range(2048):
        seen.add(tuple(int(x) for x in orc.philox4x32_10([c0, 5, 6, 7], key)))
    assert len(seen) == 2048


def test_team_word_counter_layout():
    """Team g uses word g mod 4 of the block with counter (g div 4, step, head,
    stream) and key = seed halves."""
    seed, step, head, stream = 0xA5A5A5A512345678, 17, 23, 9
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for g in [0, 1, 2, 3, 4, 5, 2047, 8191, 100003]:
        blk = orc.philox4x32_10([g >> 2, step, head, stream], key)
        assert orc.team_word(seed, step, head, stream, g) == int(blk[g & 3])


def test_uniform_open_is_cell_centre():
    assert orc.uniform_open(0) == 2.0 ** -33
    assert orc.uniform_open(0xFFFFFFFF) == 1.0 - 2.0 ** -33
    assert orc.uniform_open(0x80000000) == 0.5 + 2.0 ** -33
    assert 0.0 < orc.uniform_open(0) < orc.uniform_open(1) < 1.0


def test_gumbel_extremes_are_finite_and_bounded():
    """The 32-bit grid bounds the draw: G <= -log(-log(1 - 2^-33)) ~ 22.87 and
    G >= -log(33 log 2) ~ -3.13, so a selected team's correction can never
    underflow to zero."""
    hi = orc.gumbel(0xFFFFFFFF)
    lo = orc.gumbel(0)
    assert abs(hi - 33.0 * math.log(2.0)) < 1e-6       # -log(-log(1-e)) ~ -log(e) for tiny e
    assert abs(lo + math.log(33.0 * math.log(2.0))) < 1e-12
    assert orc.gumbel(0x80000000) == pytest.approx(-math.log(-math.log(0.5 + 2.0 ** -33)), abs=1e-15)


def test_gumbel_law_ks_and_moments():
    """10^6 draws from the keyed stream against the CDF exp(-exp(-x)); mean is
    the Euler-Mascheroni constant, variance pi^2 / 6."""
    n = 1_000_000
    g = np.concatenate([orc.gumbel_many(12345, step, 3, 1, n // 4) for step in range(4)])
    g.sort()
    cdf = np.exp(-np.exp(-g))
    i = np.arange(1, n + 1)
    ks = max(np.max(i / n - cdf), np.max(cdf - (i - 1) / n))
    assert ks < 1.95 / math.sqrt(n)                     # ~0.1 % critical value
    assert abs(g.mean() - 0.5772156649015329) < 4.5 * math.sqrt(math.pi ** 2 / 6 / n)
    # var of sample variance for Gumbel: (mu4 - sigma^4)/n with excess kurtosis 2.4
    sigma2 = math.pi ** 2 / 6
    assert abs(g.var() - sigma2) < 4.5 * sigma2 * math.sqrt((2.0 + 2.4) / n)


def test_streams_are_distinct_across_head_step_stream_seed():
    base = orc.gumbel_many(1, 2, 3, 4, 256)
    for args in [(2, 2, 3, 4), (1, 3, 3, 4), (1, 2, 4, 4), (1, 2, 3, 5)]:
        other = orc.gumbel_many(*args, 256)
        assert np.sum(base == other) <= 1
        assert abs(np.corrcoef(base, other)[0, 1]) < 0.3
    assert np.array_equal(base, orc.gumbel_many(1, 2, 3, 4, 256))
