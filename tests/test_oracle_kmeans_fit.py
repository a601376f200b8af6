"""Pins for the oracle's minibatch k-means fit (Algorithm 3, second line)."""
import numpy as np
import pytest

from oracle import santapp_oracle as orc


def _blobs(rng, n, k, d, spread=5.0, sigma=0.3):
    true = rng.standard_normal((k, d)) * spread
    lab = rng.integers(0, k, size=n)
    return true[lab] + sigma * rng.standard_normal((n, d)), true, lab


def _inertia(x, c):
    return float(((x[:, None, :] - c[None]) ** 2).sum(-1).min(1).sum())


def test_separated_blobs_are_recovered():
    rng = np.random.default_rng(0)
    x, true, lab = _blobs(rng, 3000, 8, 16)
    c, steps = orc.minibatch_kmeans(x, 8, batch=256)
    d2 = ((c[:, None, :] - true[None]) ** 2).sum(-1)
    assert sorted(d2.argmin(1).tolist()) == list(range(8))            # one centre per blob
    assert d2.min(1).max() < 0.02                                      # ~ sigma^2 d / points seen
    got, _, _ = orc.nearest_centre_parents(x, c)
    relabel = d2.argmin(1)
    assert np.array_equal(relabel[got], lab)
    assert 10 <= steps <= 100 * 12


def test_quality_matches_a_library_fit_with_the_same_settings():
    sk = pytest.importorskip("sklearn.cluster")
    rng = np.random.default_rng(1)
    x, _, _ = _blobs(rng, 4000, 24, 32, spread=1.0, sigma=0.6)        # overlapping clusters
    c, _ = orc.minibatch_kmeans(x, 24, batch=512)
    ref = sk.MiniBatchKMeans(n_clusters=24, batch_size=512, max_iter=100, max_no_improvement=10,
                             reassignment_ratio=0.01, n_init=1, tol=0.0, random_state=0).fit(x)
    lloyd = sk.KMeans(n_clusters=24, n_init=5, random_state=0).fit(x)      # full-batch reference optimum
    ours, theirs, floor = _inertia(x, c), _inertia(x, ref.cluster_centers_), _inertia(x, lloyd.cluster_centers_)
    assert ours <= 1.1 * theirs                                        # no worse than the library's minibatch fit
    assert ours >= 0.98 * floor                                        # and not implausibly good


def test_every_point_its_own_centre_when_k_equals_n():
    """k = N with distinct integer points: the start picks every point once (a chosen point has
    zero weight), and a centre that only ever receives copies of itself does not move."""
    rng = np.random.default_rng(2)
    x = rng.permutation(40)[:, None] * np.array([[1.0, 3.0, -2.0]])
    c, _ = orc.minibatch_kmeans(x, 40, batch=16, max_iter=5, ratio=0.0)
    assert sorted(map(tuple, c.tolist())) == sorted(map(tuple, x.tolist()))


def test_single_centre_is_the_mean_of_everything_sampled():
    """k = 1 isolates the cumulative-count update and the index draw: the centre must equal the
    mean of all points drawn so far, the draws recomputed here from the pinned Philox words."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal((500, 4))
    batch, seed, stream = 64, 77, 5
    c, steps = orc.minibatch_kmeans(x, 1, batch=batch, max_iter=1, patience=10 ** 6, ratio=0.0, seed=seed, stream=stream)
    assert steps == 8                                                  # max_iter * ceil(500 / 64)
    drawn = []
    for t in range(steps):
        for s in range(batch):
            w = orc.philox4x32_10([s, 3, stream, t], [seed, 0])[0]
            drawn.append((int(w) * 500) >> 32)
    assert np.allclose(c[0], x[drawn].mean(axis=0), rtol=0, atol=1e-12)


def test_stopping_rule_and_step_limit():
    rng = np.random.default_rng(4)
    x, _, _ = _blobs(rng, 2000, 6, 8)
    _, s1 = orc.minibatch_kmeans(x, 6, batch=128, patience=1)
    _, s10 = orc.minibatch_kmeans(x, 6, batch=128, patience=10)
    _, capped = orc.minibatch_kmeans(x, 6, batch=128, max_iter=1, patience=10 ** 6)
    assert 2 <= s1 < s10
    assert capped == 16                                                # ceil(2000 / 128)


def test_same_arguments_same_centres_other_seed_or_stream_other_centres():
    rng = np.random.default_rng(5)
    x, _, _ = _blobs(rng, 1500, 5, 8, spread=1.0, sigma=0.8)
    a, _ = orc.minibatch_kmeans(x, 5, batch=128, seed=9, stream=2)
    b, _ = orc.minibatch_kmeans(x, 5, batch=128, seed=9, stream=2)
    c, _ = orc.minibatch_kmeans(x, 5, batch=128, seed=10, stream=2)
    d, _ = orc.minibatch_kmeans(x, 5, batch=128, seed=9, stream=3)
    assert np.array_equal(a, b)
    assert not np.array_equal(a, c) and not np.array_equal(a, d)


def test_a_starved_centre_is_moved_back_into_the_data():
    """A single far outlier is an attractive k-means++ pick but almost never drawn afterwards, so its
    count stays far below 1 % of the largest: with the reassignment ratio on, that centre is moved
    onto a minibatch point; with the ratio off it stays on the outlier."""
    rng = np.random.default_rng(6)
    x, _, _ = _blobs(rng, 6000, 3, 8, spread=2.0, sigma=0.5)
    x[123] = 400.0
    # batch 2048: the initialisation sample (3 * batch, capped at N) is the whole set, outlier included
    kept, _ = orc.minibatch_kmeans(x, 4, batch=2048, ratio=0.0, patience=40)
    moved, _ = orc.minibatch_kmeans(x, 4, batch=2048, ratio=0.01, patience=40)
    near = lambda c: float(np.abs(c - x[123]).max(axis=1).min())
    assert near(kept) < 1e-9
    assert near(moved) > 100.0
    inliers = np.delete(x, 123, axis=0)
    assert np.all(moved >= inliers.min(axis=0) - 1e-9) and np.all(moved <= inliers.max(axis=0) + 1e-9)
