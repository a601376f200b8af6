"""Pins for the oracle's Algorithm 3 steps (centre count and nearest-centre partition)."""
import itertools

import numpy as np
import pytest
from scipy.cluster.vq import vq

from oracle import santapp_oracle as orc


@pytest.mark.parametrize("N,P,want", [
    (32768, 512, 64),      # floor(N / P)
    (32768, 16, 2048),
    (1000, 16, 62),        # floor, not ceiling
    (20, 16, 2),           # at least two centres
    (3, 16, 2),
    (2, 512, 2),
    (5, 1, 5),             # never more centres than keys
    (7, 2, 3),
])
def test_parent_count_closed_forms(N, P, want):
    assert orc.kmeans_parent_count(N, P) == want


def test_partition_matches_library_vector_quantiser():
    rng = np.random.default_rng(11)
    keys = rng.standard_normal((700, 24))
    centres = rng.standard_normal((37, 24))
    label, ps, pm = orc.nearest_centre_parents(keys, centres)
    code, _ = vq(keys, centres)
    assert np.array_equal(label, code)
    kept = np.unique(code)
    assert ps.shape[0] - 1 == kept.shape[0]
    for u, c in enumerate(kept):
        assert np.array_equal(pm[ps[u]:ps[u + 1]], np.flatnonzero(code == c))
    assert ps[-1] == 700


def test_ties_go_to_smaller_centre_and_empty_parents_are_dropped():
    # keys on a line; centres 0 and 2 are the same point, centre 1 is far away and attracts nothing
    keys = np.array([[0.0], [1.0], [2.0], [3.0]])
    centres = np.array([[1.0], [50.0], [1.0], [3.0]])
    label, ps, pm = orc.nearest_centre_parents(keys, centres)
    # token 2 is equidistant from centres 0/2 (distance 1) and 3 (distance 1): smallest index wins
    assert label.tolist() == [0, 0, 0, 3]
    assert ps.tolist() == [0, 3, 4]
    assert pm.tolist() == [0, 1, 2, 3]


def test_partition_minimises_inertia_by_brute_force():
    rng = np.random.default_rng(5)
    keys = rng.standard_normal((6, 3))
    centres = rng.standard_normal((3, 3))
    label, _, _ = orc.nearest_centre_parents(keys, centres)

    def inertia(lab):
        return sum(float(np.sum((keys[i] - centres[u]) ** 2)) for i, u in enumerate(lab))
    best = min(itertools.product(range(3), repeat=6), key=inertia)
    assert inertia(label) <= inertia(best) + 1e-12
    assert list(best) == label.tolist()


def test_members_partition_all_tokens_in_increasing_order():
    rng = np.random.default_rng(2)
    keys = rng.standard_normal((300, 8))
    centres = rng.standard_normal((40, 8)) * 3.0          # spread out: several centres stay empty
    label, ps, pm = orc.nearest_centre_parents(keys, centres)
    assert sorted(pm.tolist()) == list(range(300))
    assert ps.shape[0] - 1 == np.unique(label).shape[0] < 40
    for u in range(ps.shape[0] - 1):
        seg = pm[ps[u]:ps[u + 1]]
        assert seg.shape[0] > 0 and np.all(np.diff(seg) > 0) and np.unique(label[seg]).shape[0] == 1
    firsts = [label[pm[ps[u]]] for u in range(ps.shape[0] - 1)]
    assert firsts == sorted(firsts)


def test_teams_from_centre_parents_partition_the_prompt():
    rng = np.random.default_rng(3)
    keys = rng.standard_normal((257, 16))
    centres = rng.standard_normal((9, 16))
    _, ps, pm = orc.nearest_centre_parents(keys, centres)
    ts, tm, rep = orc.build_teams(keys, ps, pm, 4)
    M = ts.shape[0] - 1
    sizes = np.diff(ps)
    assert M == int(np.minimum(sizes, 4).sum())
    assert sorted(tm.tolist()) == list(range(257))
    for g in range(M):
        assert rep[g] in tm[ts[g]:ts[g + 1]]
