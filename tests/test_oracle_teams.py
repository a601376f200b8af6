"""Pins for the oracle's Algorithm 4 (contiguous parents) and Algorithm 2
(actual-key teams): hand-worked parents whose picks can be checked by eye,
the tie rules on exact ties and duplicate keys, and definitional properties
re-evaluated with numpy on random parents."""
import numpy as np
import pytest

from oracle import santapp_oracle as orc


def _teams(ts, tm):
    return [list(tm[ts[g]:ts[g + 1]]) for g in range(len(ts) - 1)]


def test_contiguous_parents_cover_prompt_in_order_with_short_tail():
    assert list(orc.contiguous_parents(10, 4)) == [0, 4, 8, 10]
    assert list(orc.contiguous_parents(8, 4)) == [0, 4, 8]
    assert list(orc.contiguous_parents(3, 4)) == [0, 3]
    assert list(orc.contiguous_parents(1, 1)) == [0, 1]


def test_line_example_worked_by_hand():
    """Keys 0, 1, 2, 10, 11, 20 on a line, one parent, R = 3.
    Mean 7.33 -> nearest actual key is 10 (token 3). Farthest from 10: 0 and 20
    tie at distance 10 -> smaller token index (token 0). Then 20 (token 5) is
    farthest from {10, 0}. Assignment: 1, 2 -> key 0; 11 -> key 10."""
    keys = np.array([[0.0], [1.0], [2.0], [10.0], [11.0], [20.0]])
    ts, tm, rep = orc.build_teams_contiguous(keys, P=6, R=3)
    assert list(rep) == [3, 0, 5]
    assert _teams(ts, tm) == [[3, 4], [0, 1, 2], [5]]


def test_assignment_tie_goes_to_earliest_selected_representative():
    """Token 1 at (2,1) is exactly 5 away (squared) from both representatives
    (0,0) [chosen first: nearest the mean (2/3, 0)] and (4,0) [chosen second:
    farthest from the first]; it must join the first one's team."""
    keys = np.array([[0, 0], [2, 1], [4, 0], [-1, 0], [-1, -0.5], [0, -0.5]], dtype=np.float64)
    ts, tm, rep = orc.build_teams_contiguous(keys, P=6, R=2)
    assert list(rep) == [0, 2]
    assert _teams(ts, tm) == [[0, 1, 3, 4, 5], [2]]


def test_duplicate_keys_self_ownership_keeps_every_team_nonempty():
    keys = np.full((4, 3), 7.0)
    ts, tm, rep = orc.build_teams_contiguous(keys, P=4, R=2)
    assert list(rep) == [0, 1]                 # ties resolved by increasing token index
    assert _teams(ts, tm) == [[0, 2, 3], [1]]  # all ties go to the first representative; token 1 owns itself


def test_parent_smaller_than_R_and_R_equals_P_make_singletons():
    rng = np.random.default_rng(0)
    keys = rng.standard_normal((7, 5))
    ts, tm, rep = orc.build_teams_contiguous(keys, P=4, R=4)
    assert len(rep) == 7 and np.all(np.diff(ts) == 1)
    assert sorted(tm) == list(range(7))
    assert list(tm) == list(rep)
    ts, tm, rep = orc.build_teams_contiguous(keys, P=5, R=3)    # short last parent of 2 rows: r = 2
    assert len(rep) == 3 + 2
    assert sorted(tm[ts[3]:]) == [5, 6]


def test_teams_emitted_parent_by_parent_members_ascending():
    rng = np.random.default_rng(1)
    keys = rng.standard_normal((40, 6))
    ts, tm, rep = orc.build_teams_contiguous(keys, P=16, R=4)
    assert len(rep) == 4 + 4 + 4
    for g, members in enumerate(_teams(ts, tm)):
        parent = g // 4
        assert members == sorted(members)
        assert all(parent * 16 <= i < min((parent + 1) * 16, 40) for i in members)
        assert rep[g] in members
    assert sorted(tm) == list(range(40))


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_definitional_properties_on_random_parents(seed):
    rng = np.random.default_rng(seed)
    N, d, P, R = 96, 8, 32, 6
    keys = rng.standard_normal((N, d)) + 3.0 * rng.integers(0, 3, size=(N, 1))
    ts, tm, rep = orc.build_teams_contiguous(keys, P=P, R=R)
    for p in range(N // P):
        C = np.arange(p * P, (p + 1) * P)
        reps = rep[p * R:(p + 1) * R]
        mu = keys[C].mean(0)
        d_mu = ((keys[C] - mu) ** 2).sum(1)
        assert reps[0] == C[np.argmin(d_mu)]
        for u in range(1, R):
            chosen = reps[:u]
            dmin = np.min(((keys[C][:, None, :] - keys[chosen][None, :, :]) ** 2).sum(2), axis=1)
            dmin[np.isin(C, chosen)] = -1.0
            assert reps[u] == C[np.argmax(dmin)]
        dist = ((keys[C][:, None, :] - keys[reps][None, :, :]) ** 2).sum(2)
        owner = np.argmin(dist, axis=1)
        for u in range(R):
            g = p * R + u
            members = set(tm[ts[g]:ts[g + 1]])
            assert members == set(C[owner == u])
