"""Step-by-step pins for the oracle's minibatch k-means fit (Algorithm 3, the fit).

The paper fixes the routine's settings and leaves its details to "the implementation default"; the
reading taken is stated above `orc_minibatch_kmeans`. Each test here makes ONE step of that reading
observable on a small case with integer coordinates (every sum is exact in fp64) and predicts the
outcome from the stated rule and the pinned Philox words alone, never from the function:

  greedy start      which of the L trial points becomes the next centre (the best, not the first,
                    not the worst), and that L = 2 + floor(ln k) trials are drawn
  averaging weight  the step at which a k = 1 fit stops under alpha = min(1, 2 batch / (N + 1))
  reassignment      when it happens (period 10 + floor(smallest count)), where the centre lands
                    (a point of that minibatch chosen by the tag-4 words), how many centres may move
                    (batch / 2), and the count a moved centre takes (the smallest count that stays)

Every test also checks that the obvious alternative reading would have given a different outcome on
its inputs, so that a mistake in that step cannot pass.
"""
import math

import numpy as np

from oracle import santapp_oracle as orc


# ------------------------------------------------------------------------------------------------
# the pinned random words (Philox4x32-10 is pinned in test_oracle_rng.py) and what the reading
# derives from them
# ------------------------------------------------------------------------------------------------
def word(seed, slot, tag, stream, step):
    return int(orc.philox4x32_10([slot, tag, stream, step], [seed & 0xFFFFFFFF, seed >> 32])[0])


def index(w, n):
    return (w * n) >> 32


def sample_order(seed, stream, N, n_init):
    """Head of the Fisher-Yates shuffle of 0..N-1 (tag 1)."""
    perm = list(range(N))
    for i in range(n_init):
        r = i + index(word(seed, i, 1, stream, 0), N - i)
        perm[i], perm[r] = perm[r], perm[i]
    return perm[:n_init]


def minibatch(seed, stream, t, batch, N):
    return [index(word(seed, s, 3, stream, t), N) for s in range(batch)]


def greedy_start(x, k, batch, seed, stream, trials=None, choose="best"):
    """Greedy k-means++ on 1-D integer points, written from the reading: returns the k start centres
    (values) and, per centre after the first, the index of the winning trial."""
    N = len(x)
    n_init = min(N, max(3 * batch, 3 * k))
    sample = np.array([x[i] for i in sample_order(seed, stream, N, n_init)], dtype=np.float64)
    L = (2 + int(math.floor(math.log(k)))) if trials is None else trials
    centres = [sample[index(word(seed, 0, 2, stream, 0), n_init)]]
    closest = (sample - centres[0]) ** 2
    winners = []
    for c in range(1, k):
        total = closest.sum()
        cum = np.cumsum(closest)
        picks = []
        for l in range(L):
            u = (word(seed, l, 2, stream, c) + 0.5) / 2.0 ** 32
            above = np.nonzero(cum > u * total)[0]
            picks.append(int(above[0]) if len(above) else n_init - 1)
        pots = [np.minimum(closest, (sample - sample[p]) ** 2).sum() for p in picks]
        if choose == "best":
            win = int(np.argmin(pots))                      # ties to the earlier trial
        elif choose == "worst":
            win = int(np.argmax(pots))
        else:
            win = 0
        winners.append(win)
        centres.append(sample[picks[win]])
        closest = np.minimum(closest, (sample - sample[picks[win]]) ** 2)
    return np.array(centres), winners


def one_step_from(x, centres, seed, stream, batch):
    """Centres after the first minibatch step (all counts are zero before it, so a centre that
    receives points becomes their mean and one that receives none stays)."""
    pts = np.array([x[i] for i in minibatch(seed, stream, 0, batch, len(x))], dtype=np.float64)
    lab = np.abs(pts[:, None] - centres[None, :]).argmin(axis=1)          # ties to the smaller index
    out = centres.copy()
    for u in range(len(centres)):
        if np.any(lab == u):
            out[u] = pts[lab == u].sum() / np.count_nonzero(lab == u)
    return out


def fit_1d(x, k, **kw):
    c, steps = orc.minibatch_kmeans(np.asarray(x, dtype=np.float64)[:, None], k, **kw)
    return c[:, 0], steps


# ------------------------------------------------------------------------------------------------
# greedy start
# ------------------------------------------------------------------------------------------------
def test_the_best_trial_wins_not_the_first_and_not_the_worst():
    rng = np.random.default_rng(11)
    x = rng.permutation(400)[:20].astype(np.float64)               # 20 distinct integers
    batch, stream, found = 20, 3, 0
    for seed in range(400):
        best, win = greedy_start(x, 2, batch, seed, stream)
        first, _ = greedy_start(x, 2, batch, seed, stream, choose="first")
        worst, _ = greedy_start(x, 2, batch, seed, stream, choose="worst")
        exp = one_step_from(x, best, seed, stream, batch)
        alt1, alt2 = one_step_from(x, first, seed, stream, batch), one_step_from(x, worst, seed, stream, batch)
        if win != [1] or np.array_equal(exp, alt1) or np.array_equal(exp, alt2):
            continue                                               # not a telling case: try the next seed
        got, steps = fit_1d(x, 2, batch=batch, max_iter=1, patience=10 ** 6, ratio=0.0, seed=seed, stream=stream)
        assert steps == 1
        assert np.array_equal(got, exp), (seed, got, exp)
        found += 1
        if found == 5:
            break
    assert found == 5


def test_two_plus_floor_log_k_trials_are_drawn():
    """k = 8 draws four trials per centre: on inputs where some centre's winner is the fourth trial
    a fit that drew fewer trials would start, and end its first step, elsewhere."""
    rng = np.random.default_rng(12)
    x = rng.permutation(2000)[:40].astype(np.float64)
    batch, stream, found = 40, 1, 0
    for seed in range(400):
        four, win = greedy_start(x, 8, batch, seed, stream)
        three, _ = greedy_start(x, 8, batch, seed, stream, trials=3)
        exp, alt = one_step_from(x, four, seed, stream, batch), one_step_from(x, three, seed, stream, batch)
        if 3 not in win or np.array_equal(exp, alt):
            continue
        got, _ = fit_1d(x, 8, batch=batch, max_iter=1, patience=10 ** 6, ratio=0.0, seed=seed, stream=stream)
        assert np.array_equal(got, exp), (seed, got, exp)
        found += 1
        if found == 3:
            break
    assert found == 3


# ------------------------------------------------------------------------------------------------
# averaging weight of the stop rule
# ------------------------------------------------------------------------------------------------
def _stop_step(per_point, alpha, patience):
    ewa, ewa_min, bad = 0.0, math.inf, 0
    for t, v in enumerate(per_point):
        ewa = v if t == 0 else ewa * (1.0 - alpha) + v * alpha
        if ewa < ewa_min:
            ewa_min, bad = ewa, 0
        else:
            bad += 1
            if bad >= patience:
                return t + 1
    return len(per_point)


def test_the_stop_rule_averages_with_weight_two_batches_over_n_plus_one():
    """k = 1: the centre before step t is the start point (t = 0) or the mean of everything drawn so
    far, so each minibatch's per-point inertia follows from the draws alone; the stop step under the
    stated weight is then predicted and differs from the one no averaging (alpha = 1) would give."""
    rng = np.random.default_rng(13)
    N, batch, patience, stream = 600, 16, 3, 2
    x = rng.integers(-40, 41, size=(N, 2)).astype(np.float64)
    alpha = min(1.0, 2.0 * batch / (N + 1.0))
    assert alpha < 0.06
    found = 0
    for seed in range(100):
        n_init = min(N, max(3 * batch, 3))
        start = x[sample_order(seed, stream, N, n_init)[index(word(seed, 0, 2, stream, 0), n_init)]]
        drawn, per_point, centre = [], [], start
        for t in range(200):
            idx = minibatch(seed, stream, t, batch, N)
            per_point.append(float(((x[idx] - centre) ** 2).sum() / batch))
            drawn += idx
            centre = x[drawn].sum(axis=0) / len(drawn)
        want, plain = _stop_step(per_point, alpha, patience), _stop_step(per_point, 1.0, patience)
        # keep clear of cases a last-bit difference in the running mean could flip
        ewa, trail = 0.0, []
        for t, v in enumerate(per_point[:want]):
            ewa = v if t == 0 else ewa * (1.0 - alpha) + v * alpha
            trail.append(ewa)
        gaps = [abs(trail[t] - min(trail[:t])) for t in range(1, len(trail))]
        if want == plain or want >= 150 or min(gaps) < 1e-6:
            continue
        _, steps = orc.minibatch_kmeans(x, 1, batch=batch, max_iter=100, patience=patience, ratio=0.0, seed=seed,
                                        stream=stream)
        assert steps == want, (seed, steps, want, plain)
        found += 1
        if found == 4:
            break
    assert found == 4


# ------------------------------------------------------------------------------------------------
# reassignment
# ------------------------------------------------------------------------------------------------
def _outlier_case(seed, stream, N, batch, outlier_at):
    """Main points are small integers, one point is a far outlier. Returns None unless the greedy
    start puts one centre on a main point (index 0 or 1) and the other on the outlier."""
    rng = np.random.default_rng(1000 + seed)
    x = rng.integers(0, 50, size=N).astype(np.float64)
    x[outlier_at] = 1.0e4
    start, _ = greedy_start(x, 2, batch, seed, stream)
    if sorted(start.tolist())[1] != 1.0e4 or sorted(start.tolist())[0] >= 50:
        return None
    return x, int(np.argmax(start))                                # index of the centre on the outlier


def _first_jump(counts_b, counts_a, ratio):
    """First step t at which (t + 1) is a multiple of 10 + floor(smallest count) and the outlier's
    centre is starved; counts are those after the step's update."""
    for t, (cb, ca) in enumerate(zip(counts_b, counts_a)):
        if (t + 1) % (10 + int(min(cb, ca))) == 0 and cb < ratio * max(cb, ca):
            return t
    return None


def test_reassignment_waits_for_ten_plus_the_smallest_count_and_lands_on_a_minibatch_point():
    """The outlier's centre keeps the outlier as long as it only receives copies of it, and its
    count is the number of times the outlier was drawn: on seeds where that count is 2 from step 9
    on, the first reassignment falls on step 11 (12 = 10 + 2), not on step 9 (a fixed period of 10).
    A fit of exactly 12 steps therefore ends with that centre ON the point the tag-4 word picks from
    the last minibatch; a fit of 9 steps still has it on the outlier."""
    N, batch, stream, ratio, outlier_at, found = 48, 16, 4, 0.5, 47, 0
    for seed in range(3000):
        case = _outlier_case(seed, stream, N, batch, outlier_at)
        if case is None:
            continue
        x, b = case
        draws = [minibatch(seed, stream, t, batch, N) for t in range(12)]
        cb = np.cumsum([d.count(outlier_at) for d in draws])
        ca = np.cumsum([batch - d.count(outlier_at) for d in draws])
        if not (cb[9] == 2 and cb[11] == 2) or _first_jump(cb, ca, ratio) != 11:
            continue
        lands_on = x[draws[11][index(word(seed, 0, 4, stream, 11), batch)]]
        if lands_on == 1.0e4:
            continue
        kw = dict(batch=batch, patience=10 ** 6, ratio=ratio, seed=seed, stream=stream)
        early, s9 = fit_1d(x, 2, max_iter=3, **kw)                 # 3 * ceil(48 / 16) = 9 steps
        late, s12 = fit_1d(x, 2, max_iter=4, **kw)                 # 12 steps
        assert (s9, s12) == (9, 12)
        assert early[b] == 1.0e4, (seed, early)                    # a fixed period of 10 would have moved it at step 9
        assert late[b] == lands_on, (seed, late, lands_on)
        found += 1
        if found == 3:
            break
    assert found == 3


def test_a_moved_centre_takes_the_smallest_count_that_stays():
    """Reassignment at step 10 (11 = 10 + 1), one more step after it: the moved centre then sits at
    (p * c + S) / (c + n), p the point it landed on, c the other centre's count at the time of the
    move, S and n the sum and number of step 11's points nearer to p. With count 0 instead it would
    sit at S / n."""
    N, batch, stream, ratio, outlier_at, found = 48, 16, 6, 0.5, 47, 0
    for seed in range(6000):
        case = _outlier_case(seed, stream, N, batch, outlier_at)
        if case is None:
            continue
        x, b = case
        a = 1 - b
        draws = [minibatch(seed, stream, t, batch, N) for t in range(12)]
        cb = np.cumsum([d.count(outlier_at) for d in draws])
        ca = np.cumsum([batch - d.count(outlier_at) for d in draws])
        if _first_jump(cb, ca, ratio) != 10:
            continue
        p = x[draws[10][index(word(seed, 0, 4, stream, 10), batch)]]
        if p == 1.0e4:
            continue
        # the other centre: mean of every main point drawn through step 10 (the start point has count 0)
        main = [i for d in draws[:11] for i in d if i != outlier_at]
        centre_a, count_a = x[main].sum() / len(main), float(len(main))
        pts = x[draws[11]]
        # step 11's points nearer to p than to the other centre (a tie goes to the smaller centre index)
        near_p = np.abs(pts - p) <= np.abs(pts - centre_a) if b < a else np.abs(pts - p) < np.abs(pts - centre_a)
        if not near_p.any() or np.any(pts[near_p] == 1.0e4):
            continue                                               # keep the case simple: the outlier, if drawn, goes to the other centre
        n, S = int(near_p.sum()), float(pts[near_p].sum())
        want, with_zero = (p * count_a + S) / (count_a + n), S / n
        if abs(want - with_zero) < 1e-6:
            continue
        got, steps = fit_1d(x, 2, batch=batch, max_iter=4, patience=10 ** 6, ratio=ratio, seed=seed, stream=stream)
        assert steps == 12
        assert abs(got[b] - want) < 1e-9, (seed, got[b], want, with_zero)
        found += 1
        if found == 3:
            break
    assert found == 3


def test_at_most_half_a_minibatch_of_centres_moves():
    """batch = 4, five centres of which four sit on far outliers and starve together: only the two
    with the smallest index move (onto the points the tag-4 words pick), the other two stay."""
    N, batch, stream, ratio, found = 12, 4, 7, 0.5, 0
    outliers = {8: 1.0e4, 9: 2.0e4, 10: 3.0e4, 11: 4.0e4}
    for seed in range(4000):
        rng = np.random.default_rng(2000 + seed)
        x = rng.integers(0, 50, size=N).astype(np.float64)
        for i, v in outliers.items():
            x[i] = v
        start, _ = greedy_start(x, 5, batch, seed, stream)
        if sorted(start.tolist())[1:] != sorted(outliers.values()):
            continue                                               # the start must sit on all four outliers
        on = {u: [i for i, v in outliers.items() if v == start[u]][0] for u in range(5) if start[u] >= 1.0e4}
        main_u = [u for u in range(5) if u not in on][0]
        # counts after each step: an outlier's centre receives exactly the draws of that outlier
        counts = np.zeros(5)
        t_jump = None
        for t in range(30):
            d = minibatch(seed, stream, t, batch, N)
            for u, i in on.items():
                counts[u] += d.count(i)
            counts[main_u] += sum(1 for i in d if i not in outliers)
            starved = [u for u in range(5) if counts[u] < ratio * counts.max()]
            if (t + 1) % (10 + int(counts.min())) == 0 and starved:
                t_jump, last = t, d
                break
        if t_jump is None or (t_jump + 1) % 3 != 0 or sorted(starved) != sorted(on) or len(starved) != 4:
            continue
        slots = list(range(batch))
        for i in range(2):
            r = i + index(word(seed, i, 4, stream, t_jump), batch - i)
            slots[i], slots[r] = slots[r], slots[i]
        movers, stayers = sorted(on)[:2], sorted(on)[2:]
        got, steps = fit_1d(x, 5, batch=batch, max_iter=(t_jump + 1) // 3, patience=10 ** 6, ratio=ratio, seed=seed,
                            stream=stream)
        assert steps == t_jump + 1
        assert [got[u] for u in movers] == [x[last[slots[0]]], x[last[slots[1]]]], (seed, got)
        assert [got[u] for u in stayers] == [start[u] for u in stayers], (seed, got)
        found += 1
        if found == 3:
            break
    assert found == 3
