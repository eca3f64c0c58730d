"""Pins of the oracle's slice choice (Section 5.2, Greedy-Least-Loaded): hand-worked choices, the
water-filling closed form, and the competitive bound of Appendix C, (m + 3) / 2 times the best
offline congestion, against a brute-force offline optimum on tiny instances. CPU only."""
import itertools

import numpy as np
import pytest

import oracle


def test_hand_worked_choices():
    # utilisation sums 0.5, 0.3, 0.7 -> slice 1
    assert oracle.gll_choose([10, 10, 30], [40, 20, 40], [100, 100, 100]) == 1
    # capacities differ: 30/60 = 0.5 against 45/100 = 0.45 -> slice 1, though it holds more blocks
    assert oracle.gll_choose([20, 25], [10, 20], [60, 100]) == 1
    # the peer's use counts as much as one's own (the example of Section 5.2: memory the peer is
    # using is memory this process should not count on)
    assert oracle.gll_choose([0, 30], [50, 10], [100, 100]) == 1
    # exact ties (1/3 = 2/6 = 3/9) go to the first slice; floating point would not see them as equal
    assert oracle.gll_choose([1, 1, 2], [0, 1, 1], [3, 6, 9]) == 0
    assert oracle.gll_choose([5], [5], [10]) == 0 and oracle.gll_choose([], [], []) == -1


def test_identical_units_from_one_owner_fill_like_water():
    """n unit requests of one process over k empty, equal slices: loads never differ by more than
    one, so the fullest slice holds ceil(n / k) (a reversed comparison would pile them on one)."""
    for k in (2, 3, 7):
        own = [0] * k
        for n in range(1, 40):
            own[oracle.gll_choose(own, [0] * k, [64] * k)] += 1
            assert max(own) - min(own) <= 1 and max(own) == -(-n // k)


def _slices(m):
    return list(itertools.combinations(range(m), 2))


def _gll_congestion(m, jobs):
    """jobs: [(owner, arrival, departure)], unit demand. Peak load over time and slices when every
    arrival goes to the least utilised slice incident to its owner (capacity 1 per slice, so
    utilisation = load)."""
    pairs = _slices(m)
    load = {p: 0 for p in pairs}
    place, peak = {}, 0
    events = sorted([(a, 1, r) for r, (_, a, _) in enumerate(jobs)] + [(d, 0, r) for r, (_, _, d) in enumerate(jobs)])
    for _, kind, r in events:                      # departures before arrivals at the same tick
        owner = jobs[r][0]
        if kind == 0:
            load[place[r]] -= 1
            continue
        inc = [p for p in pairs if owner in p]
        # one counter per slice: everything allocated in it, by either end
        k = oracle.gll_choose([load[p] for p in inc], [0] * len(inc), [1000] * len(inc))
        place[r] = inc[k]
        load[inc[k]] += 1
        peak = max(peak, max(load.values()))
    return peak


def _opt_congestion(m, jobs):
    pairs = _slices(m)
    choices = [[p for p in pairs if o in p] for o, _, _ in jobs]
    ticks = sorted({a for _, a, _ in jobs})
    best = len(jobs)
    for assign in itertools.product(*choices):
        peak = 0
        for t in ticks:
            load = {}
            for (o, a, d), p in zip(jobs, assign):
                if a <= t < d:
                    load[p] = load.get(p, 0) + 1
            peak = max(peak, max(load.values(), default=0))
            if peak >= best:
                break
        best = min(best, peak)
    return best


@pytest.mark.parametrize("m", [3, 4])
def test_congestion_stays_within_the_bound_of_the_offline_optimum(m):
    rng = np.random.default_rng(m)
    worst = 0.0
    for _ in range(60):
        n = int(rng.integers(3, 9))
        jobs = []
        for _ in range(n):
            a = int(rng.integers(0, 6))
            jobs.append((int(rng.integers(0, m)), a, a + int(rng.integers(1, 6))))
        g, o = _gll_congestion(m, jobs), _opt_congestion(m, jobs)
        assert o >= 1 and g >= o
        assert g <= (m + 3) / 2 * o
        worst = max(worst, g / o)
    assert worst > 1.0          # the instances are hard enough for the greedy rule to lose sometimes
