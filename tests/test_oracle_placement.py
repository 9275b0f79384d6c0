"""Pins for the oracle's table placement (Section 5.6, Eq. 6: lookup time = sum of D * L * p / BW of the
memory that holds the table; one table in one memory; the fast memory's capacity is respected)."""
import itertools

import numpy as np

import oracle


def _time(place, cost, bw_fast, bw_slow):
    return sum(c / (bw_fast if p == 0 else bw_slow) for p, c in zip(place, cost))


def test_placement_special_cases():
    size = [10, 20, 30]
    cost = [5.0, 1.0, 3.0]
    # everything fits: all tables in the fast memory
    p, t = oracle.place_tables(size, cost, 60, 8.0, 1.0)
    assert p.tolist() == [0, 0, 0] and abs(t - 9.0 / 8.0) < 1e-15
    # nothing fits
    p, t = oracle.place_tables(size, cost, 5, 8.0, 1.0)
    assert p.tolist() == [1, 1, 1] and abs(t - 9.0) < 1e-15
    # room for 30: table 0 + table 1 (cost 6) beats table 2 alone (cost 3)
    p, t = oracle.place_tables(size, cost, 30, 8.0, 1.0)
    assert p.tolist() == [0, 0, 1] and abs(t - (6.0 / 8.0 + 3.0)) < 1e-15
    # equal bandwidths: any feasible placement has the same time
    _, t = oracle.place_tables(size, cost, 30, 2.0, 2.0)
    assert abs(t - 4.5) < 1e-15
    # a small hot table wins against a big cold one (the paper's observation on size versus bandwidth demand)
    p, _ = oracle.place_tables([100, 1], [1.0, 50.0], 100, 10.0, 1.0)
    assert p.tolist() == [1, 0]


def test_placement_is_the_minimum_over_all_assignments():
    """Independent enumeration with itertools on random instances; the capacity is never exceeded."""
    rng = np.random.default_rng(0)
    for trial in range(30):
        T = int(rng.integers(1, 10))
        size = rng.integers(1, 100, T)
        cost = rng.uniform(0.1, 10.0, T)
        cap = int(rng.integers(0, size.sum() + 10))
        bw_fast, bw_slow = 6.5e12, 5.5e10
        p, t = oracle.place_tables(size, cost, cap, bw_fast, bw_slow)
        assert sum(s for s, x in zip(size, p) if x == 0) <= cap
        assert abs(_time(p, cost, bw_fast, bw_slow) - t) <= 1e-12 * t
        best = min(_time(q, cost, bw_fast, bw_slow) for q in itertools.product((0, 1), repeat=T)
                   if sum(s for s, x in zip(size, q) if x == 0) <= cap)
        assert abs(best - t) <= 1e-12 * best
