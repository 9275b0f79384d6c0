"""mts_place_tables (host code of the library, no GPU needed) against the oracle's brute force: the minimal
lookup time of Eq. 6 is unique, the placement that reaches it need not be, so the times are compared and the
placement is checked to be feasible and to give that time."""
import numpy as np
import pytest

import oracle
from paper_2305_01515_b200 import binding as mb
from paper_2305_01515_b200 import workload as wl


def _check(size, cost, cap, bw_hbm, bw_host):
    place, t, optimal = mb.place_tables(size, cost, cap, bw_hbm, bw_host)
    ref_place, ref_t = oracle.place_tables(size, cost, cap, bw_hbm, bw_host)
    assert optimal
    assert sum(s for s, p in zip(size, place) if p == 0) <= cap
    assert abs(sum(c / (bw_hbm if p == 0 else bw_host) for c, p in zip(cost, place)) - t) <= 1e-12 * max(t, 1e-300)
    assert abs(t - ref_t) <= 1e-12 * max(ref_t, 1e-300)


def test_random_instances_match_brute_force():
    rng = np.random.default_rng(1)
    for trial in range(200):
        T = int(rng.integers(1, 15))
        size = rng.integers(0, 1000, T).tolist()
        cost = (rng.uniform(0.0, 10.0, T) * (rng.random(T) > 0.1)).tolist()
        cap = int(rng.integers(0, sum(size) + 10))
        _check(size, cost, cap, 6.5e12, 5.5e10)
    _check([5, 5, 5], [1.0, 1.0, 1.0], 10, 1.0, 2.0)          # a "fast" memory that is the slower one: nothing goes there


def test_configuration_3_tables_under_a_budget():
    """The 64 tables of configuration 3 (sizes and D * L * p from the spec) under a third of their total size:
    the small, hot tables go to HBM first (Section 3.1: most of the bandwidth demand comes from small tables)."""
    spec = wl.config3()
    size = [int(t.rows * t.dim * 2) for t in spec.tables]
    cost = [t.dim * 2 * t.pooling for t in spec.tables]
    cap = sum(size) // 3
    place, t, optimal = mb.place_tables(size, cost, cap, 6.5e12, 5.5e10)
    assert optimal and sum(s for s, p in zip(size, place) if p == 0) <= cap
    in_hbm = [i for i, p in enumerate(place) if p == 0]
    traffic_share = sum(cost[i] for i in in_hbm) / sum(cost)
    assert traffic_share > 0.9 and len(in_hbm) > 32
    # never worse than the greedy order by traffic per byte
    order = sorted(range(64), key=lambda i: -cost[i] / size[i])
    room, greedy = cap, [1] * 64
    for i in order:
        if size[i] <= room:
            room -= size[i]; greedy[i] = 0
    t_greedy = sum(c / (6.5e12 if p == 0 else 5.5e10) for c, p in zip(cost, greedy))
    assert t <= t_greedy * (1 + 1e-12)


def test_bad_arguments_are_refused():
    with pytest.raises(mb.MtsError):
        mb.place_tables([1], [1.0], -1, 1.0, 1.0)
    with pytest.raises(mb.MtsError):
        mb.place_tables([1], [1.0], 1, 0.0, 1.0)
