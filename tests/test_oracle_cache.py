"""Pins for the oracle's cache (Section 5.3.1 cache class: data, tags, timestamps; Section 5.5.2
LRU in three steps; Section 5.5.4 insert / evict flow; Section 5.7 prefetch invariant)."""
from collections import OrderedDict

import numpy as np
import pytest

import oracle
from paper_2305_01515_b200 import workload as wl
from helpers import small_spec


class ListCache:
    """Naive per-set simulation with python lists; same contract, different construction:
    each set is a list of [way, key, stamp, dirty, count]; victims are taken in (stamp, way) order
    for LRU and in (count, stamp, way) order for LFU, where count = lookups of the key while it has
    been resident (every occurrence in a batch counts), starting at the inserting batch's lookups."""

    def __init__(self, S, ways, lock_depth=0, policy=0):
        self.S, self.ways, self.lock, self.policy = S, ways, lock_depth, policy
        self.sets = [[[w, -1, -1, 0, 0] for w in range(ways)] for _ in range(S)]

    def step(self, keys, step, capacity=None):
        import copy
        self.prev_sets = copy.deepcopy(self.sets)                    # state before the call
        self.prev_resident = {e[1] for s in self.sets for e in s if e[1] >= 0}
        uniq = sorted(set(int(k) for k in keys))
        times = {}
        for k in keys:
            times[int(k)] = times.get(int(k), 0) + 1
        by_set = {}
        for k in uniq:
            by_set.setdefault(oracle.cache_set_of(k, self.S), []).append(k)
        slot, hits = {}, set()
        for s, ks in by_set.items():
            for k in ks:
                for e in self.sets[s]:
                    if e[1] == k:
                        hits.add(k); slot[k] = s * self.ways + e[0]
        for s, ks in by_set.items():
            for e in self.sets[s]:
                if e[1] in hits and e[1] in ks:
                    e[2] = step
                    e[4] += times[e[1]]
        miss, evict, overflow = [], [], 0
        for s in sorted(by_set):
            if self.policy == 1:
                order = sorted(self.sets[s], key=lambda e: (e[4], e[2], e[0]))
            else:
                order = sorted(self.sets[s], key=lambda e: (e[2], e[0]))
            cands = [e for e in order if e[1] == -1 or e[2] < step - self.lock]
            todo = [k for k in by_set[s] if k not in hits]
            for j, k in enumerate(todo):
                if j < len(cands) and (capacity is None or len(miss) < capacity):
                    e = cands[j]
                    if e[1] != -1:
                        evict.append((e[1], s * self.ways + e[0], e[3]))
                    e[1], e[2], e[3], e[4] = k, step, 0, times[k]
                    slot[k] = s * self.ways + e[0]
                    miss.append((k, slot[k]))
                else:
                    slot[k] = -1; overflow += 1
        n_hit = sum(1 for k in keys if int(k) in hits)
        return slot, miss, evict, overflow, n_hit, len(hits)


def _check_invariants(c, S, ways):
    tags = c.tags
    for s in range(S):
        live = tags[s][tags[s] >= 0]
        assert len(set(live.tolist())) == len(live), "duplicate tag in a set"
        for k in live:
            assert oracle.cache_set_of(int(k), S) == s
    assert (c.ts[tags < 0] == -1).all()
    assert (tags >= 0).sum() <= S * ways


@pytest.mark.parametrize("policy", [0, 1])
@pytest.mark.parametrize("S,ways,lock", [(1, 4, 0), (5, 4, 0), (7, 32, 1), (3, 2, 1), (16, 8, 2)])
def test_lookup_insert_vs_list_simulation(S, ways, lock, policy):
    """LRU and LFU against the list simulation; the Zipf keys repeat inside a batch (multiplicities
    up to dozens) and small universes give many equal counts, so count ties are frequent."""
    rng = np.random.default_rng(S * 100 + ways)
    c = oracle.Cache(S, ways, 4, wl.FP32, policy, lock, with_data=False)
    ref = ListCache(S, ways, lock, policy)
    occupancy = 0
    for step in range(40):
        n = int(rng.integers(0, 3 * S * ways // 2 + 2))
        keys = (rng.zipf(1.3, n) % (6 * S * ways)).astype(np.int64)
        res = c.lookup_insert(keys, step)
        slot, miss, evict, overflow, n_hit, n_uhit = ref.step(keys, step)
        cnt = res["counters"]
        assert cnt["lookups"] == n and cnt["unique"] == len(set(keys.tolist()))
        assert cnt["hit_lookups"] + cnt["miss_lookups"] == n
        assert cnt["unique_hits"] + cnt["unique_misses"] == cnt["unique"]
        assert cnt["hit_lookups"] == n_hit and cnt["unique_hits"] == n_uhit
        assert cnt["overflow"] == overflow and cnt["inserted"] == len(miss) and cnt["evicted"] == len(evict)
        assert cnt["unique_misses"] == cnt["inserted"] + cnt["overflow"]
        assert [slot[int(k)] for k in keys] == res["slot_of_lookup"].tolist()
        assert miss == list(zip(res["miss_keys"].tolist(), res["miss_slots"].tolist()))
        assert [(k, s) for k, s, _ in evict] == list(zip(res["evict_keys"].tolist(), res["evict_slots"].tolist()))
        assert [d for _, _, d in evict] == res["evict_dirty"].tolist()
        assert cnt["evicted_dirty"] == sum(d for _, _, d in evict)
        occupancy += cnt["inserted"] - cnt["evicted"]
        assert occupancy == int((c.tags >= 0).sum())
        _check_invariants(c, S, ways)
        for s_i in range(S):
            for e in ref.sets[s_i]:
                if e[1] >= 0:
                    assert int(c.freq[s_i][e[0]]) == e[4], "use count"
        # mark the slots of every second distinct key dirty on both sides
        for k in sorted(set(keys.tolist()))[::2]:
            sl = slot[k]
            if sl >= 0:
                c.dirty[sl] = 1
                for e in ref.sets[sl // ways]:
                    if e[0] == sl % ways:
                        e[3] = 1
    c.close()


@pytest.mark.parametrize("policy", [0, 1])
def test_full_miss_list_turns_further_misses_into_overflow(policy):
    """A miss list of `capacity` entries: the first `capacity` placements (in set, key order) stand, every
    later missing key is not inserted and its would-be victim keeps its way.  Checked against the list
    simulation, and against the unlimited call when the capacity is not reached."""
    S, ways = 6, 4
    rng = np.random.default_rng(11 + policy)
    c = oracle.Cache(S, ways, 4, wl.FP32, policy, 1, with_data=False)
    twin = oracle.Cache(S, ways, 4, wl.FP32, policy, 1, with_data=False)      # same calls, generous capacity
    ref = ListCache(S, ways, 1, policy)
    cut = whole = 0
    for step in range(30):
        keys = (rng.zipf(1.3, 40) % 150).astype(np.int64)
        cap = int(rng.integers(0, 12))
        # the same call without a limit, on a copy of the state
        twin.tags[:], twin.ts[:], twin.freq[:], twin.dirty[:] = c.tags, c.ts, c.freq, c.dirty
        free = twin.lookup_insert(keys, step)
        res = c.lookup_insert(keys, step, list_capacity=cap)
        slot, miss, evict, overflow, n_hit, n_uhit = ref.step(keys, step, capacity=cap)
        cnt = res["counters"]
        assert cnt["inserted"] == len(miss) <= cap and cnt["evicted"] == len(evict) and cnt["overflow"] == overflow
        assert cnt["unique_misses"] == cnt["inserted"] + cnt["overflow"]
        assert [slot[int(k)] for k in keys] == res["slot_of_lookup"].tolist()
        assert miss == list(zip(res["miss_keys"].tolist(), res["miss_slots"].tolist()))
        assert [(k, s) for k, s, _ in evict] == list(zip(res["evict_keys"].tolist(), res["evict_slots"].tolist()))
        _check_invariants(c, S, ways)
        if free["counters"]["inserted"] <= cap:          # the limit was not reached: nothing may differ
            whole += 1
            assert free["counters"] == cnt
            assert (free["slot_of_lookup"] == res["slot_of_lookup"]).all()
            assert (twin.tags == c.tags).all() and (twin.ts == c.ts).all() and (twin.freq == c.freq).all()
        else:
            cut += 1
            # the placements that fit are the first ones of the unlimited call
            assert free["miss_keys"][:cap].tolist() == res["miss_keys"].tolist()
    assert cut > 5 and whole > 2
    c.close(); twin.close()


def test_textbook_fully_associative_lru():
    """S = 1, one key per call, lock_depth 0 is the textbook LRU: compare with an OrderedDict."""
    ways = 4
    c = oracle.Cache(1, ways, 4, wl.FP32, 0, 0, with_data=False)
    lru = OrderedDict()
    rng = np.random.default_rng(5)
    for step, k in enumerate(rng.integers(0, 9, 400).tolist()):
        res = c.lookup_insert(np.array([k], np.int64), step)
        hit = k in lru
        if hit:
            lru.move_to_end(k)
        else:
            victim = None
            if len(lru) == ways:
                victim, _ = lru.popitem(last=False)
            lru[k] = True
            assert res["evict_keys"].tolist() == ([] if victim is None else [victim])
        assert res["counters"]["hit_lookups"] == (1 if hit else 0)
    c.close()


def test_cyclic_scan_never_hits_and_fitting_working_set_only_cold_misses():
    ways = 8
    c = oracle.Cache(1, ways, 4, wl.FP32, 0, 0, with_data=False)
    hits = 0
    for step in range(5 * (ways + 1)):
        hits += c.lookup_insert(np.array([step % (ways + 1)], np.int64), step)["counters"]["hit_lookups"]
    assert hits == 0
    c.close()
    S = 64
    c = oracle.Cache(S, 32, 4, wl.FP32, 0, 0, with_data=False)
    rng = np.random.default_rng(9)
    universe = rng.choice(10_000_000, 300, replace=False).astype(np.int64)   # ~4.7 per 32-way set
    misses = 0
    seen = set()
    for step in range(30):
        keys = rng.choice(universe, 100)
        cnt = c.lookup_insert(keys, step)["counters"]
        assert cnt["overflow"] == 0 and cnt["evicted"] == 0
        misses += cnt["unique_misses"]
        seen |= set(keys.tolist())
    assert misses == len(seen)
    c.close()


def test_lock_window_protects_rows_of_batches_in_flight():
    """Section 5.7: a prefetched row is not evicted before its batch has trained."""
    S, ways, lock = 2, 4, 1
    c = oracle.Cache(S, ways, 4, wl.FP32, 0, lock, with_data=False)
    rng = np.random.default_rng(2)
    prev = set()
    for step in range(50):
        keys = rng.integers(0, 40, 6).astype(np.int64)
        res = c.lookup_insert(keys, step)
        assert not (set(res["evict_keys"].tolist()) & prev), "evicted a row of the batch in flight"
        placed = {int(k) for k, s in zip(keys, res["slot_of_lookup"]) if s >= 0}
        prev = placed
    c.close()


def test_free_ways_are_usable_from_the_first_step_whatever_the_lock_depth():
    """Section 5.5.2: a missed index takes a free slot when there is one; eviction (and with it the
    lock window) only matters once the set is full."""
    c = oracle.Cache(2, 4, 4, wl.FP32, 0, 3, with_data=False)
    res = c.lookup_insert(np.arange(6, dtype=np.int64), 0)
    assert res["counters"]["overflow"] == 0 and res["counters"]["inserted"] == 6 and res["counters"]["evicted"] == 0
    c.close()


def test_set_hash_definition_and_range():
    """set = floor(((key * 0x9E3779B97F4A7C15) mod 2^64) * S / 2^64), checked with python integers."""
    rng = np.random.default_rng(0)
    for S in (1, 2, 3, 1000, 1_700_001, 2 ** 31 + 11):
        for key in rng.integers(0, 2 ** 40, 200).tolist() + [0, 1, 2 ** 32 - 1]:
            x = (key * 0x9E3779B97F4A7C15) % (1 << 64)
            assert oracle.cache_set_of(key, S) == (x * S) >> 64
    counts = np.bincount([oracle.cache_set_of(k, 97) for k in range(97 * 200)], minlength=97)
    assert counts.min() > 120 and counts.max() < 280     # consecutive keys spread over the sets


def test_lfu_keeps_frequent_rows():
    """LFU variant (Section 5.5.2): the victim is the least frequently used entry."""
    c = oracle.Cache(1, 2, 4, wl.FP32, 1, 0, with_data=False)
    for step in range(5):
        c.lookup_insert(np.array([7], np.int64), step)          # key 7: count 5
    c.lookup_insert(np.array([8], np.int64), 5)                 # key 8: count 1, most recent
    res = c.lookup_insert(np.array([9], np.int64), 6)
    assert res["evict_keys"].tolist() == [8]                    # LRU would have evicted 7
    c.close()
    c = oracle.Cache(1, 2, 4, wl.FP32, 0, 0, with_data=False)
    for step in range(5):
        c.lookup_insert(np.array([7], np.int64), step)
    c.lookup_insert(np.array([8], np.int64), 5)
    assert c.lookup_insert(np.array([9], np.int64), 6)["evict_keys"].tolist() == [7]
    c.close()


def _one_set(policy, ways=2, lock=0):
    return oracle.Cache(1, ways, 4, wl.FP32, policy, lock, with_data=False)


def test_lfu_counts_lookups_not_distinct_keys():
    """Key 7 is looked up three times in one batch, key 8 once in each of two batches: by lookups 8 is
    the less used (2 < 3) and is evicted; counting batches (or distinct keys) would evict 7."""
    c = _one_set(1)
    c.lookup_insert(np.array([7, 7, 7], np.int64), 0)
    c.lookup_insert(np.array([8], np.int64), 1)
    c.lookup_insert(np.array([8], np.int64), 2)
    assert c.freq[0].tolist() == [3, 2]
    res = c.lookup_insert(np.array([9], np.int64), 3)
    assert res["evict_keys"].tolist() == [8]
    c.close()


def test_lfu_count_ties_fall_back_to_timestamp_then_way():
    c = _one_set(1, ways=3)
    c.lookup_insert(np.array([1, 2, 3], np.int64), 0)       # ways 0, 1, 2 (ascending key), counts 1, 1, 1
    c.lookup_insert(np.array([1], np.int64), 1)             # key 1: count 2
    c.lookup_insert(np.array([3], np.int64), 2)             # key 3: count 2, newer than key 1
    c.lookup_insert(np.array([2], np.int64), 3)             # key 2: count 2, newest
    res = c.lookup_insert(np.array([10], np.int64), 4)      # all counts equal: the oldest stamp goes
    assert res["evict_keys"].tolist() == [1]
    c.close()
    c = _one_set(1, ways=3)
    c.lookup_insert(np.array([1, 2, 3], np.int64), 0)       # same count, same stamp: lowest way first
    res = c.lookup_insert(np.array([10, 11], np.int64), 1)
    assert res["evict_keys"].tolist() == [1, 2] and res["evict_slots"].tolist() == [0, 1]
    c.close()


def test_lfu_count_restarts_when_a_key_is_inserted_again():
    c = _one_set(1)
    for step in range(6):
        c.lookup_insert(np.array([7], np.int64), step)                       # key 7: count 6
    c.lookup_insert(np.array([8, 8], np.int64), 6)                          # key 8: count 2
    assert c.lookup_insert(np.array([9, 9, 9], np.int64), 7)["evict_keys"].tolist() == [8]   # key 9: count 3
    assert c.lookup_insert(np.array([8, 8, 8, 8], np.int64), 8)["evict_keys"].tolist() == [9]
    assert sorted(c.freq[0].tolist()) == [4, 6]               # key 8 starts again at this batch's 4 lookups
    c.close()


def test_lfu_lock_window_overrides_the_count():
    """A rarely used row stamped inside the lock window is not a candidate; the frequently used one goes."""
    c = _one_set(1, lock=1)
    for step in range(4):
        c.lookup_insert(np.array([7, 7], np.int64), step)                    # key 7: count 8, stamp 3
    c.lookup_insert(np.array([8], np.int64), 4)                             # key 8: count 1, stamp 4
    res = c.lookup_insert(np.array([9], np.int64), 5)                       # 8 is locked (4 >= 5 - 1)
    assert res["evict_keys"].tolist() == [7]
    c.close()


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("sets,lock", [(1, 0), (3, 0), (40, 1)])
def test_cache_is_transparent(dtype, sets, lock):
    """Weights (after flush) and momentum after K batches through any cache geometry are
    bit-identical to the uncached run: pins prefetch, dirty tracking, writeback, overflow."""
    spec = small_spec(T=2, rows=(90, 60), dims=(8, 8), B=6, pooling=4.0, dtype=dtype, alpha=1.1, seed=6)
    W_ref = wl.all_weights_numpy(spec); m_ref = np.zeros(int(spec.row_offset[-1]), np.float32)
    W_host = W_ref.copy(); m = m_ref.copy()
    c = oracle.Cache(sets, 4, 8, dtype, 0, lock)
    outs = []
    args = (spec.dtype, spec.dims, spec.out_offset[:-1], spec.weight_offset[:-1])
    B = spec.batch
    total_overflow = 0
    for k in range(12):
        idx, off = wl.gen_batch(spec, k)
        grad = wl.gen_grad(spec, k)
        o_ref = oracle.tbe_forward(*args, W_ref, B, idx, off)
        oracle.tbe_backward_rowwise_adagrad(*args, spec.row_offset, W_ref, m_ref, B, idx, off, grad, 0.01, 1e-8)
        keys = np.concatenate([spec.row_offset[t] + idx[off[t * B]:off[(t + 1) * B]] for t in range(2)])
        res = c.lookup_insert(keys, k)
        total_overflow += res["counters"]["overflow"]
        staging = c.prefetch_misses(W_host, res)
        c.writeback_evicted(W_host, res, staging)
        cd = [c.data, c.data]; dirty = [c.dirty, c.dirty]
        o = oracle.tbe_forward(*args, W_host, B, idx, off, 0, res["slot_of_lookup"], cd)
        oracle.tbe_backward_rowwise_adagrad(*args, spec.row_offset, W_host, m, B, idx, off, grad, 0.01, 1e-8,
                                            0, res["slot_of_lookup"], cd, dirty)
        np.testing.assert_array_equal(o, o_ref)
    c.flush(W_host)
    assert (c.dirty == 0).all()
    np.testing.assert_array_equal(W_host.view(np.uint8), W_ref.view(np.uint8))
    np.testing.assert_array_equal(m, m_ref)
    if sets == 1:
        assert total_overflow > 0      # the tiny cache really exercised the bypass path
    c.close()
