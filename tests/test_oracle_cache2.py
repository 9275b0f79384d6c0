"""Pins for the oracle's two-level exclusive cache (Section 5.3.2: two levels, exclusive; Section 5.5.4:
promotion of second-level hits and fetched rows, demotion of first-level LRU rows, eviction of
second-level LRU rows to the lowest tier)."""
from collections import OrderedDict

import numpy as np
import pytest

import oracle
from paper_2305_01515_b200 import workload as wl
from helpers import small_spec
from test_oracle_cache import ListCache


class SecondLevel:
    """List simulation of the second level: per set a list of [way, key, stamp, dirty, count]; rows leave when
    they are requested again, first-level victims enter in (set, key) order taking free ways first, then ways
    outside the lock window in (stamp, way) order [LFU: (count, stamp, way)]."""

    def __init__(self, S, ways, lock=0, policy=0):
        self.S, self.ways, self.lock, self.policy = S, ways, lock, policy
        self.sets = [[[w, -1, -1, 0, 0] for w in range(ways)] for _ in range(S)]

    def find(self, key):
        s = oracle.cache_set_of(key, self.S)
        for e in self.sets[s]:
            if e[1] == key:
                return s * self.ways + e[0], e
        return -1, None

    def remove(self, key):
        _, e = self.find(key)
        e[1], e[2], e[3], e[4] = -1, -1, 0, 0

    def insert(self, victims, step):
        """victims: [(key, stamp, dirty, count)] -> ({key: slot or -1}, [(evicted key, slot, dirty)])."""
        by_set = {}
        for v in victims:
            by_set.setdefault(oracle.cache_set_of(v[0], self.S), []).append(v)
        dst, out = {}, []
        for s in sorted(by_set):
            order = sorted(self.sets[s], key=(lambda e: (e[4], e[2], e[0])) if self.policy == 1 else (lambda e: (e[2], e[0])))
            cands = [e for e in order if e[1] == -1 or e[2] < step - self.lock]
            for j, (key, stamp, dirty, count) in enumerate(sorted(by_set[s])):
                if j < len(cands):
                    e = cands[j]
                    if e[1] != -1:
                        out.append((e[1], s * self.ways + e[0], e[3]))
                    e[1], e[2], e[3], e[4] = key, stamp, dirty, count
                    dst[key] = s * self.ways + e[0]
                else:
                    dst[key] = -1
        return dst, out


@pytest.mark.parametrize("policy", [0, 1])
@pytest.mark.parametrize("S1,S2,ways,lock", [(1, 1, 4, 0), (3, 5, 4, 1), (4, 2, 8, 2), (3, 2, 2, 1)])
def test_two_levels_vs_one_level_cache_and_list_simulation(S1, S2, ways, lock, policy):
    rng = np.random.default_rng(S1 * 31 + S2 * 7 + ways + policy)
    l1 = oracle.Cache(S1, ways, 4, wl.FP32, policy, lock, with_data=False)
    l2 = oracle.Cache(S2, ways, 4, wl.FP32, policy, lock, with_data=False)
    c2 = oracle.Cache2(l1, l2)
    one = oracle.Cache(S1, ways, 4, wl.FP32, policy, lock, with_data=False)      # the first level alone
    sim1 = ListCache(S1, ways, lock, policy)
    sim2 = SecondLevel(S2, ways, lock, policy)
    l2_hits = promoted = demoted = bypass = dropped = ev2_total = 0
    for step in range(60):
        n = int(rng.integers(0, 2 * (S1 + S2) * ways + 2))
        keys = (rng.zipf(1.25, n) % (5 * (S1 + S2) * ways)).astype(np.int64)
        res = c2.lookup_insert(keys, step)
        ref = one.lookup_insert(keys, step)
        cnt = res["counters"]
        # the first level decides exactly like a one-level cache
        assert {k: cnt[k] for k in oracle.COUNTER_NAMES} == ref["counters"]
        assert (res["slot_of_lookup"] == ref["slot_of_lookup"]).all()
        assert (res["fetch_keys"] == ref["miss_keys"]).all() and (res["fetch_slots"] == ref["miss_slots"]).all()
        assert (res["ev1_keys"] == ref["evict_keys"]).all() and (res["ev1_slots"] == ref["evict_slots"]).all()
        assert (res["ev1_dirty"] == ref["evict_dirty"]).all()
        # the second level against the list simulation, driven by the one-level list simulation
        slot, miss, evict, overflow, n_hit, n_uhit = sim1.step(keys, step)
        stamps = {e[1]: (e[2], e[4]) for s in sim1.prev_sets for e in s if e[1] >= 0}
        uniq = sorted(set(keys.tolist()))
        hits2 = {k: sim2.find(k)[0] for k in uniq if sim2.find(k)[0] >= 0}
        assert not (set(hits2) & {k for k in uniq if k in sim1.prev_resident}), "a key in both levels"
        src = {k: hits2.get(k, -1) for k, _ in miss}
        assert res["fetch_src"].tolist() == [src[k] for k, _ in miss]
        drop = sorted((k, hits2[k]) for k in hits2 if slot[k] < 0)
        assert sorted(zip(res["drop_keys"].tolist(), res["drop_slots"].tolist())) == drop
        dirty2 = {k: sim2.find(k)[1][3] for k in hits2}
        for k in hits2:
            sim2.remove(k)
        dst, out = sim2.insert([(k, stamps[k][0], d, stamps[k][1]) for k, _, d in evict], step)
        assert res["ev1_dst"].tolist() == [dst[k] for k, _, _ in evict]
        assert list(zip(res["ev2_keys"].tolist(), res["ev2_slots"].tolist(), res["ev2_dirty"].tolist())) == out
        assert cnt["l2_unique_hits"] == len(hits2) and cnt["promoted"] == len(hits2) - len(drop)
        assert cnt["l2_hit_lookups"] == sum(1 for k in keys.tolist() if k in hits2)
        assert cnt["demoted"] == sum(1 for v in dst.values() if v >= 0) and cnt["l2_bypass"] == sum(1 for v in dst.values() if v < 0)
        assert cnt["l2_evicted"] == len(out) and cnt["l2_evicted_dirty"] == sum(d for _, _, d in out)
        assert cnt["l2_dropped"] == len(drop) and cnt["l2_dropped_dirty"] == sum(dirty2[k] for k, _ in drop)
        l2_hits += len(hits2); promoted += cnt["promoted"]; demoted += cnt["demoted"]
        bypass += cnt["l2_bypass"]; dropped += cnt["l2_dropped"]; ev2_total += len(out)
        # a promoted row takes its dirty byte along
        for k, s1 in miss:
            if k in hits2 and dirty2[k]:
                assert l1.dirty[s1] == 1
        # exclusivity and the state of the second level
        t1 = set(l1.tags[l1.tags >= 0].tolist()); t2 = l2.tags[l2.tags >= 0].tolist()
        assert len(t2) == len(set(t2)) and not (t1 & set(t2))
        for s in range(S2):
            for e in sim2.sets[s]:
                sl = s * ways + e[0]
                assert int(l2.tags.reshape(-1)[sl]) == e[1] and int(l2.ts.reshape(-1)[sl]) == e[2]
                assert int(l2.dirty[sl]) == e[3] and int(l2.freq.reshape(-1)[sl]) == e[4]
        # the backward pass dirties every first-level slot the batch used (all three models)
        used = np.unique(res["slot_of_lookup"][res["slot_of_lookup"] >= 0])
        l1.dirty[used] = 1; one.dirty[used] = 1
        for sl in used.tolist():
            for e in sim1.sets[sl // ways]:
                if e[0] == sl % ways:
                    e[3] = 1
    assert l2_hits > 10 and promoted > 3 and promoted + dropped > 10 and demoted > 20 and ev2_total > 5
    if lock > 0 and ways <= 4:
        assert bypass + dropped > 0
    l1.close(); l2.close(); one.close()


def test_one_key_per_call_is_one_lru_of_the_combined_capacity():
    """S = 1 in both levels, one key per call, no lock window: promotion on every hit and demotion of the
    first level's LRU row make the two levels one LRU stack of w1 + w2 entries (textbook property of an
    exclusive hierarchy), compared with an OrderedDict."""
    w1, w2 = 3, 5
    l1 = oracle.Cache(1, w1, 4, wl.FP32, 0, 0, with_data=False)
    l2 = oracle.Cache(1, w2, 4, wl.FP32, 0, 0, with_data=False)
    c2 = oracle.Cache2(l1, l2)
    lru = OrderedDict()
    rng = np.random.default_rng(8)
    hits = 0
    for step, k in enumerate((rng.zipf(1.2, 600) % 14).tolist()):
        cnt = c2.lookup_insert(np.array([k], np.int64), step)["counters"]
        hit = k in lru
        assert (cnt["hit_lookups"] + cnt["l2_hit_lookups"] == 1) == hit, step
        hits += hit
        if hit:
            lru.move_to_end(k)
        else:
            if len(lru) == w1 + w2:
                victim, _ = lru.popitem(last=False)
                assert cnt["l2_evicted"] == 1
            lru[k] = True
        resident = set(l1.tags[l1.tags >= 0].tolist()) | set(l2.tags[l2.tags >= 0].tolist())
        assert resident == set(lru)
    assert 100 < hits < 590
    l1.close(); l2.close()


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("S1,S2,lock", [(1, 1, 0), (2, 3, 1), (3, 2, 2), (3, 1, 1)])
def test_two_level_cache_is_transparent(dtype, S1, S2, lock):
    """Weights in the store (after flushing both levels) and the Adagrad states after K batches are
    bit-identical to the uncached run: pins promotion, demotion, both evictions, the dropped and the
    bypassing rows and the dirty bytes that travel with the rows."""
    spec = small_spec(T=2, rows=(90, 60), dims=(8, 8), B=6, pooling=4.0, dtype=dtype, alpha=1.1, seed=6)
    W_ref = wl.all_weights_numpy(spec); m_ref = np.zeros(int(spec.row_offset[-1]), np.float32)
    store = W_ref.copy(); m = m_ref.copy()
    l1 = oracle.Cache(S1, 4, 8, dtype, 0, lock)
    l2 = oracle.Cache(S2, 4, 8, dtype, 0, lock)
    c2 = oracle.Cache2(l1, l2)
    args = (spec.dtype, spec.dims, spec.out_offset[:-1], spec.weight_offset[:-1])
    B = spec.batch
    tot = dict.fromkeys(oracle.COUNTER_NAMES2, 0)
    for k in range(16):
        idx, off = wl.gen_batch(spec, k)
        grad = wl.gen_grad(spec, k)
        o_ref = oracle.tbe_forward(*args, W_ref, B, idx, off)
        oracle.tbe_backward_rowwise_adagrad(*args, spec.row_offset, W_ref, m_ref, B, idx, off, grad, 0.01, 1e-8)
        keys = np.concatenate([spec.row_offset[t] + idx[off[t * B]:off[(t + 1) * B]] for t in range(2)])
        res = c2.lookup_insert(keys, k)
        for name, v in res["counters"].items():
            tot[name] += v
        c2.move(store, res)
        cd = [l1.data, l1.data]; dirty = [l1.dirty, l1.dirty]
        o = oracle.tbe_forward(*args, store, B, idx, off, 0, res["slot_of_lookup"], cd)
        oracle.tbe_backward_rowwise_adagrad(*args, spec.row_offset, store, m, B, idx, off, grad, 0.01, 1e-8,
                                            0, res["slot_of_lookup"], cd, dirty)
        np.testing.assert_array_equal(o, o_ref)
    c2.flush(store)
    assert (l1.dirty == 0).all() and (l2.dirty == 0).all()
    np.testing.assert_array_equal(store.view(np.uint8), W_ref.view(np.uint8))
    np.testing.assert_array_equal(m, m_ref)
    assert tot["promoted"] > 0 and tot["demoted"] > 0 and tot["l2_evicted_dirty"] > 0
    if S1 == 1:
        assert tot["overflow"] > 0
    if S2 == 1 and S1 > 1:
        assert tot["l2_bypass_dirty"] > 0          # more victims in one call than the second level's set has ways
    l1.close(); l2.close()
