"""GPU cache (tag/state lookup, LRU/LFU replacement, data movement) vs the CPU oracle: slots,
lists, counters and exported state must match bit for bit; data must match after flush."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_01515_b200 import binding as mb
from paper_2305_01515_b200 import workload as wl
from paper_2305_01515_b200.harness import DeviceModel
from helpers import FWD_RTOL, as_tensor, assert_close_mag, custom_spec, oracle_args, to_dev

pytestmark = pytest.mark.gpu


class GpuCache:
    def __init__(self, S, key_space, dim, dtype, policy, lock, cap):
        self.c = mb.cache_create(S, key_space, dim, dtype, policy, lock)
        d = "cuda:0"
        self.cap = cap
        self.slot = torch.empty(cap, dtype=torch.int32, device=d)
        self.mk = torch.empty(cap, dtype=torch.int64, device=d); self.ms = torch.empty(cap, dtype=torch.int32, device=d)
        self.ek = torch.empty(cap, dtype=torch.int64, device=d); self.es = torch.empty(cap, dtype=torch.int32, device=d)
        self.ed = torch.empty(cap, dtype=torch.uint8, device=d)
        self.cnt = torch.empty(mb.NUM_COUNTERS, dtype=torch.int64, device=d)
        self.ok = torch.empty(cap, dtype=torch.int64, device=d)
        self.wsb = mb.cache_workspace_bytes(self.c, cap)
        self.ws = torch.empty(self.wsb, dtype=torch.uint8, device=d)
        self.n = S * 32

    def lookup_insert(self, keys, step, list_capacity=None):
        N = len(keys)
        mb.cache_lookup_insert(self.c, to_dev(keys) if N else None, N, step, self.slot, self.mk, self.ms, self.ek,
                               self.es, self.ed, self.cap if list_capacity is None else list_capacity, self.cnt,
                               self.ws, self.wsb, overflow_keys=self.ok)
        torch.cuda.synchronize()
        cnt = dict(zip(mb.COUNTER_NAMES, self.cnt.cpu().tolist()))
        nm, ne = cnt["inserted"], cnt["evicted"]
        self.overflow_keys = np.sort(self.ok[:min(cnt["overflow"], self.cap if list_capacity is None else list_capacity)].cpu().numpy())
        return dict(slot_of_lookup=self.slot[:N].cpu().numpy(), miss_keys=self.mk[:nm].cpu().numpy(),
                    miss_slots=self.ms[:nm].cpu().numpy(), evict_keys=self.ek[:ne].cpu().numpy(),
                    evict_slots=self.es[:ne].cpu().numpy(), evict_dirty=self.ed[:ne].cpu().numpy(), counters=cnt)

    def state(self):
        d = "cuda:0"
        tags = torch.empty(self.n, dtype=torch.int64, device=d); ts = torch.empty_like(tags); fr = torch.empty_like(tags)
        dirty = torch.empty(self.n, dtype=torch.uint8, device=d)
        mb.cache_export_state(self.c, tags, ts, fr, dirty)
        torch.cuda.synchronize()
        return tags.cpu().numpy(), ts.cpu().numpy(), fr.cpu().numpy(), dirty.cpu().numpy()


def _compare(res, ref):
    assert res["counters"] == ref["counters"]
    for k in ("slot_of_lookup", "miss_keys", "miss_slots", "evict_keys", "evict_slots", "evict_dirty"):
        np.testing.assert_array_equal(res[k], ref[k], err_msg=k)


@pytest.mark.parametrize("S,lock,policy,universe", [(1, 0, 0, 60), (5, 0, 0, 400), (64, 1, 0, 5000),
                                                    (3, 2, 0, 300), (64, 0, 1, 4000), (1000, 1, 0, 200000)])
def test_tag_path_matches_oracle_bit_for_bit(S, lock, policy, universe):
    rng = np.random.default_rng(S + 7 * lock + policy)
    cap = 20000
    g = GpuCache(S, universe, 64, wl.FP16, policy, lock, cap)
    o = oracle.Cache(S, 32, 64, wl.FP16, policy, lock, with_data=False)
    for step in range(25):
        n = int(rng.integers(0, min(cap, 40 * S * 4) + 2))
        keys = (rng.zipf(1.2, n) * 7919 % universe).astype(np.int64)
        if step == 3:
            keys = np.zeros(0, np.int64)                       # empty batch
        res = g.lookup_insert(keys, step)
        ref = o.lookup_insert(keys, step)
        _compare(res, ref)
        np.testing.assert_array_equal(g.overflow_keys, np.unique(keys[ref["slot_of_lookup"] < 0]))
        # the backward pass would dirty the batch's slots: mark every second placed slot on both sides
        sl = np.unique(ref["slot_of_lookup"][ref["slot_of_lookup"] >= 0])[::2]
        if len(sl):
            o.dirty[sl] = 1
            ones = torch.ones(len(sl), dtype=torch.uint8, device="cuda:0")
            dirty_t = as_tensor(g.c.dirty_ptr, g.n, torch.uint8)
            dirty_t[to_dev(sl.astype(np.int64))] = ones
        tags, ts, fr, dirty = g.state()
        np.testing.assert_array_equal(tags, o.tags.reshape(-1))
        np.testing.assert_array_equal(ts, o.ts.reshape(-1))
        np.testing.assert_array_equal(fr, o.freq.reshape(-1))
        np.testing.assert_array_equal(dirty, o.dirty)
    o.close()
    g.c.destroy()


def _scattered_keys(rng, n, universe):
    """Skewed keys spread over the whole key range (every digit of the sort sees many values)."""
    hot = rng.zipf(1.15, n).astype(np.uint64)
    spread = (hot * np.uint64(0x9E3779B97F4A7C15) >> np.uint64(11)) % np.uint64(universe)
    fresh = rng.integers(0, universe, n).astype(np.uint64)
    return np.where(rng.random(n) < 0.8, spread, fresh).astype(np.int64)


@pytest.mark.parametrize("S,universe,cap", [(300, 1 << 20, 60000), (5000, 3 << 20, 60000), (1, 131072, 60000),
                                            (70000, 100_000_000, 400000), (1 << 17, 1_000_000_000, 60000),
                                            (2500, (1 << 32) - 2, 300000), (64, 500, 60000)])
def test_tag_path_wide_keys_and_set_counts(S, universe, cap):
    """Key ranges of 9 to 32 bits and set counts of 0 to 17 bits: every digit width and pass count of the
    key sort and of the sort by set (one pass of 8 or 9 bits, two of 7 to 11, three of 9 to 11)."""
    rng = np.random.default_rng(S % 1000 + universe % 1000)
    g = GpuCache(S, universe, 8, wl.FP16, 0, 1, cap)
    o = oracle.Cache(S, 32, 8, wl.FP16, 0, 1, with_data=False)
    for step in range(6):
        n = int(rng.integers(cap // 2, cap))
        keys = _scattered_keys(rng, n, universe)
        res = g.lookup_insert(keys, step)
        ref = o.lookup_insert(keys, step)
        _compare(res, ref)
        np.testing.assert_array_equal(g.overflow_keys, np.unique(keys[ref["slot_of_lookup"] < 0]))
    tags, ts, fr, dirty = g.state()
    np.testing.assert_array_equal(tags, o.tags.reshape(-1))
    np.testing.assert_array_equal(ts, o.ts.reshape(-1))
    assert g.c.status() == 0
    o.close()
    g.c.destroy()


@pytest.mark.parametrize("policy", [0, 1])
def test_full_miss_list_is_served_as_overflow(policy):
    """list_capacity smaller than the placements of a call: the surplus keys are not inserted (slot -1), their
    victims keep their ways, counters / lists / state equal the oracle's, and the status word says so."""
    S, universe, cap = 40, 30000, 8000
    rng = np.random.default_rng(5 + policy)
    g = GpuCache(S, universe, 64, wl.FP16, policy, 1, cap)
    o = oracle.Cache(S, 32, 64, wl.FP16, policy, 1, with_data=False)
    twin = oracle.Cache(S, 32, 64, wl.FP16, policy, 1, with_data=False)
    cut_calls = 0
    for step in range(12):
        keys = _scattered_keys(rng, int(rng.integers(2000, cap)), universe)
        limit = int(rng.choice([0, 1, 7, 200, 255, 256, 257, 600, cap]))
        # what the call would place without a limit (on a copy of the oracle's state)
        twin.tags[:], twin.ts[:], twin.freq[:], twin.dirty[:] = o.tags, o.ts, o.freq, o.dirty
        wanted = twin.lookup_insert(keys, step)["counters"]["inserted"]
        res = g.lookup_insert(keys, step, list_capacity=limit)
        ref = o.lookup_insert(keys, step, list_capacity=limit)
        _compare(res, ref)
        assert res["counters"]["inserted"] == min(wanted, limit)
        if res["counters"]["overflow"] <= limit:           # the overflow list shares the capacity in this entry point
            np.testing.assert_array_equal(g.overflow_keys, np.unique(keys[ref["slot_of_lookup"] < 0]))
        status = g.c.status()
        assert (status & 4 != 0) == (wanted > limit), (status, wanted, limit)
        cut_calls += 1 if status & 4 else 0
        sl = np.unique(ref["slot_of_lookup"][ref["slot_of_lookup"] >= 0])[::2]
        if len(sl):
            o.dirty[sl] = 1
            dirty_t = as_tensor(g.c.dirty_ptr, g.n, torch.uint8)
            dirty_t[to_dev(sl.astype(np.int64))] = torch.ones(len(sl), dtype=torch.uint8, device="cuda:0")
        tags, ts, fr, dirty = g.state()
        np.testing.assert_array_equal(tags, o.tags.reshape(-1))
        np.testing.assert_array_equal(ts, o.ts.reshape(-1))
        np.testing.assert_array_equal(fr, o.freq.reshape(-1))
        np.testing.assert_array_equal(dirty, o.dirty)
    assert cut_calls >= 4
    o.close(); twin.close()
    g.c.destroy()


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("frac,lock", [(0.02, 0), (0.3, 1)])
def test_cached_training_matches_oracle_and_is_transparent(dtype, frac, lock):
    """K cached train steps (lookup_insert, prefetch, writeback, forward, backward) vs the same
    steps in the oracle; after flush the host weights also match the oracle's uncached run."""
    rows, dims = [3000, 1500, 800, 2000], [64, 64, 128, 128]
    spec = custom_spec(rows, dims, 64, dtype, [6, 10, 4, 8], [1.05, 0.9, 1.2, 1.0], seed=21)
    spec.cached = True
    spec.cache_fraction = frac
    W0 = wl.all_weights_numpy(spec)
    # oracle, cached
    W_host = W0.copy(); m_o = np.zeros(int(spec.row_offset[-1]), np.float32)
    groups = spec.dim_groups()
    ocaches = []
    for dim, t0, t1 in groups:
        rows_g = int(spec.row_offset[t1] - spec.row_offset[t0])
        ocaches.append(oracle.Cache(wl.cache_sets_for(rows_g, frac), 32, dim, dtype, 0, lock))
    # oracle, uncached
    W_plain = W0.copy(); m_plain = np.zeros_like(m_o)
    model = DeviceModel(spec, weights=W0, lock_depth=lock)
    B = spec.batch
    es = 4 if dtype == wl.FP32 else 2
    total_overflow = 0
    for k in range(10):
        idx, off = wl.gen_batch(spec, k)
        grad = wl.gen_grad(spec, k)
        N = len(idx)
        model.reserve(N)
        d_idx, d_off = to_dev(idx), to_dev(off)
        model.cache_step(d_idx, d_off, off, k)
        out = model.forward(d_idx, d_off, N)
        model.backward(d_idx, d_off, N, to_dev(grad))
        torch.cuda.synchronize()
        # oracle side
        slot = np.full(N, -1, np.int32)
        cd = [None] * spec.T; cdirty = [None] * spec.T
        for g, (dim, t0, t1) in enumerate(groups):
            lo, hi = int(off[t0 * B]), int(off[t1 * B])
            keys = np.concatenate([spec.row_offset[t] - spec.row_offset[t0] + idx[off[t * B]:off[(t + 1) * B]]
                                   for t in range(t0, t1)]) if hi > lo else np.zeros(0, np.int64)
            res = ocaches[g].lookup_insert(keys, k)
            host_g = W_host[spec.weight_offset[t0]:spec.weight_offset[t1]]
            staging = ocaches[g].prefetch_misses(host_g, res)
            ocaches[g].writeback_evicted(host_g, res, staging)
            slot[lo:hi] = res["slot_of_lookup"]
            for t in range(t0, t1):
                cd[t] = ocaches[g].data; cdirty[t] = ocaches[g].dirty
            cnt = dict(zip(mb.COUNTER_NAMES, model.lists[g]["counters"].cpu().tolist()))
            assert cnt == res["counters"]
            total_overflow += cnt["overflow"]
            nm = cnt["inserted"]
            np.testing.assert_array_equal(model.lists[g]["miss_slots"][:nm].cpu().numpy(), res["miss_slots"])
        np.testing.assert_array_equal(model.slot_of_lookup[:N].cpu().numpy(), slot)
        ref, mag = oracle.tbe_forward(*oracle_args(spec), W_host, B, idx, off, 0, slot, cd, want_mag=True)
        assert_close_mag(out.cpu().numpy(), ref, mag, FWD_RTOL[dtype], f"cached forward {k}")
        oracle.tbe_backward_rowwise_adagrad(*oracle_args(spec), spec.row_offset, W_host, m_o, B, idx, off, grad,
                                            spec.lr, spec.eps, 0, slot, cd, cdirty)
        oracle.tbe_backward_rowwise_adagrad(*oracle_args(spec), spec.row_offset, W_plain, m_plain, B, idx, off, grad,
                                            spec.lr, spec.eps)
        # keep the trajectories together: copy the oracle's cache rows, host rows and momentum to the GPU
        W_gpu_host = model.host_weights.numpy()
        magw = np.abs(W_host.astype(np.float64)) + 1e-3
        assert_close_mag(W_gpu_host, W_host, magw, FWD_RTOL[dtype], f"host rows {k}")
        for g, oc in enumerate(ocaches):
            n_el = oc.data.size
            gt = as_tensor(model.caches[g].data_ptr, n_el, model.tdtype)
            ref_rows = oc.data.reshape(-1)
            assert_close_mag(gt.cpu().numpy(), ref_rows, np.abs(ref_rows.astype(np.float64)) + 1e-3, FWD_RTOL[dtype],
                             f"cache rows {k}")
            gt.copy_(torch.from_numpy(ref_rows))
            gd = as_tensor(model.caches[g].dirty_ptr, len(oc.dirty), torch.uint8).cpu().numpy()
            np.testing.assert_array_equal(gd, oc.dirty)
        got_m = model.momentum.cpu().numpy()
        assert_close_mag(got_m, m_o, m_o, 1e-5, f"momentum {k}")
        model.momentum.copy_(torch.from_numpy(m_o))
        model.host_weights.copy_(torch.from_numpy(W_host))
    model.flush()
    torch.cuda.synchronize()
    for oc, (dim, t0, t1) in zip(ocaches, groups):
        oc.flush(W_host[spec.weight_offset[t0]:spec.weight_offset[t1]])
    np.testing.assert_array_equal(model.host_weights.numpy().view(np.uint8), W_host.view(np.uint8))
    np.testing.assert_array_equal(W_host.view(np.uint8), W_plain.view(np.uint8))      # transparency (oracle)
    np.testing.assert_array_equal(m_o, m_plain)
    if frac < 0.05:
        assert total_overflow > 0          # the small cache really sent rows around the cache
    for oc in ocaches:
        oc.close()
    model.close()


@pytest.mark.parametrize("dim,dtype", [(128, wl.FP16), (8, wl.FP16), (1024, wl.FP32)])
def test_gpu_cached_run_equals_gpu_uncached_run_bitwise(dim, dtype):
    """Transparency on the GPU alone: cached and uncached training give identical bits (rows of
    256 B, of 16 B and of 4 KB go through the bulk-copy fetch)."""
    rows, dims = [5000, 2500], [dim, dim]
    spec = custom_spec(rows, dims, 128, dtype, [8, 12], [1.05, 1.1], seed=33)
    W0 = wl.all_weights_numpy(spec)
    plain = DeviceModel(spec, weights=W0)
    import copy
    cspec = copy.deepcopy(spec); cspec.cached = True; cspec.cache_fraction = 0.05
    cached = DeviceModel(cspec, weights=W0, lock_depth=0)
    for k in range(8):
        idx, off = wl.gen_batch(spec, k)
        grad = to_dev(wl.gen_grad(spec, k))
        N = len(idx)
        d_idx, d_off = to_dev(idx), to_dev(off)
        cached.reserve(N)
        cached.cache_step(d_idx, d_off, off, k)
        o1 = cached.forward(d_idx, d_off, N)
        o0 = plain.forward(d_idx, d_off, N)
        assert torch.equal(o0, o1)
        cached.backward(d_idx, d_off, N, grad)
        plain.backward(d_idx, d_off, N, grad)
    cached.flush()
    torch.cuda.synchronize()
    assert all(c.status() == 0 for c in cached.caches)
    assert (cached.weights_numpy().view(np.uint8) == plain.weights_numpy().view(np.uint8)).all()
    assert torch.equal(cached.momentum, plain.momentum)
    plain.close(); cached.close()
