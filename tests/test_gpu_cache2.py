"""Two-level exclusive cache on the GPU (first level in HBM, second level in pinned host memory, backing
store in host memory; Sections 5.3.2 and 5.5.4 of the paper) against the CPU oracle: slots, the four lists,
counters and the exported state of both levels bit for bit; after training through it and flushing, the
store and the Adagrad states bit-identical to the oracle's two-level run and to the uncached run."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_01515_b200 import binding as mb
from paper_2305_01515_b200 import workload as wl
from helpers import FWD_RTOL, as_tensor, assert_close_mag, custom_spec, oracle_args, to_dev

pytestmark = pytest.mark.gpu

LISTS = (("fetch_keys", torch.int64), ("fetch_slots", torch.int32), ("fetch_src", torch.int32),
         ("ev1_keys", torch.int64), ("ev1_slots", torch.int32), ("ev1_dirty", torch.uint8), ("ev1_dst", torch.int32),
         ("ev2_keys", torch.int64), ("ev2_slots", torch.int32), ("ev2_dirty", torch.uint8),
         ("drop_keys", torch.int64), ("drop_slots", torch.int32), ("drop_dirty", torch.uint8))


class GpuCache2:
    def __init__(self, S1, S2, key_space, dim, dtype, policy, lock, cap):
        d = "cuda:0"
        esz = 4 if dtype == wl.FP32 else 2
        self.l2_rows = torch.zeros(S2 * 32 * dim * esz, dtype=torch.uint8).pin_memory()
        self.l1 = mb.cache_create(S1, key_space, dim, dtype, policy, lock)
        self.l2 = mb.Cache(S2, key_space, dim, dtype, policy, lock, host_rows=self.l2_rows)
        self.cap = cap
        self.slot = torch.empty(cap, dtype=torch.int32, device=d)
        self.lists = {name: torch.zeros(cap, dtype=t, device=d) for name, t in LISTS}
        self.cnt = torch.empty(mb.NUM_COUNTERS2, dtype=torch.int64, device=d)
        self.wsb = mb.cache2_workspace_bytes(self.l1, self.l2, cap, cap)
        self.ws = torch.empty(self.wsb, dtype=torch.uint8, device=d)
        self.staging = torch.empty(cap * dim * esz, dtype=torch.uint8, device=d)

    def lookup_insert(self, keys, step):
        N = len(keys)
        mb.cache2_lookup_insert(self.l1, self.l2, to_dev(keys) if N else None, N, step, self.slot, self.lists, self.cap,
                                self.cnt, self.ws, self.wsb)
        torch.cuda.synchronize()
        c = dict(zip(mb.COUNTER_NAMES2, self.cnt.cpu().tolist()))
        n = {"fetch": c["inserted"], "ev1": c["evicted"], "ev2": c["l2_evicted"], "drop": c["l2_dropped"]}
        res = {name: self.lists[name][:n[name.split("_")[0]]].cpu().numpy() for name, _ in LISTS}
        res["slot_of_lookup"] = self.slot[:N].cpu().numpy()
        res["counters"] = c
        return res

    def move(self, store):
        mb.cache2_move(self.l1, self.l2, store, self.lists, self.cap, self.cnt, self.staging)

    def state(self, level):
        c = self.l1 if level == 1 else self.l2
        n = c.num_sets * 32
        d = "cuda:0"
        tags = torch.empty(n, dtype=torch.int64, device=d); ts = torch.empty_like(tags); fr = torch.empty_like(tags)
        dirty = torch.empty(n, dtype=torch.uint8, device=d)
        mb.cache_export_state(c, tags, ts, fr, dirty)
        torch.cuda.synchronize()
        return tags.cpu().numpy(), ts.cpu().numpy(), fr.cpu().numpy(), dirty.cpu().numpy()

    def close(self):
        self.l1.destroy(); self.l2.destroy()


def _compare(res, ref):
    assert res["counters"] == ref["counters"]
    for name, _ in LISTS:
        if name.startswith("drop"):
            continue
        np.testing.assert_array_equal(res[name], ref[name], err_msg=name)
    np.testing.assert_array_equal(res["slot_of_lookup"], ref["slot_of_lookup"])
    a = sorted(zip(res["drop_keys"].tolist(), res["drop_slots"].tolist(), res["drop_dirty"].tolist()))
    b = sorted(zip(ref["drop_keys"].tolist(), ref["drop_slots"].tolist(), ref["drop_dirty"].tolist()))
    assert a == b, "drop list"


@pytest.mark.parametrize("S1,S2,lock,policy,universe", [(1, 1, 0, 0, 150), (5, 9, 1, 0, 1500), (64, 40, 2, 0, 20000),
                                                        (16, 64, 1, 1, 9000), (300, 700, 1, 0, 200000)])
def test_two_level_tag_path_matches_oracle_bit_for_bit(S1, S2, lock, policy, universe):
    rng = np.random.default_rng(S1 + 3 * S2 + lock + policy)
    cap = 30000
    g = GpuCache2(S1, S2, universe, 64, wl.FP16, policy, lock, cap)
    o1 = oracle.Cache(S1, 32, 64, wl.FP16, policy, lock, with_data=False)
    o2 = oracle.Cache(S2, 32, 64, wl.FP16, policy, lock, with_data=False)
    o = oracle.Cache2(o1, o2)
    tot = dict.fromkeys(mb.COUNTER_NAMES2, 0)
    for step in range(30):
        n = int(rng.integers(0, min(cap, 60 * (S1 + S2)) + 2))
        hot = rng.zipf(1.2, n).astype(np.uint64)
        keys = ((hot * np.uint64(2654435761)) % np.uint64(universe)).astype(np.int64)
        if step == 4:
            keys = np.zeros(0, np.int64)
        res = g.lookup_insert(keys, step)
        ref = o.lookup_insert(keys, step)
        _compare(res, ref)
        for k, v in res["counters"].items():
            tot[k] += v
        # the backward pass would dirty the batch's first-level slots: every second one here, on both sides
        sl = np.unique(ref["slot_of_lookup"][ref["slot_of_lookup"] >= 0])[::2]
        if len(sl):
            o1.dirty[sl] = 1
            dirty_t = as_tensor(g.l1.dirty_ptr, S1 * 32, torch.uint8)
            dirty_t[to_dev(sl.astype(np.int64))] = torch.ones(len(sl), dtype=torch.uint8, device="cuda:0")
        for level, oc in ((1, o1), (2, o2)):
            tags, ts, fr, dirty = g.state(level)
            np.testing.assert_array_equal(tags, oc.tags.reshape(-1), err_msg=f"tags level {level}")
            np.testing.assert_array_equal(ts, oc.ts.reshape(-1), err_msg=f"timestamps level {level}")
            np.testing.assert_array_equal(fr, oc.freq.reshape(-1), err_msg=f"counts level {level}")
            np.testing.assert_array_equal(dirty, oc.dirty, err_msg=f"dirty level {level}")
        t1 = set(o1.tags[o1.tags >= 0].tolist()); t2 = set(o2.tags[o2.tags >= 0].tolist())
        assert not (t1 & t2)
    assert tot["promoted"] > 0 and tot["demoted"] > 0 and tot["l2_evicted"] > 0
    assert g.l1.status() == 0 and g.l2.status() == 0
    o1.close(); o2.close(); g.close()


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("S1,S2,lock", [(1, 1, 0), (3, 2, 1), (6, 1, 1), (10, 30, 0)])
def test_training_through_two_levels_matches_oracle_and_uncached_run(dtype, S1, S2, lock):
    """lookup_insert2 + data movement + forward + backward for 12 batches on one table group; the store, both
    levels' rows and the states follow the oracle's two-level run; after the flush the store equals the
    oracle's uncached run bit for bit (exclusive levels, dirty bytes travelling with the rows, rows that are
    dropped from the second level or bypass it)."""
    rows, dims = [2500, 1500], [64, 64]
    spec = custom_spec(rows, dims, 48, dtype, [8, 6], [1.05, 0.9], seed=31)
    W0 = wl.all_weights_numpy(spec)
    n_rows = int(spec.row_offset[-1])
    esz = 4 if dtype == wl.FP32 else 2
    tdt = torch.float32 if dtype == wl.FP32 else torch.float16
    # GPU side: store in pinned host memory, tables described as one cached group
    store = torch.from_numpy(W0.copy()).pin_memory()
    mom = torch.zeros(n_rows, dtype=torch.float32, device="cuda:0")
    cap = 4000
    g = GpuCache2(S1, S2, n_rows, 64, dtype, 0, lock, cap)
    tables = mb.tables_create(spec.dtype, spec.rows, spec.dims, spec.weight_offset[:-1], np.zeros(2, np.int32), None, store, mom)
    keys_dev = torch.empty(cap, dtype=torch.int64, device="cuda:0")
    out = torch.empty((spec.batch, spec.total_dim), dtype=torch.float32, device="cuda:0")
    wsb = mb.tbe_backward_workspace_bytes(tables, spec.batch, cap)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda:0")
    # oracle side
    W_store = W0.copy(); m_o = np.zeros(n_rows, np.float32)
    W_plain = W0.copy(); m_plain = np.zeros(n_rows, np.float32)
    o1 = oracle.Cache(S1, 32, 64, dtype, 0, lock); o2 = oracle.Cache(S2, 32, 64, dtype, 0, lock)
    o = oracle.Cache2(o1, o2)
    B = spec.batch
    tot = dict.fromkeys(mb.COUNTER_NAMES2, 0)
    for k in range(12):
        idx, off = wl.gen_batch(spec, k)
        grad = wl.gen_grad(spec, k)
        N = len(idx)
        assert N <= cap
        d_idx, d_off = to_dev(idx), to_dev(off)
        mb.linearize_keys(tables, 0, 2, B, d_idx, d_off, 0, N, keys_dev)
        mb.cache2_lookup_insert(g.l1, g.l2, keys_dev, N, k, g.slot, g.lists, cap, g.cnt, g.ws, g.wsb)
        g.move(store)
        mb.tbe_forward(tables, B, d_idx, d_off, N, mb.POOL_SUM, g.slot, [g.l1.data_ptr], out, out.shape[1])
        mb.tbe_backward_rowwise_adagrad(tables, B, d_idx, d_off, N, mb.POOL_SUM, to_dev(grad), grad.shape[1], spec.lr,
                                        spec.eps, g.slot, [g.l1.data_ptr], [g.l1.dirty_ptr], ws, wsb)
        torch.cuda.synchronize()
        # oracle
        keys = np.concatenate([spec.row_offset[t] + idx[off[t * B]:off[(t + 1) * B]] for t in range(2)])
        ref = o.lookup_insert(keys, k)
        cnt = dict(zip(mb.COUNTER_NAMES2, g.cnt.cpu().tolist()))
        assert cnt == ref["counters"], k
        for name, v in cnt.items():
            tot[name] += v
        np.testing.assert_array_equal(g.slot[:N].cpu().numpy(), ref["slot_of_lookup"])
        np.testing.assert_array_equal(g.lists["fetch_src"][:cnt["inserted"]].cpu().numpy(), ref["fetch_src"])
        np.testing.assert_array_equal(g.lists["ev1_dst"][:cnt["evicted"]].cpu().numpy(), ref["ev1_dst"])
        o.move(W_store, ref)
        cd = [o1.data, o1.data]; cdirty = [o1.dirty, o1.dirty]
        o_ref, mag = oracle.tbe_forward(*oracle_args(spec), W_store, B, idx, off, 0, ref["slot_of_lookup"], cd, want_mag=True)
        assert_close_mag(out.cpu().numpy(), o_ref, mag, FWD_RTOL[dtype], f"two-level forward {k}")
        oracle.tbe_backward_rowwise_adagrad(*oracle_args(spec), spec.row_offset, W_store, m_o, B, idx, off, grad, spec.lr,
                                            spec.eps, 0, ref["slot_of_lookup"], cd, cdirty)
        oracle.tbe_backward_rowwise_adagrad(*oracle_args(spec), spec.row_offset, W_plain, m_plain, B, idx, off, grad,
                                            spec.lr, spec.eps)
        # rows of both levels and of the store follow the oracle; then keep the two sides on one trajectory
        mag_s = np.abs(W_store.astype(np.float64)) + 1e-3
        assert_close_mag(store.numpy(), W_store, mag_s, FWD_RTOL[dtype], f"store rows {k}")
        l1_rows = as_tensor(g.l1.data_ptr, o1.data.size, tdt)
        assert_close_mag(l1_rows.cpu().numpy(), o1.data.reshape(-1), np.abs(o1.data.reshape(-1).astype(np.float64)) + 1e-3,
                         FWD_RTOL[dtype], f"first-level rows {k}")
        l2_rows = g.l2_rows.view(tdt)
        occupied = np.repeat(o2.tags.reshape(-1) >= 0, 64)
        assert_close_mag(l2_rows.numpy()[occupied], o2.data.reshape(-1)[occupied],
                         np.abs(o2.data.reshape(-1)[occupied].astype(np.float64)) + 1e-3, FWD_RTOL[dtype], f"second-level rows {k}")
        np.testing.assert_array_equal(as_tensor(g.l1.dirty_ptr, S1 * 32, torch.uint8).cpu().numpy(), o1.dirty)
        np.testing.assert_array_equal(as_tensor(g.l2.dirty_ptr, S2 * 32, torch.uint8).cpu().numpy(), o2.dirty)
        assert_close_mag(mom.cpu().numpy(), m_o, m_o, 1e-5, f"two-level momentum {k}")
        l1_rows.copy_(torch.from_numpy(o1.data.reshape(-1)))
        l2_rows.copy_(torch.from_numpy(o2.data.reshape(-1)))
        store.copy_(torch.from_numpy(W_store))
        mom.copy_(torch.from_numpy(m_o))
    mb.cache_flush(g.l1, store)
    mb.cache_flush(g.l2, store)
    torch.cuda.synchronize()
    o.flush(W_store)
    np.testing.assert_array_equal(store.numpy().view(np.uint8), W_store.view(np.uint8))
    np.testing.assert_array_equal(W_store.view(np.uint8), W_plain.view(np.uint8))          # transparency (oracle)
    np.testing.assert_array_equal(m_o, m_plain)
    assert tot["promoted"] > 0 and tot["demoted"] > 0
    if S2 == 1 and S1 > 1:
        assert tot["l2_bypass"] > 0
    if S1 == 1:
        assert tot["overflow"] > 0
    assert g.l1.status() == 0 and g.l2.status() == 0 and tables.status() == 0
    o1.close(); o2.close(); g.close(); tables.destroy()


def test_two_level_model_equals_uncached_model_bitwise():
    """Several table groups (two dims), each behind its own pair of levels, through the trainer's sequential
    schedule: after the flush the host rows and the states equal the all-HBM run bit for bit, and rows really
    travelled between the levels."""
    import copy

    from paper_2305_01515_b200.harness import DeviceModel
    from paper_2305_01515_b200.pipeline import CachedTrainer

    rows, dims = [20000, 9000, 4000, 12000], [64, 64, 128, 128]
    spec = custom_spec(rows, dims, 256, wl.FP16, [8, 12, 20, 5], [1.05, 0.9, 1.2, 1.0], seed=79)
    spec.reuse_prob, spec.reuse_window = 0.6, 4
    stream = wl.BatchStream(spec)
    K = 12
    host_batches = [stream.next() for _ in range(K)]
    grads = [to_dev(wl.gen_grad(spec, k)) for k in range(K)]
    W0 = wl.all_weights_numpy(spec)
    n_max = max(len(b[0]) for b in host_batches)
    plain = DeviceModel(spec, weights=W0, max_lookups=n_max)
    batches = [(to_dev(i), to_dev(o), o) for i, o in host_batches]
    for k in range(K):
        i, o, _ = batches[k]
        plain.backward(i, o, i.numel(), grads[k])
    cspec = copy.deepcopy(spec); cspec.cached = True; cspec.cache_fraction = 0.02
    m = DeviceModel(cspec, weights=W0, lock_depth=0, l2_fraction=0.05, max_lookups=n_max)
    tr = CachedTrainer(m, pipelined=False)
    tr.run(batches, grads)
    m.flush()
    torch.cuda.synchronize()
    hist = np.stack(tr.history)
    assert hist.shape == (K, 2, mb.NUM_COUNTERS2)
    names = mb.COUNTER_NAMES2
    assert hist[:, :, names.index("promoted")].sum() > 50 and hist[:, :, names.index("demoted")].sum() > 500
    assert hist[:, :, names.index("l2_evicted_dirty")].sum() > 0
    assert (m.weights_numpy().view(np.uint16) == plain.weights_numpy().view(np.uint16)).all()
    assert torch.equal(m.momentum, plain.momentum)
    assert all(c.status() == 0 for c in m.caches + m.l2)
    m.close(); plain.close()
