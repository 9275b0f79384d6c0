"""Configurations 4 and 5 (rows in pinned host memory behind set-associative caches in HBM, Sections
5.3.1, 5.5.1-5.5.4, 5.7 of the paper) against the CPU oracle and against the uncached GPU run:

  - the 64-table, three-dim structure of configuration 4 at a reduced budget over its whole 200-batch
    stream through the pipelined trainer (both forms of the row fetch): per batch counters, slots of all
    lookups and miss / evict lists bit for bit against the oracle's tag-only simulation; after the flush,
    host weights and Adagrad states bit-identical to the GPU run without a cache, and a sample of rows
    (hottest, touched once, overflowed, untouched) replayed by the oracle from the initial weights;
  - the tag path at the sizes bench.py runs (configuration 4 at its benched budget, configuration 5 at
    50 M rows x 16 K x 50) for several batches, bit for bit against the tag-only oracle;
  - one model that keeps some tables in HBM and some behind caches, in one forward / backward launch.
"""
import copy

import numpy as np
import pytest
import torch

import oracle
from paper_2305_01515_b200 import binding as mb
from paper_2305_01515_b200 import workload as wl
from paper_2305_01515_b200.harness import DeviceModel
from paper_2305_01515_b200.pipeline import CachedTrainer
from helpers import FWD_RTOL, as_tensor, assert_close_mag, custom_spec, oracle_args, to_dev

pytestmark = pytest.mark.gpu


def _group_keys(spec, groups, idx, off):
    B = spec.batch
    return [np.concatenate([spec.row_offset[t] - spec.row_offset[t0] + idx[off[t * B]:off[(t + 1) * B]]
                            for t in range(t0, t1)]) for _, t0, t1 in groups]


LIST_KEEP = 200000      # list entries kept per batch and cache for the comparison (steady-state lists are shorter)


def _capture(model, batches, store):
    """after_backward hook: device copies of what the tag step of batch t produced."""
    def hook(t):
        cx = model.ctx[t % DeviceModel.N_CTX]
        n = batches[t][0].numel()
        rec = {"slot": cx["slot"][:n].clone()}
        for g, L in enumerate(cx["lists"]):
            for k in ("miss_keys", "miss_slots", "evict_keys", "evict_slots", "evict_dirty", "counters"):
                rec[(g, k)] = L[k].clone() if k == "counters" else L[k][:min(L["capacity"], LIST_KEEP)].clone()
        store.append(rec)
    return hook


def test_config4_structure_200_batches_pipelined():
    K = 200
    spec = wl.config4(hbm_budget_gb=1.0, batch=1024, n_batches=K)            # 64 tables, 3 dims, 4 GB of host rows
    assert spec.T == 64 and len(spec.dim_groups()) == 3
    stream = wl.BatchStream(spec)
    host_batches = [stream.next() for _ in range(K)]
    n_max = max(len(b[0]) for b in host_batches)
    grads_h = [wl.gen_grad(spec, k) for k in range(4)]
    grads = [to_dev(g) for g in grads_h]
    glist = [grads[k % 4] for k in range(K)]
    batches = [(to_dev(i), to_dev(o), o) for i, o in host_batches]
    groups = spec.dim_groups()

    # GPU without a cache: the same tables in HBM
    plain_spec = copy.deepcopy(spec); plain_spec.cached = False
    plain = DeviceModel(plain_spec, max_lookups=n_max)
    for k in range(K):
        i, o, _ = batches[k]
        plain.backward(i, o, i.numel(), glist[k])
    torch.cuda.synchronize()
    W_plain = plain.dev_weights.clone()
    m_plain = plain.momentum.clone()
    plain.close()
    del plain

    # oracle, tags only
    ocaches = []
    for dim, t0, t1 in groups:
        rows_g = int(spec.row_offset[t1] - spec.row_offset[t0])
        ocaches.append(oracle.Cache(wl.cache_sets_for(rows_g, spec.cache_fraction), 32, dim, spec.dtype, 0, 2, with_data=False))
    refs = []
    overflow_keys = [set() for _ in groups]
    for k, (idx, off) in enumerate(host_batches):
        per = []
        for g, keys in enumerate(_group_keys(spec, groups, idx, off)):
            res = ocaches[g].lookup_insert(keys, k)
            used = res["slot_of_lookup"][res["slot_of_lookup"] >= 0]
            ocaches[g].dirty[used] = 1                    # the backward dirties every slot it updates
            overflow_keys[g].update(np.unique(keys[res["slot_of_lookup"] < 0]).tolist())
            per.append(res)
        refs.append(per)
    for oc in ocaches:
        oc.close()

    for host_gather in (False, True):
        model = DeviceModel(spec, lock_depth=2, max_lookups=n_max)
        tr = CachedTrainer(model, pipelined=True, host_gather=host_gather)
        got = []
        tr.run(batches, glist, after_backward=_capture(model, batches, got))
        model.flush()
        torch.cuda.synchronize()
        assert all(c.status() == 0 for c in model.caches) and model.tables.status() == 0
        B = spec.batch
        for k in range(K):
            off = host_batches[k][1]
            for g, (dim, t0, t1) in enumerate(groups):
                ref = refs[k][g]
                cnt = dict(zip(mb.COUNTER_NAMES, got[k][(g, "counters")].cpu().tolist()))
                assert cnt == ref["counters"], (host_gather, k, g)
                assert (tr.history[k][g] == got[k][(g, "counters")].cpu().numpy()).all()
                lo, hi = int(off[t0 * B]), int(off[t1 * B])
                np.testing.assert_array_equal(got[k]["slot"][lo:hi].cpu().numpy(), ref["slot_of_lookup"])
                nm, ne = min(cnt["inserted"], LIST_KEEP), min(cnt["evicted"], LIST_KEEP)
                np.testing.assert_array_equal(got[k][(g, "miss_keys")][:nm].cpu().numpy(), ref["miss_keys"][:nm])
                np.testing.assert_array_equal(got[k][(g, "miss_slots")][:nm].cpu().numpy(), ref["miss_slots"][:nm])
                np.testing.assert_array_equal(got[k][(g, "evict_keys")][:ne].cpu().numpy(), ref["evict_keys"][:ne])
                np.testing.assert_array_equal(got[k][(g, "evict_slots")][:ne].cpu().numpy(), ref["evict_slots"][:ne])
                np.testing.assert_array_equal(got[k][(g, "evict_dirty")][:ne].cpu().numpy(), ref["evict_dirty"][:ne])
        del got
        # transparency: bit-identical to the GPU run without a cache
        W_cached = model.host_weights.to("cuda:0")
        assert torch.equal(model.momentum.view(torch.int32), m_plain.view(torch.int32)), f"states, host_gather={host_gather}"
        if not torch.equal(W_cached.view(torch.int16), W_plain.view(torch.int16)):
            report = []
            for g, (dim, t0, t1) in enumerate(groups):
                a, b = int(spec.weight_offset[t0]), int(spec.weight_offset[t1])
                bad = (W_cached[a:b].view(-1, dim) != W_plain[a:b].view(-1, dim)).any(dim=1).nonzero().flatten().cpu().numpy()
                in_ovf = sum(1 for k in bad.tolist() if k in overflow_keys[g])
                report.append(f"group {g} (dim {dim}): {len(bad)} rows differ, {in_ovf} of them overflowed at some batch; "
                              f"first keys {bad[:8].tolist()}")
            raise AssertionError(f"weights differ from the uncached run, host_gather={host_gather}: " + "; ".join(report))
        del W_cached
        model.close()
        del model, tr

    # oracle replay of sampled rows over the 200 batches, from the counter-based initial weights
    rng = np.random.default_rng(4)
    W_plain_h = W_plain.cpu().numpy()
    m_plain_h = m_plain.cpu().numpy()
    B = spec.batch
    for g, (dim, t0, t1) in enumerate(groups):
        for t in (t0, (t0 + t1) // 2, t1 - 1):
            rows_t = int(spec.rows[t])
            counts = np.zeros(rows_t, np.int64)
            for idx, off in host_batches:
                counts += np.bincount(idx[off[t * B]:off[(t + 1) * B]], minlength=rows_t)
            parts = [np.argsort(counts)[-3:]]
            for sel, n in ((counts == 1, 20), (counts > 1, 20), (counts == 0, 5)):
                pool = np.nonzero(sel)[0]
                if len(pool):
                    parts.append(rng.choice(pool, min(n, len(pool)), replace=False))
            base_key = int(spec.row_offset[t] - spec.row_offset[t0])
            ov = [k - base_key for k in overflow_keys[g] if base_key <= k < base_key + rows_t]
            if ov:
                parts.append(np.array(ov[:20], np.int64))
            sample = np.unique(np.concatenate(parts))
            Wsub = wl.weights_numpy(spec, t, sample).reshape(-1)
            msub = np.zeros(len(sample), np.float32)
            mag_total = np.zeros(Wsub.size, np.float64)
            for k, (idx, off) in enumerate(host_batches):
                seg = idx[off[t * B]:off[(t + 1) * B]]
                keep = np.isin(seg, sample)
                if not keep.any():
                    continue
                lens = np.diff(off[t * B:(t + 1) * B + 1])
                bag_of = np.repeat(np.arange(B), lens)
                sub_idx = np.searchsorted(sample, seg[keep])
                sub_off = np.concatenate([[0], np.cumsum(np.bincount(bag_of[keep], minlength=B))]).astype(np.int64)
                gk = np.ascontiguousarray(grads_h[k % 4][:, spec.out_offset[t]:spec.out_offset[t + 1]])
                smag = np.zeros(Wsub.size, np.float64)
                W_before = np.abs(Wsub.astype(np.float64))
                oracle.tbe_backward_rowwise_adagrad(spec.dtype, [dim], [0], [0], [0, len(sample)], Wsub, msub, B, sub_idx,
                                                    sub_off, gk, spec.lr, spec.eps, step_mag=smag)
                touched = smag.reshape(len(sample), dim).any(axis=1).repeat(dim)
                mag_total += np.where(touched, W_before + smag, 0.0)
            a = int(spec.weight_offset[t])
            got_w = W_plain_h[a:a + rows_t * dim].reshape(rows_t, dim)[sample].reshape(-1)
            got_m = m_plain_h[int(spec.row_offset[t]) + sample]
            # 200 steps without resynchronising the two sides: the per-step bound rtol * (|W| + step) adds up
            # over the steps that touched the row
            assert_close_mag(got_w, Wsub, mag_total, FWD_RTOL[spec.dtype], f"cfg4 replay table {t} weights")
            assert_close_mag(got_m, msub, msub * 4.0, 1e-5, f"cfg4 replay table {t} momentum")
            untouched = counts[sample] == 0
            assert (got_w.reshape(len(sample), dim)[untouched] == wl.weights_numpy(spec, t, sample[untouched])).all()


def _tag_path_at_size(spec, n_batches, lock=2):
    """lookup_insert of every cache group for `n_batches` batches through the C ABI, from the batch's sparse
    input, against the tag-only oracle.  Row data is never touched, so the host tier is not allocated."""
    groups = spec.dim_groups()
    dummy = torch.zeros(64, dtype=torch.float16, device="cuda:0")
    dummy_h = torch.zeros(64, dtype=torch.float16).pin_memory()
    cache_id = np.zeros(spec.T, np.int32)
    for g, (_, t0, t1) in enumerate(groups):
        cache_id[t0:t1] = g
    mom = torch.zeros(1, dtype=torch.float32, device="cuda:0")
    tables = mb.tables_create(spec.dtype, spec.rows, spec.dims, spec.weight_offset[:-1], cache_id, dummy, dummy_h, mom)
    stream = wl.BatchStream(spec)
    B = spec.batch
    gc, oc = [], []
    for dim, t0, t1 in groups:
        rows_g = int(spec.row_offset[t1] - spec.row_offset[t0])
        S = wl.cache_sets_for(rows_g, spec.cache_fraction)
        gc.append(mb.cache_create(S, rows_g, dim, spec.dtype, mb.POLICY_LRU, lock))
        oc.append(oracle.Cache(S, 32, dim, spec.dtype, 0, lock, with_data=False))
    bufs = None
    for k in range(n_batches):
        idx, off = stream.next()
        N = len(idx)
        if bufs is None or bufs["n"] < N:
            n = int(N * 1.1)
            d = "cuda:0"
            wsb = max(mb.cache_workspace_bytes(c, n) for c in gc)
            bufs = dict(n=n, slot=torch.empty(n, dtype=torch.int32, device=d), mk=torch.empty(n, dtype=torch.int64, device=d),
                        ms=torch.empty(n, dtype=torch.int32, device=d), ek=torch.empty(n, dtype=torch.int64, device=d),
                        es=torch.empty(n, dtype=torch.int32, device=d), ed=torch.empty(n, dtype=torch.uint8, device=d),
                        ok=torch.empty(n, dtype=torch.int64, device=d), cnt=torch.empty(mb.NUM_COUNTERS, dtype=torch.int64, device=d),
                        srow=torch.empty(n, dtype=torch.int32, device=d), sbag=torch.empty(n, dtype=torch.int32, device=d),
                        sslot=torch.empty(n, dtype=torch.int32, device=d), ws=torch.empty(wsb, dtype=torch.uint8, device=d), wsb=wsb)
        d_idx, d_off = to_dev(idx), to_dev(off)
        keys_all = _group_keys(spec, groups, idx, off)
        for g, (dim, t0, t1) in enumerate(groups):
            lo, hi = int(off[t0 * B]), int(off[t1 * B])
            mb.cache_lookup_insert_tables(gc[g], tables, t0, t1, B, d_idx, d_off, lo, hi - lo, k, bufs["slot"], bufs["mk"],
                                          bufs["ms"], bufs["ek"], bufs["es"], bufs["ed"], bufs["n"], bufs["ok"], bufs["n"],
                                          bufs["cnt"], bufs["ws"], bufs["wsb"], sorted_rows_out=bufs["srow"],
                                          sorted_bag_out=bufs["sbag"], sorted_slot_out=bufs["sslot"])
            torch.cuda.synchronize()
            ref = oc[g].lookup_insert(keys_all[g], k)
            cnt = dict(zip(mb.COUNTER_NAMES, bufs["cnt"].cpu().tolist()))
            assert cnt == ref["counters"], (k, g)
            np.testing.assert_array_equal(bufs["slot"][lo:hi].cpu().numpy(), ref["slot_of_lookup"])
            nm, ne = cnt["inserted"], cnt["evicted"]
            np.testing.assert_array_equal(bufs["mk"][:nm].cpu().numpy(), ref["miss_keys"])
            np.testing.assert_array_equal(bufs["ms"][:nm].cpu().numpy(), ref["miss_slots"])
            np.testing.assert_array_equal(bufs["ek"][:ne].cpu().numpy(), ref["evict_keys"])
            np.testing.assert_array_equal(bufs["es"][:ne].cpu().numpy(), ref["evict_slots"])
            np.testing.assert_array_equal(bufs["ed"][:ne].cpu().numpy(), ref["evict_dirty"])
            # the backward would dirty every slot of the batch
            used = np.unique(ref["slot_of_lookup"][ref["slot_of_lookup"] >= 0])
            oc[g].dirty[used] = 1
            ones = torch.ones(len(used), dtype=torch.uint8, device="cuda:0")
            as_tensor(gc[g].dirty_ptr, gc[g].num_sets * 32, torch.uint8)[to_dev(used.astype(np.int64))] = ones
            # the exported order: linear row ids ascending, equal rows by position, with the bag and the slot of
            # every lookup in that order
            srow = bufs["srow"][lo:hi].cpu().numpy().view(np.uint32).astype(np.int64)
            lin = keys_all[g] + int(spec.row_offset[t0])
            order = np.argsort(lin, kind="stable")
            np.testing.assert_array_equal(srow, lin[order])
            bag_of = np.repeat(np.arange(t0 * B, t1 * B), np.diff(off[t0 * B:t1 * B + 1]))
            np.testing.assert_array_equal(bufs["sbag"][lo:hi].cpu().numpy().view(np.uint32).astype(np.int64), bag_of[order])
            np.testing.assert_array_equal(bufs["sslot"][lo:hi].cpu().numpy(), ref["slot_of_lookup"][order])
        assert tables.status() == 0
    for c in gc:
        assert c.status() == 0
        c.destroy()
    for c in oc:
        c.close()
    tables.destroy()


def test_config4_tag_path_at_bench_size():
    _tag_path_at_size(wl.config4(hbm_budget_gb=wl.BENCH_CFG4_BUDGET_GB, n_batches=5), 5)


def test_config5_tag_path_at_bench_size():
    spec = wl.config5(n_batches=6)
    spec.reuse_prob, spec.reuse_window = 0.0, 0
    _tag_path_at_size(spec, 6)


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
def test_model_mixing_hbm_and_cached_tables(dtype):
    """Tables 0, 3, 4 live in HBM, tables 1, 2 (dim 64) and 5 (dim 128) behind two caches; forward and backward
    each run as ONE launch over all six tables.  Every step against the oracle, the whole run against the
    all-HBM GPU run bit for bit."""
    rows, dims = [3000, 1500, 800, 2000, 500, 4000], [64, 64, 64, 128, 256, 128]
    host_tables = [False, True, True, False, False, True]
    spec = custom_spec(rows, dims, 96, dtype, [6, 10, 4, 8, 3, 12], [1.05, 0.9, 1.2, 1.0, 0.0, 1.1], seed=23)
    spec.cache_fraction = 0.05
    W0 = wl.all_weights_numpy(spec)
    mixed = DeviceModel(spec, weights=W0, lock_depth=0, host_tables=host_tables)
    plain = DeviceModel(spec, weights=W0)
    assert [(d, a, b) for d, a, b in mixed.groups] == [(64, 1, 3), (128, 5, 6)]
    W_ref = W0.copy(); m_ref = np.zeros(int(spec.row_offset[-1]), np.float32)
    overflow = 0
    for k in range(8):
        idx, off = wl.gen_batch(spec, k)
        grad = wl.gen_grad(spec, k)
        N = len(idx)
        d_idx, d_off, d_grad = to_dev(idx), to_dev(off), to_dev(grad)
        mixed.reserve(N)
        mixed.cache_step(d_idx, d_off, off, k)
        o_mixed = mixed.forward(d_idx, d_off, N)
        o_plain = plain.forward(d_idx, d_off, N)
        assert torch.equal(o_mixed, o_plain)
        ref, mag = oracle.tbe_forward(*oracle_args(spec), W_ref, spec.batch, idx, off, 0, want_mag=True)
        assert_close_mag(o_mixed.cpu().numpy(), ref, mag, FWD_RTOL[dtype], f"mixed forward {k}")
        mixed.backward(d_idx, d_off, N, d_grad)
        plain.backward(d_idx, d_off, N, d_grad)
        W_before = W_ref.copy()
        smag = np.zeros(W_ref.size, np.float64)
        oracle.tbe_backward_rowwise_adagrad(*oracle_args(spec), spec.row_offset, W_ref, m_ref, spec.batch, idx, off,
                                            grad, spec.lr, spec.eps, step_mag=smag)
        overflow += sum(int(L["counters"][mb.COUNTER_NAMES.index("overflow")].item()) for L in mixed.lists)
        # keep the trajectories together
        plain_w = plain.weights_numpy()
        assert_close_mag(plain_w, W_ref, np.abs(W_before.astype(np.float64)) + smag, FWD_RTOL[dtype], f"mixed weights {k}")
        assert_close_mag(plain.momentum.cpu().numpy(), m_ref, m_ref, 1e-5, f"mixed momentum {k}")
        W_ref = plain_w.copy(); m_ref = plain.momentum.cpu().numpy().copy()
    mixed.flush()
    torch.cuda.synchronize()
    assert overflow > 0
    assert (mixed.weights_numpy().view(np.uint8) == plain.weights_numpy().view(np.uint8)).all()
    assert torch.equal(mixed.momentum, plain.momentum)
    mixed.close(); plain.close()
