"""The seeded input generators: shapes, determinism, locality range, numpy/torch twins."""
import os

import numpy as np
import torch

import oracle
from paper_2305_01515_b200 import workload as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(path):
    with open(path) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_eq4_example_printed_in_the_paper():
    """Section 4.2: 6.25 M requests/s at a 70% hit rate leave 1.875 M; 75 M leave 22.5 M."""
    for demand, hit, remain in _rows(os.path.join(GOLD, "eq4_iops_example.txt")):
        got = oracle.eq4_iops(float(demand), 1.0, 1.0, 1.0 - float(hit))
        assert abs(got - float(remain)) <= 1e-9 * float(remain)


def test_eq3_is_consistent_with_table2():
    """Table 2: doubling D at equal QPS, T, L doubles the demand (1300 -> 2600 GB/s)."""
    rows = {r[0]: [float(x) for x in r[1:]] for r in _rows(os.path.join(GOLD, "table2_eq3_consistency.txt"))}
    bw1, d1, p1, l1 = rows["model1"]; bw1p, d1p, p1p, l1p = rows["model1p"]
    qps_t = bw1 * 1e9 / oracle.eq3_bandwidth(1.0, 1.0, d1, p1, l1)        # QPS * T of model 1
    assert abs(oracle.eq3_bandwidth(qps_t, 1.0, d1p, p1p, l1p) - bw1p * 1e9) < 1e-3
    assert oracle.eq3_bandwidth(2.0, 3.0, 128, 4, 33) == 2 * 3 * 128 * 4 * 33 * 2


def test_configs_have_the_stated_shapes():
    c1 = wl.config1()
    assert c1.T == 4 and (c1.rows == 10_000).all() and (c1.dims == 64).all() and c1.batch == 512
    idx, off = wl.gen_batch(c1)
    assert len(idx) == 4 * 512 * 20 and (np.diff(off) == 20).all() and idx.max() < 10_000
    c2 = wl.config2()
    assert c2.T == 26 and (c2.rows == 1_000_000).all() and c2.weight_bytes == 6_656_000_000
    c3 = wl.config3()
    assert c3.T == 64 and set(c3.dims.tolist()) <= {64, 128, 256}
    assert (np.diff(c3.dims) >= 0).all()                      # one contiguous range per dim
    assert c3.rows.min() >= 10_000 and c3.rows.max() <= 10_000_000
    c4 = wl.config4(hbm_budget_gb=1.0)
    assert abs(c4.weight_bytes / 4e9 - 1.0) < 0.01 and c4.cached and c4.reuse_prob == 0.7
    c5 = wl.config5()
    assert c5.T == 1 and c5.rows[0] == 50_000_000


def test_batches_are_reproducible_and_in_range():
    spec = wl.config2(row_scale=0.01, batch=64, tables=3)
    a = wl.gen_batch(spec, 2); b = wl.gen_batch(spec, 2)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all()
    idx, off = a
    assert off[0] == 0 and off[-1] == len(idx) and (np.diff(off) >= 0).all() and len(off) == 3 * 64 + 1
    B = spec.batch
    for t in range(3):
        seg = idx[off[t * B]:off[(t + 1) * B]]
        assert seg.min() >= 0 and seg.max() < spec.rows[t]
    lens = np.diff(off)
    assert 25 < lens.mean() < 35


def test_zipf_locality_is_in_the_papers_range():
    """Section 3.2: most accesses come from a small share of the rows (power law)."""
    tab = wl._finish_tables([wl.TableSpec(rows=200_000, dim=8, pooling=1, alpha=0.9)], np.random.default_rng(0))[0]
    rows = wl.draw_rows(tab, np.random.default_rng(1), 400_000)
    counts = np.sort(np.bincount(rows, minlength=tab.rows))[::-1]
    share = counts[: tab.rows // 5].sum() / counts.sum()
    assert share > 0.6
    # scattered: hot rows are not neighbours
    hot = np.argsort(np.bincount(rows, minlength=tab.rows))[-50:]
    assert np.median(np.diff(np.sort(hot))) > 50


def test_temporal_reuse_stream():
    spec = wl.config4(hbm_budget_gb=0.0005, batch=32, tables=4, n_batches=12)
    s = wl.BatchStream(spec)
    seen = [set() for _ in range(spec.T)]
    fracs = []
    B = spec.batch
    for k in range(12):
        idx, off = s.next()
        if k >= 8:
            old = sum(int(np.isin(idx[off[t * B]:off[(t + 1) * B]], list(seen[t])).sum()) for t in range(spec.T))
            fracs.append(old / max(1, len(idx)))
        for t in range(spec.T):
            seen[t] |= set(idx[off[t * B]:off[(t + 1) * B]].tolist())
    assert min(fracs) > 0.6


def test_weight_generator_twins_agree_bitwise():
    for dtype in (wl.FP32, wl.FP16):
        spec = wl.ModelSpec("w", [wl.TableSpec(1000, 24, 1, 0.0), wl.TableSpec(77, 8, 1, 0.0)], dtype, 1, "fixed", seed=3)
        for t in range(2):
            a = wl.weights_numpy(spec, t)
            b = wl.weights_torch(spec, t, "cpu", chunk_rows=300).numpy()
            assert a.dtype == b.dtype and (a.view(np.uint8) == b.view(np.uint8)).all()
            sel = np.array([5, 0, 76], np.int64)
            assert (wl.weights_numpy(spec, t, sel) == a[sel]).all()
            assert np.abs(a.astype(np.float64)).max() <= 0.05 and abs(float(a.astype(np.float64).mean())) < 0.01
