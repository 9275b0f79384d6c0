"""Pins for the oracle's pooled lookup (Section 2.1.1: select rows of a table and pool them)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_01515_b200 import workload as wl
from helpers import small_spec, storage_dtype


def _problem(spec, k=0):
    W = wl.all_weights_numpy(spec)
    idx, off = wl.gen_batch(spec, k)
    return W, idx, off


def _oracle_fwd(spec, W, idx, off, mode=0, **kw):
    return oracle.tbe_forward(spec.dtype, spec.dims, spec.out_offset[:-1], spec.weight_offset[:-1], W,
                              spec.batch, idx, off, mode, **kw)


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_forward_vs_python_loops(dtype, mode):
    """Brute force on a tiny input: explicit loops over bags, rows and columns."""
    spec = small_spec(dtype=dtype)
    W, idx, off = _problem(spec)
    out = _oracle_fwd(spec, W, idx, off, mode)
    B = spec.batch
    for t in range(spec.T):
        D = int(spec.dims[t])
        base = int(spec.weight_offset[t])
        for b in range(B):
            lo, hi = int(off[t * B + b]), int(off[t * B + b + 1])
            for d in range(D):
                s = 0.0
                for i in range(lo, hi):
                    w = float(W[base + int(idx[i]) * D + d])
                    s = (w if i == lo else max(s, w)) if mode == 2 else s + w
                if mode == 1 and hi > lo:
                    s /= (hi - lo)
                assert out[b, spec.out_offset[t] + d] == np.float32(s)


@pytest.mark.parametrize("mode", ["sum", "mean", "max"])
def test_forward_vs_torch_embedding_bag(mode):
    """Special case that is a library routine: per table, torch's embedding_bag in fp64."""
    spec = small_spec(T=3, rows=(50, 31, 17), dims=(16, 8, 32), B=9, pooling=4.0, dtype=wl.FP16, seed=3)
    W, idx, off = _problem(spec)
    out = _oracle_fwd(spec, W, idx, off, {"sum": 0, "mean": 1, "max": 2}[mode])
    B = spec.batch
    for t in range(spec.T):
        D = int(spec.dims[t])
        Wt = torch.from_numpy(W[spec.weight_offset[t]:spec.weight_offset[t + 1]].astype(np.float64)).view(-1, D)
        lo, hi = int(off[t * B]), int(off[(t + 1) * B])
        o = torch.from_numpy(off[t * B:(t + 1) * B] - lo)
        ref = torch.nn.functional.embedding_bag(torch.from_numpy(idx[lo:hi]), Wt, o, mode=mode)
        got = out[:, spec.out_offset[t]:spec.out_offset[t + 1]]
        np.testing.assert_array_equal(got, ref.numpy().astype(np.float32))


def test_forward_closed_forms():
    spec = small_spec(T=2, rows=(13, 6), dims=(4, 8), B=6, pooling=2.5, seed=5)
    idx, off = wl.gen_batch(spec, 0)
    B = spec.batch
    lens = np.diff(off)
    # all-ones table: sum pooling returns the bag length, mean pooling 1 (0 for an empty bag)
    W = np.ones(int(spec.weight_offset[-1]), np.float32)
    out = _oracle_fwd(spec, W, idx, off, 0)
    for t in range(spec.T):
        want = lens[t * B:(t + 1) * B].astype(np.float32)
        assert (out[:, spec.out_offset[t]:spec.out_offset[t + 1]] == want[:, None]).all()
    outm = _oracle_fwd(spec, W, idx, off, 1)
    for t in range(spec.T):
        want = (lens[t * B:(t + 1) * B] > 0).astype(np.float32)
        assert (outm[:, spec.out_offset[t]:spec.out_offset[t + 1]] == want[:, None]).all()
    # one-hot rows (table 0 has more rows than columns: use row r -> e_{r mod D}): histogram
    D0 = int(spec.dims[0])
    W = np.zeros(int(spec.weight_offset[-1]), np.float32)
    for r in range(int(spec.rows[0])):
        W[r * D0 + r % D0] = 1.0
    out = _oracle_fwd(spec, W, idx, off, 0)
    for b in range(B):
        h = np.bincount(idx[off[b]:off[b + 1]] % D0, minlength=D0)
        assert (out[b, :D0] == h).all()
    assert (out[:, D0:] == 0).all()


def test_forward_gather_when_pooling_is_one():
    spec = small_spec(T=2, rows=(9, 12), dims=(8, 8), B=5, pooling=1, bag_dist="fixed", seed=7)
    W, idx, off = _problem(spec)
    out = _oracle_fwd(spec, W, idx, off, 0)
    B = spec.batch
    for t in range(spec.T):
        Wt = W[spec.weight_offset[t]:spec.weight_offset[t + 1]].reshape(-1, 8)
        np.testing.assert_array_equal(out[:, 8 * t:8 * t + 8], Wt[idx[t * B:(t + 1) * B]])


def test_forward_duplicates_count_each_time_and_linearity():
    spec = small_spec(T=1, rows=(4,), dims=(4,), B=1, pooling=3, bag_dist="fixed")
    W = np.arange(16, dtype=np.float32)
    idx = np.array([2, 2, 1], np.int64)
    off = np.array([0, 3], np.int64)
    out = _oracle_fwd(spec, W, idx, off, 0)
    np.testing.assert_array_equal(out[0], 2 * W[8:12] + W[4:8])
    out2 = _oracle_fwd(spec, 3 * W, idx, off, 0)
    np.testing.assert_array_equal(out2, 3 * out)


def test_forward_mag_is_sum_of_absolute_values():
    spec = small_spec(dtype=wl.FP16, seed=11)
    W, idx, off = _problem(spec)
    out, mag = _oracle_fwd(spec, W, idx, off, 0, want_mag=True)
    outabs = _oracle_fwd(spec, np.abs(W), idx, off, 0)
    np.testing.assert_allclose(mag, outabs, rtol=1e-6)
    assert (mag + 1e-12 >= np.abs(out)).all()


def test_half_conversion_matches_numpy():
    """binary16 encode/decode against numpy's float16 (an independent implementation)."""
    for h in range(0, 1 << 16, 7):
        v = oracle.half_to_double(h)
        ref = float(np.array([h], np.uint16).view(np.float16)[0])
        assert (np.isnan(v) and np.isnan(ref)) or v == ref
    rng = np.random.default_rng(0)
    xs = np.concatenate([rng.standard_normal(3000) * 10.0 ** rng.integers(-9, 6, 3000),
                         [0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e9, -1e9, 2.0 ** -24, 2.0 ** -25,
                          2.0 ** -25 * 1.0000001, 6.1e-5, 6.103515625e-05]])
    # exact ties between neighbouring halves must go to even
    hs = rng.integers(0, 0x7bff, 2000).astype(np.uint16)
    a = hs.view(np.float16).astype(np.float64)
    b = (hs + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    xs = np.concatenate([xs, (a + b) / 2, -(a + b) / 2])
    with np.errstate(over="ignore"):
        ref = xs.astype(np.float16).view(np.uint16)
    for x, r in zip(xs, ref):
        assert oracle.double_to_half(x) == int(r), x


def test_max_pooling_closed_forms():
    """Max pooling (Section 2.1.1 names sum, mean and max): an all-negative table keeps its sign (the maximum
    is not started from 0), a bag of one row is that row, an empty bag gives 0, a repeated row changes nothing."""
    spec = small_spec(T=1, rows=(6,), dims=(4,), B=4, dtype=wl.FP32)
    W = -(np.arange(24, dtype=np.float32) + 1.0)                       # row r = -(4r+1 .. 4r+4)
    idx = np.array([2, 5, 2, 3, 0, 0, 1], np.int64)
    off = np.array([0, 3, 4, 4, 7], np.int64)                          # bags: [2,5,2], [3], [], [0,0,1]
    out, mag = _oracle_fwd(spec, W, idx, off, 2, want_mag=True)
    np.testing.assert_array_equal(out[0], W.reshape(6, 4)[2])
    np.testing.assert_array_equal(out[1], W.reshape(6, 4)[3])
    np.testing.assert_array_equal(out[2], np.zeros(4, np.float32))
    np.testing.assert_array_equal(out[3], W.reshape(6, 4)[0])
    np.testing.assert_array_equal(mag[0], np.abs(W.reshape(6, 4)[5]))    # largest magnitude seen in the bag
