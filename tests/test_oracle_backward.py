"""Pins for the oracle's backward + row-wise Adagrad (Section 2.1.2: optimizer with few states
per row; Section 5.9: aggregate, run the optimizer, update the touched rows)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_01515_b200 import workload as wl
from helpers import small_spec


def _bwd(spec, W, m, idx, off, grad, lr=0.01, eps=1e-8, mode=0):
    return oracle.tbe_backward_rowwise_adagrad(
        spec.dtype, spec.dims, spec.out_offset[:-1], spec.weight_offset[:-1], spec.row_offset, W, m,
        spec.batch, idx, off, grad, lr, eps, mode)


def test_hand_worked_step():
    """D = 4, g = (1,2,3,4), m0 = 0, lr = 0.01, eps = 1e-8, worked by hand:
    mean(g^2) = 30/4 = 7.5, sqrt = 2.7386128, step = lr*g/sqrt; a second identical step has
    m = 15, sqrt = 3.8729833."""
    spec = small_spec(T=1, rows=(3,), dims=(4,), B=1, pooling=1, bag_dist="fixed")
    W = np.zeros(12, np.float32)
    m = np.zeros(3, np.float32)
    idx = np.array([1], np.int64); off = np.array([0, 1], np.int64)
    g = np.array([[1, 2, 3, 4]], np.float32)
    uniq = _bwd(spec, W, m, idx, off, g)
    assert list(uniq) == [1]
    assert m[1] == np.float32(7.5) and m[0] == 0 and m[2] == 0
    np.testing.assert_allclose(W[4:8], [-0.00365148, -0.00730297, -0.01095445, -0.01460593], rtol=2e-6)
    assert (W[:4] == 0).all() and (W[8:] == 0).all()
    before = W.copy()
    _bwd(spec, W, m, idx, off, g)
    assert m[1] == np.float32(15.0)
    np.testing.assert_allclose(W[4:8] - before[4:8], -0.00258199 * g[0], rtol=2e-6)


@pytest.mark.parametrize("D", [1, 4])
def test_matches_torch_adagrad_when_rowwise_equals_elementwise(D):
    """Library special case: when a row's gradient is the same in every column (always true for
    D = 1), mean(g^2) = g^2 and the row-wise rule is textbook element-wise Adagrad."""
    spec = small_spec(T=2, rows=(6, 9), dims=(D, D), B=5, pooling=2.0, seed=4)
    rng = np.random.default_rng(0)
    W = rng.standard_normal(int(spec.weight_offset[-1])).astype(np.float32)
    m = np.zeros(int(spec.row_offset[-1]), np.float32)
    params = [torch.tensor(W[spec.weight_offset[t]:spec.weight_offset[t + 1]].astype(np.float64)
                           ).view(-1, D).requires_grad_() for t in range(2)]
    opt = torch.optim.Adagrad(params, lr=float(np.float32(0.01)), lr_decay=0, weight_decay=0,
                              initial_accumulator_value=0, eps=float(np.float32(1e-8)))
    B = spec.batch
    for k in range(3):
        idx, off = wl.gen_batch(spec, k)
        col = rng.standard_normal((B, 2)).astype(np.float32)
        grad = np.repeat(col, D, axis=1)            # constant across each table's columns
        _bwd(spec, W, m, idx, off, grad)
        opt.zero_grad()
        loss = 0
        for t in range(2):
            lo, hi = int(off[t * B]), int(off[(t + 1) * B])
            o = torch.from_numpy(off[t * B:(t + 1) * B] - lo)
            pooled = torch.nn.functional.embedding_bag(torch.from_numpy(idx[lo:hi]), params[t], o, mode="sum")
            loss = loss + (pooled * torch.from_numpy(grad[:, t * D:(t + 1) * D].astype(np.float64))).sum()
        loss.backward()
        opt.step()
    for t in range(2):
        got = W[spec.weight_offset[t]:spec.weight_offset[t + 1]].reshape(-1, D)
        np.testing.assert_allclose(got, params[t].detach().numpy(), rtol=3e-6, atol=1e-7)
        acc = opt.state[params[t]]["sum"].numpy()
        np.testing.assert_allclose(m[spec.row_offset[t]:spec.row_offset[t + 1]], acc[:, 0], rtol=3e-6)


def test_gradient_aggregation_vs_dense_autograd():
    """The aggregated gradient per row is the autograd gradient of the pooled output w.r.t. the
    table; check it through the step it produces from m0 = 0 with distinct columns:
    W_new - W_old = -lr * g / (sqrt(mean g^2) + eps) is solved for g."""
    for mode, tmode in ((0, "sum"), (1, "mean")):
        spec = small_spec(T=2, rows=(5, 8), dims=(4, 8), B=6, pooling=3.0, seed=8)
        rng = np.random.default_rng(1)
        W0 = rng.standard_normal(int(spec.weight_offset[-1])).astype(np.float32)
        W = W0.copy(); m = np.zeros(int(spec.row_offset[-1]), np.float32)
        idx, off = wl.gen_batch(spec, 0)
        grad = wl.gen_grad(spec, 0)
        B = spec.batch
        uniq = _bwd(spec, W, m, idx, off, grad, lr=0.5, eps=0.0, mode=mode)
        lin = np.concatenate([spec.row_offset[t] + idx[off[t * B]:off[(t + 1) * B]] for t in range(2)])
        np.testing.assert_array_equal(uniq, np.unique(lin))
        for t in range(2):
            D = int(spec.dims[t])
            P = torch.zeros(int(spec.rows[t]), D, dtype=torch.float64, requires_grad=True)
            lo, hi = int(off[t * B]), int(off[(t + 1) * B])
            o = torch.from_numpy(off[t * B:(t + 1) * B] - lo)
            pooled = torch.nn.functional.embedding_bag(torch.from_numpy(idx[lo:hi]), P, o, mode=tmode)
            (pooled * torch.from_numpy(grad[:, spec.out_offset[t]:spec.out_offset[t + 1]].astype(np.float64))).sum().backward()
            g = P.grad.numpy()
            msq = (g * g).mean(axis=1)
            np.testing.assert_allclose(m[spec.row_offset[t]:spec.row_offset[t + 1]], msq, rtol=2e-6, atol=1e-30)
            dW = (W - W0)[spec.weight_offset[t]:spec.weight_offset[t + 1]].reshape(-1, D)
            touched = msq > 0
            want = -0.5 * g[touched] / np.sqrt(msq[touched])[:, None]
            np.testing.assert_allclose(dW[touched], want, rtol=1e-5, atol=1e-6)
            assert (dW[~touched] == 0).all()


def test_untouched_rows_keep_their_bits_and_momentum_grows():
    spec = small_spec(T=3, rows=(40, 25, 60), dims=(8, 4, 8), B=4, pooling=2.0, dtype=wl.FP16, seed=2)
    W = wl.all_weights_numpy(spec); W0 = W.copy()
    m = np.full(int(spec.row_offset[-1]), 0.25, np.float32); m0 = m.copy()
    idx, off = wl.gen_batch(spec, 0)
    uniq = _bwd(spec, W, m, idx, off, wl.gen_grad(spec, 0))
    touched = np.zeros(len(m), bool); touched[uniq] = True
    assert (m[~touched] == m0[~touched]).all() and (m >= m0).all() and (m[touched] > m0[touched]).all()
    for t in range(spec.T):
        D = int(spec.dims[t])
        a = W.view(np.uint16)[spec.weight_offset[t]:spec.weight_offset[t + 1]].reshape(-1, D)
        b = W0.view(np.uint16)[spec.weight_offset[t]:spec.weight_offset[t + 1]].reshape(-1, D)
        tt = touched[spec.row_offset[t]:spec.row_offset[t + 1]]
        assert (a[~tt] == b[~tt]).all()


def test_permutation_invariance_and_duplicates():
    """Order of lookups inside a bag does not matter; a row looked up k times in bags that carry
    the same gradient gets k times the single-lookup gradient."""
    spec = small_spec(T=1, rows=(6,), dims=(4,), B=2, pooling=4, bag_dist="fixed")
    rng = np.random.default_rng(3)
    W0 = rng.standard_normal(24).astype(np.float32)
    grad = rng.standard_normal((2, 4)).astype(np.float32)
    idx = np.array([0, 3, 3, 5, 3, 1, 0, 2], np.int64); off = np.array([0, 4, 8], np.int64)
    Wa, ma = W0.copy(), np.zeros(6, np.float32)
    _bwd(spec, Wa, ma, idx, off, grad)
    perm = np.array([3, 1, 0, 2, 7, 6, 5, 4])
    Wb, mb = W0.copy(), np.zeros(6, np.float32)
    _bwd(spec, Wb, mb, idx[perm], off, grad)
    np.testing.assert_array_equal(Wa, Wb); np.testing.assert_array_equal(ma, mb)
    # row 5 occurs once in bag 0; row 3 twice in bag 0 and once in bag 1
    g5 = grad[0].astype(np.float64); g3 = 2 * grad[0].astype(np.float64) + grad[1]
    np.testing.assert_allclose(ma[5], (g5 * g5).mean(), rtol=1e-6)
    np.testing.assert_allclose(ma[3], (g3 * g3).mean(), rtol=1e-6)


def test_one_step_per_row_per_batch_not_per_occurrence():
    spec = small_spec(T=1, rows=(2,), dims=(4,), B=1, pooling=3, bag_dist="fixed")
    W = np.zeros(8, np.float32); m = np.zeros(2, np.float32)
    g = np.array([[1, 2, 3, 4]], np.float32)
    _bwd(spec, W, m, np.array([1, 1, 1], np.int64), np.array([0, 3], np.int64), g)
    # aggregated gradient is 3g: m = 9 * 7.5, and the step equals that of g (scale invariant at m0 = 0)
    assert m[1] == np.float32(67.5)
    np.testing.assert_allclose(W[4:8], [-0.00365148, -0.00730297, -0.01095445, -0.01460593], rtol=2e-6)
