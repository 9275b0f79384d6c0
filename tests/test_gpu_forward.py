"""GPU pooled lookup vs the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_01515_b200 import binding as mb
from paper_2305_01515_b200 import workload as wl
from paper_2305_01515_b200.harness import DeviceModel
from helpers import FWD_RTOL, assert_close_mag, custom_spec, oracle_args, to_dev

pytestmark = pytest.mark.gpu


def _run_and_compare(spec, k=0, mode=0, batch=None):
    W = wl.all_weights_numpy(spec)
    idx, off = batch if batch is not None else wl.gen_batch(spec, k)
    ref, mag = oracle.tbe_forward(*oracle_args(spec), W, spec.batch, idx, off, mode, want_mag=True)
    m = DeviceModel(spec, weights=W)
    out = torch.full((spec.batch, spec.total_dim), float("nan"), dtype=torch.float32, device="cuda:0")
    m.forward(to_dev(idx), to_dev(off), len(idx), out=out, pooling_mode=mode)
    torch.cuda.synchronize()
    assert m.tables.status() == 0
    assert_close_mag(out.cpu().numpy(), ref, mag, FWD_RTOL[spec.dtype], "forward")
    m.close()


@pytest.mark.parametrize("mode", [0, 1])
def test_config1_full(mode):
    _run_and_compare(wl.config1(), mode=mode)


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("mode", [0, 1])
def test_mixed_dims_and_ragged_bags(dtype, mode):
    """Every lane-group width (1..32 chunks and rows wider than one warp pass), bags from empty
    to several 32-lookup tiles with a ragged tail."""
    dims = [8, 16, 24, 64, 128, 200, 256, 512] if dtype == wl.FP16 else [4, 8, 12, 64, 128, 100, 256, 512]
    rows = [50, 1000, 37, 5000, 20000, 300, 777, 129]
    pool = [0.7, 3, 40, 70, 20, 5, 33, 2]
    spec = custom_spec(rows, dims, 97, dtype, pool, [0, 1.1, 0, 1.05, 0.9, 0, 1.3, 0], seed=3)
    _run_and_compare(spec, mode=mode)


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("mode", [0, 1])
def test_rows_of_at_most_one_warp_pass(dtype, mode):
    """No row wider than 32 16-byte chunks and no cached table: the launch takes the kernel specialised
    for that case.  Every lane-group width from 1 to 32 chunks (whole powers of two and not), a table
    change inside a warp's run of bags (batch 97 is no multiple of the bags per warp), empty bags and
    bags of several 32-lookup tiles with a ragged tail."""
    dims = [8, 16, 24, 64, 128, 200, 256, 104] if dtype == wl.FP16 else [4, 8, 12, 64, 128, 100, 32, 52]
    rows = [50, 1000, 37, 5000, 20000, 300, 777, 129]
    pool = [0.7, 3, 40, 70, 20, 5, 33, 2]
    spec = custom_spec(rows, dims, 97, dtype, pool, [0, 1.1, 0, 1.05, 0.9, 0, 1.3, 0], seed=4)
    _run_and_compare(spec, mode=mode)


def test_dim_1024_fp32_and_fp16():
    for dtype in (wl.FP32, wl.FP16):
        _run_and_compare(custom_spec([300, 40], [1024, 64], 33, dtype, [6, 2], seed=5))


def test_empty_batch_and_all_empty_bags():
    spec = custom_spec([10, 20], [64, 128], 16, wl.FP16, [3, 3])
    off = np.zeros(2 * 16 + 1, np.int64)
    _run_and_compare(spec, batch=(np.zeros(0, np.int64), off))


def test_config2_scaled_and_config3_scaled():
    _run_and_compare(wl.config2(row_scale=0.02, batch=256))
    _run_and_compare(wl.config3(row_scale=0.01, batch=128, tables=16))


def test_out_of_range_index_is_clamped_and_flagged():
    spec = custom_spec([10], [64], 2, wl.FP32, [2], bag_dist="fixed")
    W = wl.all_weights_numpy(spec)
    idx = np.array([3, 10_000, -5, 9], np.int64)
    off = np.array([0, 2, 4], np.int64)
    m = DeviceModel(spec, weights=W)
    out = m.forward(to_dev(idx), to_dev(off), 4)
    torch.cuda.synchronize()
    assert m.tables.status() == 1 and m.tables.status() == 0      # sticky, cleared by the read
    ref = oracle.tbe_forward(*oracle_args(spec), W, 2, np.array([3, 9, 0, 9], np.int64), off)
    np.testing.assert_allclose(out.cpu().numpy(), ref, rtol=1e-6)
    m.close()


def test_config2_full_size_sampled_bags():
    """Full configuration 2 as bench.py runs it; the oracle recomputes a sample of bags from
    the counter-based weights (compact sub-problem: only the rows those bags touch)."""
    spec = wl.config2()
    idx, off = wl.gen_batch(spec, 0)
    m = DeviceModel(spec)
    out = m.forward(to_dev(idx), to_dev(off), len(idx)).cpu().numpy()
    assert m.tables.status() == 0
    rng = np.random.default_rng(0)
    B = spec.batch
    for t in rng.choice(spec.T, 4, replace=False):
        bs = np.sort(rng.choice(B, 64, replace=False))
        rows_needed = np.unique(np.concatenate([idx[off[t * B + b]:off[t * B + b + 1]] for b in bs] + [np.zeros(1, np.int64)]))
        Wsub = wl.weights_numpy(spec, int(t), rows_needed).reshape(-1)
        sub_idx = np.concatenate([np.searchsorted(rows_needed, idx[off[t * B + b]:off[t * B + b + 1]]) for b in bs])
        lens = np.array([off[t * B + b + 1] - off[t * B + b] for b in bs])
        sub_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        ref, mag = oracle.tbe_forward(spec.dtype, [128], [0], [0], Wsub, len(bs), sub_idx, sub_off, 0, want_mag=True)
        got = out[bs][:, spec.out_offset[t]:spec.out_offset[t + 1]]
        assert_close_mag(got, ref, mag, FWD_RTOL[spec.dtype], f"table {t}")
    m.close()


def test_config3_full_size_sampled_bags_and_rows():
    """Full configuration 3 (64 heterogeneous tables, 17 GB) as bench.py runs it: the oracle
    recomputes a sample of bags (forward) and of rows (backward) from the counter-based weights."""
    spec = wl.config3()
    idx, off = wl.gen_batch(spec, 0)
    grad = wl.gen_grad(spec, 0)
    m = DeviceModel(spec)
    d_idx, d_off = to_dev(idx), to_dev(off)
    out = m.forward(d_idx, d_off, len(idx)).cpu().numpy()
    m.backward(d_idx, d_off, len(idx), to_dev(grad))
    torch.cuda.synchronize()
    assert m.tables.status() == 0
    rng = np.random.default_rng(3)
    B = spec.batch
    picked = [int(np.argmax(spec.dims == d)) for d in (64, 128, 256)] + [spec.T - 1]
    for t in picked:
        D = int(spec.dims[t])
        # forward on 48 sampled bags
        bs = np.sort(rng.choice(B, 48, replace=False))
        rows_needed = np.unique(np.concatenate([idx[off[t * B + b]:off[t * B + b + 1]] for b in bs] + [np.zeros(1, np.int64)]))
        Wsub = wl.weights_numpy(spec, t, rows_needed).reshape(-1)
        sub_idx = np.concatenate([np.searchsorted(rows_needed, idx[off[t * B + b]:off[t * B + b + 1]]) for b in bs])
        lens = np.array([off[t * B + b + 1] - off[t * B + b] for b in bs])
        sub_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        ref, mag = oracle.tbe_forward(spec.dtype, [D], [0], [0], Wsub, len(bs), sub_idx, sub_off, 0, want_mag=True)
        assert_close_mag(out[bs][:, spec.out_offset[t]:spec.out_offset[t + 1]], ref, mag, FWD_RTOL[spec.dtype], f"fwd table {t}")
        # backward on sampled rows: the hottest, some touched once, some untouched
        seg = idx[off[t * B]:off[(t + 1) * B]]
        counts = np.bincount(seg, minlength=int(spec.rows[t]))
        groups = [np.argsort(counts)[-2:]]
        for sel in (counts == 1, counts > 1, counts == 0):
            cand = np.nonzero(sel)[0]
            if len(cand):
                groups.append(rng.choice(cand, min(20, len(cand)), replace=False))
        sample = np.unique(np.concatenate(groups))
        keep = np.isin(seg, sample)
        bag_of = np.repeat(np.arange(B), np.diff(off[t * B:(t + 1) * B + 1]))
        sub_idx = np.searchsorted(sample, seg[keep])
        sub_off = np.concatenate([[0], np.cumsum(np.bincount(bag_of[keep], minlength=B))]).astype(np.int64)
        Wsub = wl.weights_numpy(spec, t, sample).reshape(-1)
        W_before = Wsub.astype(np.float64)
        msub = np.zeros(len(sample), np.float32)
        smag = np.zeros(Wsub.size, np.float64)
        g = np.ascontiguousarray(grad[:, spec.out_offset[t]:spec.out_offset[t + 1]])
        oracle.tbe_backward_rowwise_adagrad(spec.dtype, [D], [0], [0], [0, len(sample)], Wsub, msub, B, sub_idx, sub_off,
                                            g, spec.lr, spec.eps, step_mag=smag)
        base = int(spec.weight_offset[t])
        got_w = m.dev_weights[base:base + int(spec.rows[t]) * D].view(-1, D)[to_dev(sample)].cpu().numpy().reshape(-1)
        got_m = m.momentum[int(spec.row_offset[t]) + to_dev(sample)].cpu().numpy()
        assert_close_mag(got_w, Wsub, np.abs(W_before) + smag, FWD_RTOL[spec.dtype], f"bwd table {t} weights")
        assert_close_mag(got_m, msub, msub, 1e-5, f"bwd table {t} momentum")
    m.close()


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("mode", [0, 1])
def test_fp16_output(dtype, mode):
    """mts_tbe_forward_f16: the pooled sum is accumulated in fp32 and rounded once to binary16.  Against the
    oracle's fp64 sums: the fp32 tolerance of the sum plus half a binary16 ulp of the rounded value."""
    dims = [8, 64, 128, 200, 256, 512] if dtype == wl.FP16 else [4, 64, 128, 100, 256, 512]
    spec = custom_spec([50, 5000, 20000, 300, 777, 129], dims, 97, dtype, [0.7, 70, 20, 5, 33, 2],
                       [0, 1.05, 0.9, 0, 1.3, 0], seed=4)
    W = wl.all_weights_numpy(spec)
    idx, off = wl.gen_batch(spec, 0)
    ref, mag = oracle.tbe_forward(*oracle_args(spec), W, spec.batch, idx, off, mode, want_mag=True)
    m = DeviceModel(spec, weights=W)
    out = torch.full((spec.batch, spec.total_dim), float("nan"), dtype=torch.float16, device="cuda:0")
    m.forward(to_dev(idx), to_dev(off), len(idx), out=out, pooling_mode=mode)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    ref = np.asarray(ref, np.float64).reshape(got.shape)
    mag = np.asarray(mag, np.float64).reshape(got.shape)
    # binary16: 11 significant bits -> half an ulp is at most 2^-11 relative (normal range; the values here
    # are far above the subnormal range or exactly 0)
    bound = FWD_RTOL[spec.dtype] * (np.abs(ref) + mag) + 2.0 ** -11 * np.abs(ref) + 2.0 ** -25
    assert np.isfinite(got).all()
    assert (np.abs(got - ref) <= bound).all(), float(np.max(np.abs(got - ref) - bound))
    m.close()


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
def test_max_pooling_is_exact(dtype):
    """Max pooling selects stored values, so the fp32 output equals the oracle's bit for bit: every lane-group
    width, empty bags (0), bags of one row, negative-only bags, bags longer than a 32-lookup tile."""
    dims = [8, 16, 24, 64, 128, 200, 256, 512] if dtype == wl.FP16 else [4, 8, 12, 64, 128, 100, 256, 512]
    rows = [50, 1000, 37, 5000, 20000, 300, 777, 129]
    spec = custom_spec(rows, dims, 97, dtype, [0.7, 3, 40, 70, 20, 5, 33, 2], [0, 1.1, 0, 1.05, 0.9, 0, 1.3, 0], seed=13)
    W = wl.all_weights_numpy(spec)
    W[: int(spec.weight_offset[1])] = -np.abs(W[: int(spec.weight_offset[1])]) - 0.25      # table 0: all negative
    idx, off = wl.gen_batch(spec, 0)
    ref = oracle.tbe_forward(*oracle_args(spec), W, spec.batch, idx, off, 2)
    m = DeviceModel(spec, weights=W)
    out = torch.full((spec.batch, spec.total_dim), float("nan"), dtype=torch.float32, device="cuda:0")
    m.forward(to_dev(idx), to_dev(off), len(idx), out=out, pooling_mode=mb.POOL_MAX)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    lens = np.diff(off)
    assert (lens == 0).any() and (lens == 1).any() and (lens > 40).any()
    m.close()
    # the 32-piece kernel family too (no wide row in the model)
    spec2 = custom_spec(rows[:5], dims[:5], 97, dtype, [0.7, 3, 40, 70, 20], [0, 1.1, 0, 1.05, 0.9], seed=14)
    W2 = wl.all_weights_numpy(spec2)
    idx2, off2 = wl.gen_batch(spec2, 0)
    ref2 = oracle.tbe_forward(*oracle_args(spec2), W2, spec2.batch, idx2, off2, 2)
    m2 = DeviceModel(spec2, weights=W2)
    out2 = m2.forward(to_dev(idx2), to_dev(off2), len(idx2), pooling_mode=mb.POOL_MAX)
    np.testing.assert_array_equal(out2.cpu().numpy().view(np.uint32), ref2.view(np.uint32))
    m2.close()


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("mode", [0, 1])
def test_bf16_output(dtype, mode):
    """mts_tbe_forward_bf16: the fp32 pooled value rounded once to bfloat16 (8 significant bits: half an ulp is
    at most 2^-8 relative), both kernel families."""
    for dims in ([8, 64, 128, 200, 256, 512] if dtype == wl.FP16 else [4, 64, 128, 100, 256, 512],
                 [8, 64, 128, 200] if dtype == wl.FP16 else [4, 64, 128, 100]):
        n = len(dims)
        spec = custom_spec([50, 5000, 20000, 300, 777, 129][:n], dims, 97, dtype, [0.7, 70, 20, 5, 33, 2][:n],
                           [0, 1.05, 0.9, 0, 1.3, 0][:n], seed=4)
        W = wl.all_weights_numpy(spec)
        idx, off = wl.gen_batch(spec, 0)
        ref, mag = oracle.tbe_forward(*oracle_args(spec), W, spec.batch, idx, off, mode, want_mag=True)
        m = DeviceModel(spec, weights=W)
        out = torch.full((spec.batch, spec.total_dim), float("nan"), dtype=torch.bfloat16, device="cuda:0")
        m.forward(to_dev(idx), to_dev(off), len(idx), out=out, pooling_mode=mode)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy().astype(np.float64)
        ref = np.asarray(ref, np.float64).reshape(got.shape)
        mag = np.asarray(mag, np.float64).reshape(got.shape)
        bound = FWD_RTOL[spec.dtype] * (np.abs(ref) + mag) + 2.0 ** -8 * np.abs(ref) + 2.0 ** -40
        assert np.isfinite(got).all()
        assert (np.abs(got - ref) <= bound).all(), float(np.max(np.abs(got - ref) - bound))
        # and it is the fp32 output rounded to nearest even, bit for bit
        out32 = m.forward(to_dev(idx), to_dev(off), len(idx), pooling_mode=mode)
        assert torch.equal(out32.to(torch.bfloat16), out)
        m.close()
