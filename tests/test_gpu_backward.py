"""GPU backward + row-wise Adagrad vs the CPU oracle through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_01515_b200 import binding as mb
from paper_2305_01515_b200 import workload as wl
from paper_2305_01515_b200.harness import DeviceModel
from helpers import FWD_RTOL, assert_close_mag, custom_spec, oracle_args, to_dev

pytestmark = pytest.mark.gpu


def _weights_f64(spec, W):
    return W.astype(np.float64)


def _run_steps(spec, n_steps=2, mode=0, batches=None, lr=None, grad_f16=False, m0=None, grad_fn=None):
    """n_steps train steps on GPU and oracle; compares weights, momentum and unique rows.
    grad_f16: the upstream gradient is rounded to binary16 first; the oracle gets those values in fp32 (the
    conversion is exact), the GPU gets the binary16 tensor (mts_tbe_backward_apply_f16)."""
    lr = spec.lr if lr is None else lr
    W0 = wl.all_weights_numpy(spec)
    W_ref = W0.copy()
    m_ref = np.zeros(int(spec.row_offset[-1]), np.float32) if m0 is None else m0.astype(np.float32).copy()
    model = DeviceModel(spec, weights=W0)
    model.momentum.copy_(torch.from_numpy(m_ref))
    for k in range(n_steps):
        idx, off = batches[k] if batches is not None else wl.gen_batch(spec, k)
        grad = wl.gen_grad(spec, k) if grad_fn is None else grad_fn(k)
        if grad_f16:
            grad = grad.astype(np.float16).astype(np.float32)
        N = len(idx)
        W_before = W_ref.copy()
        m_before = m_ref.copy()
        step_mag = np.zeros(W_ref.size, np.float64)
        uniq_ref = oracle.tbe_backward_rowwise_adagrad(*oracle_args(spec), spec.row_offset, W_ref, m_ref,
                                                       spec.batch, idx, off, grad, lr, spec.eps, mode,
                                                       step_mag=step_mag)
        uniq = torch.full((max(N, 1),), -1, dtype=torch.int64, device="cuda:0")
        nu = torch.full((1,), -1, dtype=torch.int64, device="cuda:0")
        grad_dev = to_dev(grad).to(torch.float16) if grad_f16 else to_dev(grad)
        model.backward(to_dev(idx), to_dev(off), N, grad_dev, lr=lr, pooling_mode=mode,
                       uniq_rows_out=uniq, n_unique_out=nu)
        torch.cuda.synchronize()
        assert model.tables.status() == 0
        U = int(nu.item())
        assert U == len(uniq_ref)
        np.testing.assert_array_equal(uniq[:U].cpu().numpy(), uniq_ref)          # bit-exact unique-row set
        W_gpu = model.weights_numpy()
        m_gpu = model.momentum.cpu().numpy()
        rtol = FWD_RTOL[spec.dtype]
        # tolerance: |got - ref| <= rtol * (|ref| + |W_old| + lr * sum|grad terms| / (sqrt(m) + eps));
        # momentum: relative to m_new
        mag_w = np.abs(_weights_f64(spec, W_before)) + step_mag
        assert_close_mag(W_gpu, W_ref, mag_w, rtol, f"weights after step {k}")
        assert_close_mag(m_gpu, m_ref, m_ref, 1e-5, f"momentum after step {k}")
        # untouched rows keep their bits
        touched = np.zeros(len(m_ref), bool); touched[uniq_ref] = True
        assert (m_gpu[~touched] == m_before[~touched]).all()
        for t in range(spec.T):
            D = int(spec.dims[t])
            a = W_gpu[spec.weight_offset[t]:spec.weight_offset[t + 1]].reshape(-1, D)
            b = W_before[spec.weight_offset[t]:spec.weight_offset[t + 1]].reshape(-1, D)
            tt = touched[spec.row_offset[t]:spec.row_offset[t + 1]]
            assert (a[~tt].view(np.uint8) == b[~tt].view(np.uint8)).all()
        # keep both sides on the same trajectory: continue from the oracle's state
        store = model.dev_weights
        store.copy_(torch.from_numpy(W_ref))
        model.momentum.copy_(torch.from_numpy(m_ref))
    model.close()


@pytest.mark.parametrize("mode", [0, 1])
def test_config1_full(mode):
    _run_steps(wl.config1(), n_steps=2, mode=mode)


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
def test_mixed_dims_skew_and_long_segments(dtype):
    """Rows hit thousands of times (segments spanning many 128-lookup chunks), rows hit once,
    every column-group width, chunk borders inside and between rows."""
    dims = [8, 64, 128, 200, 256, 512] if dtype == wl.FP16 else [4, 64, 128, 100, 256, 512]
    rows = [3, 5000, 20000, 7, 777, 129]
    pool = [40, 30, 20, 90, 33, 2]
    spec = custom_spec(rows, dims, 193, dtype, pool, [0, 1.3, 0.9, 0, 1.2, 0], seed=11)
    _run_steps(spec, n_steps=2)


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("mode", [0, 1])
def test_narrow_and_wide_tables_interleaved(dtype, mode):
    """Tables of up to 128 columns and of 129..256 columns in no order: the reduce step runs once per width
    class and every chunk of 128 sorted lookups belongs to exactly one of the two launches.  Tables with a
    handful of lookups sit between large ones, so that chunks span several tables of both classes; a row
    with thousands of lookups crosses many chunks in each class."""
    dims = [256, 64, 200, 8, 128, 256, 32, 136, 128]
    rows = [3000, 5, 2, 40000, 9, 1, 700, 20000, 3]
    pool = [25, 0.2, 0.1, 30, 0.3, 40, 12, 18, 0.05]
    spec = custom_spec(rows, dims, 257, dtype, pool, [1.2, 0, 0, 1.0, 0, 0, 0.9, 1.3, 0], seed=19)
    _run_steps(spec, n_steps=2, mode=mode)
    _run_steps(spec, n_steps=1, mode=mode, grad_f16=True)


def test_mean_pooling_fp16():
    spec = custom_spec([100, 3000], [64, 128], 65, wl.FP16, [5, 25], [1.1, 1.05], seed=2)
    _run_steps(spec, n_steps=2, mode=1)


def test_single_row_table_one_giant_segment():
    spec = custom_spec([1, 2], [128, 64], 300, wl.FP32, [30, 7], seed=4)
    _run_steps(spec, n_steps=1)


def test_lookup_counts_around_chunk_and_tile_borders():
    """N = 1, 127, 128, 129, 4095, 4096, 4097 lookups (chunk = 128 lookups, sort tile = 4096)."""
    for n in (1, 127, 128, 129, 4095, 4096, 4097):
        spec = custom_spec([50], [64], 1, wl.FP32, [n], bag_dist="fixed", seed=n)
        _run_steps(spec, n_steps=1)


def test_zero_gradient_leaves_weights_and_state_alone():
    """All-zero upstream gradient on fresh state: m stays 0, the step size is lr / eps times a zero gradient."""
    for dtype in (wl.FP32, wl.FP16):
        spec = custom_spec([40, 3000], [64, 256], 33, dtype, [6, 20], [0, 1.1], seed=8)
        zero = lambda k: np.zeros((spec.batch, spec.total_dim), np.float32)
        _run_steps(spec, n_steps=2, grad_fn=zero)
        # zero gradient for one table only, and for single columns
        def partly(k):
            g = wl.gen_grad(spec, k)
            g[:, :64] = 0.0
            g[:, 64::7] = 0.0
            return g
        _run_steps(spec, n_steps=2, grad_fn=partly)


def test_step_on_rows_whose_state_is_already_large_or_tiny():
    """Adagrad state far from its initial value: 1e6 (tiny steps), 1e-12 (steps near lr * g / eps scale)
    and a mix, two steps each."""
    spec = custom_spec([500, 2000], [128, 64], 64, wl.FP32, [10, 15], [1.05, 0.9], seed=9)
    n = int(spec.row_offset[-1])
    rng = np.random.default_rng(3)
    for m0 in (np.full(n, 1e6), np.full(n, 1e-12), 10.0 ** rng.uniform(-10, 6, n)):
        _run_steps(spec, n_steps=2, m0=m0)


def test_empty_batch_is_a_no_op():
    spec = custom_spec([10, 20], [64, 128], 16, wl.FP16, [3, 3])
    off = np.zeros(2 * 16 + 1, np.int64)
    _run_steps(spec, n_steps=1, batches=[(np.zeros(0, np.int64), off)])


def test_config2_scaled_and_config3_scaled():
    _run_steps(wl.config2(row_scale=0.02, batch=256), n_steps=2)
    _run_steps(wl.config3(row_scale=0.01, batch=128, tables=16), n_steps=2)


def test_two_runs_are_bit_identical():
    spec = wl.config2(row_scale=0.01, batch=512, tables=6)
    idx, off = wl.gen_batch(spec, 0)
    grad = wl.gen_grad(spec, 0)
    res = []
    for _ in range(2):
        m = DeviceModel(spec)
        m.backward(to_dev(idx), to_dev(off), len(idx), to_dev(grad))
        res.append((m.weights_numpy(), m.momentum.cpu().numpy()))
        m.close()
    assert (res[0][0].view(np.uint16) == res[1][0].view(np.uint16)).all()
    assert (res[0][1].view(np.uint32) == res[1][1].view(np.uint32)).all()


def test_workspace_too_small_and_misaligned_are_rejected():
    spec = custom_spec([10], [64], 2, wl.FP32, [2], bag_dist="fixed")
    m = DeviceModel(spec)
    idx, off = wl.gen_batch(spec, 0)
    grad = to_dev(wl.gen_grad(spec, 0))
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(mb.MtsError) as e:
        mb.tbe_backward_rowwise_adagrad(m.tables, 2, to_dev(idx), to_dev(off), len(idx), 0, grad, 64, 0.01, 1e-8,
                                        None, None, None, ws, 1024)
    assert e.value.code == mb.ERR_WORKSPACE
    m.close()


def test_config2_full_size_sampled_rows():
    """Full configuration 2 as bench.py runs it: the oracle replays a sample of rows (all their
    lookups in the batch) from the counter-based initial weights."""
    spec = wl.config2()
    idx, off = wl.gen_batch(spec, 0)
    grad = wl.gen_grad(spec, 0)
    m = DeviceModel(spec)
    m.backward(to_dev(idx), to_dev(off), len(idx), to_dev(grad))
    torch.cuda.synchronize()
    B = spec.batch
    rng = np.random.default_rng(1)
    for t in (0, 13, 25):
        seg = idx[off[t * B]:off[(t + 1) * B]]
        counts = np.bincount(seg, minlength=int(spec.rows[t]))
        hot = np.argsort(counts)[-3:]                                  # the hottest rows (long segments)
        cold = rng.choice(np.nonzero(counts == 1)[0], 40, replace=False)
        mid = rng.choice(np.nonzero(counts > 1)[0], 40, replace=False)
        untouched = rng.choice(np.nonzero(counts == 0)[0], 10, replace=False)
        sample = np.unique(np.concatenate([hot, cold, mid, untouched]))
        keep = np.isin(seg, sample)
        lens = np.diff(off[t * B:(t + 1) * B + 1])
        bag_of = np.repeat(np.arange(B), lens)
        sub_idx = np.searchsorted(sample, seg[keep])
        sub_len = np.bincount(bag_of[keep], minlength=B)
        sub_off = np.concatenate([[0], np.cumsum(sub_len)]).astype(np.int64)
        Wsub = wl.weights_numpy(spec, t, sample).reshape(-1)
        W_before = Wsub.copy()
        msub = np.zeros(len(sample), np.float32)
        g = np.ascontiguousarray(grad[:, spec.out_offset[t]:spec.out_offset[t + 1]])
        smag = np.zeros(Wsub.size, np.float64)
        oracle.tbe_backward_rowwise_adagrad(spec.dtype, [128], [0], [0], [0, len(sample)], Wsub, msub, B, sub_idx,
                                            sub_off, g, spec.lr, spec.eps, step_mag=smag)
        base = int(spec.weight_offset[t])
        got_w = m.dev_weights[base:base + int(spec.rows[t]) * 128].view(-1, 128)[to_dev(sample)].cpu().numpy().reshape(-1)
        got_m = m.momentum[int(spec.row_offset[t]) + to_dev(sample)].cpu().numpy()
        mag = np.abs(W_before.astype(np.float64)) + smag
        assert_close_mag(got_w, Wsub, mag, FWD_RTOL[spec.dtype], f"table {t} weights")
        assert_close_mag(got_m, msub, msub, 1e-5, f"table {t} momentum")
    m.close()


@pytest.mark.gpu
def test_backward_in_two_calls_matches_one_call():
    """mts_tbe_backward_sort on a second stream + mts_tbe_backward_apply give the bits of the one-call backward."""
    import torch
    from paper_2305_01515_b200 import workload as wl
    from paper_2305_01515_b200.harness import DeviceModel
    spec = wl.config1()
    dev = torch.device("cuda:0")
    idx_h, off_h = wl.gen_batch(spec, 0)[:2]
    grad_h = wl.gen_grad(spec, 0)
    idx, off = torch.from_numpy(idx_h).to(dev), torch.from_numpy(off_h).to(dev)
    grad = torch.from_numpy(grad_h).to(dev)
    n = idx.numel()
    results = []
    for split in (False, True):
        m = DeviceModel(spec, dev)
        main = torch.cuda.current_stream(dev)
        for _ in range(2):                          # two steps: the second reuses the workspace
            if split:
                side = torch.cuda.Stream(dev)
                fork, done = torch.cuda.Event(), torch.cuda.Event()
                fork.record(main)
                side.wait_event(fork)
                uniq = torch.empty(n, dtype=torch.int64, device=dev)
                nuniq = torch.zeros(1, dtype=torch.int64, device=dev)
                m.backward_sort(idx, off, n, uniq_rows_out=uniq, n_unique_out=nuniq, stream=side)
                done.record(side)
                main.wait_event(done)
                m.backward_apply(off, n, grad, stream=main)
            else:
                uniq = torch.empty(n, dtype=torch.int64, device=dev)
                nuniq = torch.zeros(1, dtype=torch.int64, device=dev)
                m.backward(idx, off, n, grad, uniq_rows_out=uniq, n_unique_out=nuniq, stream=main)
        torch.cuda.synchronize(dev)
        k = int(nuniq.item())
        results.append((m.dev_weights.clone(), m.momentum.clone(), uniq[:k].clone()))
    assert torch.equal(results[0][0], results[1][0])
    assert torch.equal(results[0][1], results[1][1])
    assert torch.equal(results[0][2], results[1][2])


@pytest.mark.gpu
@pytest.mark.parametrize("rows,pool,B", [
    ([250, 200, 256, 100, 255], [7, 0.02, 30, 3, 12], 257),          # 1 pass per table instead of 2; a nearly empty table
    ([60000, 65536, 40000], [40, 25, 33], 600),                      # 2 passes instead of 3; several tiles per table
    ([200, 70000, 3, 131072], [30, 25, 9, 20], 700),                 # 17 bits: two passes of 9; tables 0 and 2 have no bit left in the second
    ([1 << 20, 1000, 1 << 18, 5], [30, 40, 20, 3], 900),             # 20 bits: two passes of 10; table 1 is only copied in the second
    ([3 << 20, 900000], [35, 30], 1500),                             # 22 bits: two passes of 11
])
def test_tables_sorted_separately(rows, pool, B):
    """Table sets for which the lookups of each table are sorted on their own (fewer digit passes)."""
    spec = custom_spec(rows, [8 if max(rows) > 200000 else 64] * len(rows), B, wl.FP16, pool, [1.1] * len(rows), seed=5)
    _run_steps(spec, n_steps=2)


@pytest.mark.gpu
@pytest.mark.parametrize("rows", [[100_000_000], [1_200_000_000], [900_000_000, 3_000_000_000]])
def test_unsegmented_sort_of_wide_row_ids(rows):
    """Row ids of 27, 31 and 32 bits in one sort (three passes of 9, 11 and 11 bits): the distinct rows of the
    batch are compared with numpy's; the tables themselves are never allocated (sort only)."""
    spec = custom_spec(rows, [8] * len(rows), 500, wl.FP16, [40] * len(rows), [0.9] * len(rows), seed=6)
    idx, off = wl.gen_batch(spec, 0)
    N = len(idx)
    dummy = torch.zeros(64, dtype=torch.float16, device="cuda:0")
    mom = torch.zeros(1, dtype=torch.float32, device="cuda:0")
    tables = mb.tables_create(spec.dtype, spec.rows, spec.dims, spec.weight_offset[:-1], None, dummy, None, mom)
    wsb = mb.tbe_backward_workspace_bytes(tables, spec.batch, N)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda:0")
    uniq = torch.full((N,), -1, dtype=torch.int64, device="cuda:0")
    nu = torch.zeros(1, dtype=torch.int64, device="cuda:0")
    mb.tbe_backward_sort(tables, spec.batch, to_dev(idx), to_dev(off), N, ws, wsb, uniq, nu)
    torch.cuda.synchronize()
    lin = np.concatenate([spec.row_offset[t] + idx[off[t * spec.batch]:off[(t + 1) * spec.batch]] for t in range(spec.T)])
    ref = np.unique(lin)
    assert int(nu.item()) == len(ref)
    np.testing.assert_array_equal(uniq[:len(ref)].cpu().numpy(), ref)
    tables.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
@pytest.mark.parametrize("mode", [0, 1])
def test_fp16_gradient(dtype, mode):
    """Upstream gradient in binary16: every column-group width, long and short rows, sum and mean."""
    dims = [8, 64, 128, 200, 256, 512] if dtype == wl.FP16 else [4, 64, 128, 100, 256, 512]
    spec = custom_spec([3, 5000, 20000, 7, 777, 129], dims, 193, dtype, [40, 30, 20, 90, 33, 2],
                       [0, 1.3, 0.9, 0, 1.2, 0], seed=12)
    _run_steps(spec, n_steps=2, mode=mode, grad_f16=True)


@pytest.mark.gpu
def test_fp16_gradient_rows_of_128_columns():
    _run_steps(wl.config2(row_scale=0.02, batch=256), n_steps=2, grad_f16=True)
