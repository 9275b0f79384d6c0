"""The allocation-free backward entry point, mts_tbe_backward_rowwise_adagrad_static.

It serves callers that cannot hand the library a workspace because they cannot allocate device
memory at all: code running inside a framework that has claimed the whole GPU for its own pool,
or a step function that must never risk the device-wide stall an allocation can cause.  Its
scratch is a fixed array inside the library, so this file checks the two things that can go wrong
with that: the result must equal the regular entry point's result, also on a second call that
finds the first call's leftovers in the array, and a batch that does not fit must be refused
cleanly.  The file name makes pytest collect it last, after every other test has run.
"""
import numpy as np
import pytest
import torch

from paper_2305_01515_b200 import binding as mb
from paper_2305_01515_b200 import workload as wl
from paper_2305_01515_b200.harness import DeviceModel
from helpers import custom_spec, to_dev

pytestmark = pytest.mark.gpu


def _pair(spec):
    W = wl.all_weights_numpy(spec)
    return DeviceModel(spec, weights=W), DeviceModel(spec, weights=W), W


@pytest.mark.parametrize("dtype", [wl.FP32, wl.FP16])
def test_static_scratch_backward_matches_workspace_backward_twice(dtype):
    """Two train steps in a row through both entry points, from the same start; the second call
    of the static variant runs on scratch that still holds the first call's data."""
    spec = custom_spec([3000, 500, 7], [64, 128, 128], 200, dtype, [20, 35, 50], [1.05, 0.0, 0.0], seed=41)
    ref, new, W0 = _pair(spec)
    for k in range(2):
        idx, off = wl.gen_batch(spec, k)                      # a different, differently sized batch per call
        grad = to_dev(wl.gen_grad(spec, k))
        N = len(idx)
        d_idx, d_off = to_dev(idx), to_dev(off)
        uniq_a = torch.full((N,), -1, dtype=torch.int64, device="cuda:0"); nu_a = torch.zeros(1, dtype=torch.int64, device="cuda:0")
        uniq_b = torch.full((N,), -1, dtype=torch.int64, device="cuda:0"); nu_b = torch.zeros(1, dtype=torch.int64, device="cuda:0")
        ref.backward(d_idx, d_off, N, grad, uniq_rows_out=uniq_a, n_unique_out=nu_a)
        mb.tbe_backward_rowwise_adagrad_static(new.tables, spec.batch, d_idx, d_off, N, mb.POOL_SUM, grad,
                                               grad.shape[1], spec.lr, spec.eps, uniq_rows_out=uniq_b,
                                               n_unique_out=nu_b)
        torch.cuda.synchronize()
        assert int(nu_a.item()) == int(nu_b.item()) > 0
        assert torch.equal(uniq_a[:int(nu_a.item())], uniq_b[:int(nu_b.item())])
        # both entry points run the same deterministic kernels: the results agree bit for bit
        Wa, Wb = ref.weights_numpy(), new.weights_numpy()
        ma, mbm = ref.momentum.cpu().numpy(), new.momentum.cpu().numpy()
        assert (Wa.view(np.uint8) == Wb.view(np.uint8)).all(), f"weights, call {k}"
        assert (ma.view(np.uint32) == mbm.view(np.uint32)).all(), f"momentum, call {k}"
        assert (Wa.view(np.uint8) != W0.view(np.uint8)).any()
        assert (ma > 0).sum() >= int(nu_a.item())
    ref.close(); new.close()


def test_static_scratch_backward_refuses_a_batch_that_does_not_fit():
    spec = custom_spec([50], [64], 1, wl.FP32, [300_000], bag_dist="fixed")      # 300,000 lookups: too many
    m = DeviceModel(spec)
    idx, off = wl.gen_batch(spec, 0)
    grad = to_dev(wl.gen_grad(spec, 0))
    assert mb.tbe_backward_workspace_bytes(m.tables, 1, len(idx)) > mb.STATIC_SCRATCH_BYTES
    w_before = m.weights_numpy()
    with pytest.raises(mb.MtsError) as e:
        mb.tbe_backward_rowwise_adagrad_static(m.tables, 1, to_dev(idx), to_dev(off), len(idx), mb.POOL_SUM, grad, 64,
                                               0.01, 1e-8)
    assert e.value.code == mb.ERR_CAPACITY and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert (m.weights_numpy() == w_before).all()                                  # nothing ran
    m.close()
