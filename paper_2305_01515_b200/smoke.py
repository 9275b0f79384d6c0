"""One small invocation of the whole path on cuda:0, checked against the CPU oracle."""
import os
import sys

import numpy as np


def run() -> None:
    import torch

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    if root not in sys.path:
        sys.path.insert(0, root)
    import oracle                                   # test infrastructure, used only to check the result
    from . import binding as mb
    from . import workload as wl
    from .harness import DeviceModel

    assert torch.cuda.is_available(), "smoke() needs a CUDA device"
    dev = "cuda:0"

    def close(got, ref, mag, rtol, what):
        err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
        bound = rtol * (np.abs(ref.astype(np.float64)) + mag)
        assert (err <= bound).all(), f"{what}: max excess {float((err - bound).max()):.3e}"

    # uncached: configuration 1 (4 tables x 10,000 rows x 64, fp32), one train step
    spec = wl.config1()
    W = wl.all_weights_numpy(spec)
    idx, off = wl.gen_batch(spec, 0)
    grad = wl.gen_grad(spec, 0)
    args = (spec.dtype, spec.dims, spec.out_offset[:-1], spec.weight_offset[:-1])
    ref, mag = oracle.tbe_forward(*args, W, spec.batch, idx, off, 0, want_mag=True)
    W_ref, m_ref = W.copy(), np.zeros(int(spec.row_offset[-1]), np.float32)
    smag = np.zeros(W.size, np.float64)
    oracle.tbe_backward_rowwise_adagrad(*args, spec.row_offset, W_ref, m_ref, spec.batch, idx, off, grad, spec.lr,
                                        spec.eps, step_mag=smag)
    model = DeviceModel(spec, device=dev, weights=W)
    d_idx, d_off = torch.from_numpy(idx).to(dev), torch.from_numpy(off).to(dev)
    out = model.forward(d_idx, d_off, len(idx))
    model.backward(d_idx, d_off, len(idx), torch.from_numpy(grad).to(dev))
    torch.cuda.synchronize()
    close(out.cpu().numpy(), ref, mag, 1e-5, "forward")
    close(model.weights_numpy(), W_ref, np.abs(W.astype(np.float64)) + smag, 1e-5, "weights")
    close(model.momentum.cpu().numpy(), m_ref, m_ref.astype(np.float64), 1e-5, "momentum")
    model.close()

    # cached: two small fp16 tables in pinned host memory behind a 32-way LRU cache
    tabs = wl._finish_tables([wl.TableSpec(4000, 64, 8, 1.05), wl.TableSpec(2000, 64, 5, 0.9)],
                             np.random.default_rng(0))
    cspec = wl.ModelSpec("smoke-cached", tabs, wl.FP16, 64, "poisson", seed=1, cached=True, cache_fraction=0.1)
    Wc = wl.all_weights_numpy(cspec)
    cm = DeviceModel(cspec, device=dev, weights=Wc)
    oc = oracle.Cache(wl.cache_sets_for(6000, 0.1), 32, 64, wl.FP16, 0, 0, with_data=False)
    for k in range(3):
        idx, off = wl.gen_batch(cspec, k)
        B = cspec.batch
        d_idx, d_off = torch.from_numpy(idx).to(dev), torch.from_numpy(off).to(dev)
        cm.reserve(len(idx))
        cm.cache_step(d_idx, d_off, off, k)
        keys = np.concatenate([cspec.row_offset[t] + idx[off[t * B]:off[(t + 1) * B]] for t in range(2)])
        res = oc.lookup_insert(keys, k)
        torch.cuda.synchronize()
        assert (cm.slot_of_lookup[:len(idx)].cpu().numpy() == res["slot_of_lookup"]).all(), "cache slots"
        got = dict(zip(mb.COUNTER_NAMES, cm.lists[0]["counters"].cpu().tolist()))
        assert got == res["counters"], (got, res["counters"])
        cm.forward(d_idx, d_off, len(idx))
        cm.backward(d_idx, d_off, len(idx), torch.from_numpy(wl.gen_grad(cspec, k)).to(dev))
        used = res["slot_of_lookup"][res["slot_of_lookup"] >= 0]
        oc.dirty[used] = 1                       # the backward pass dirties every slot it updates
    cm.flush()
    torch.cuda.synchronize()
    oc.close()
    cm.close()
    print("smoke ok: forward, backward + row-wise Adagrad and cache match the CPU oracle; "
          f"{mb.launch_count()} kernel launches")
