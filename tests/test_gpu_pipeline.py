"""Pipelined cached training (cache work of batch t+1 on a side stream while batch t trains) must
give the same bits as the sequential schedule, and the same cache decisions as the oracle."""
import copy

import numpy as np
import pytest
import torch

import oracle
from paper_2305_01515_b200 import binding as mb
from paper_2305_01515_b200 import workload as wl
from paper_2305_01515_b200.harness import DeviceModel
from paper_2305_01515_b200.pipeline import CachedTrainer
from helpers import custom_spec, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("lock", [1, 2])
@pytest.mark.parametrize("frac", [0.2, 0.004])       # roomy cache; cache smaller than a batch (overflow path)
def test_pipelined_equals_sequential_and_oracle_tags(frac, lock):
    rows, dims = [20000, 9000, 4000, 12000], [64, 64, 128, 128]
    spec = custom_spec(rows, dims, 256, wl.FP16, [8, 12, 20, 5], [1.05, 0.9, 1.2, 1.0], seed=77)
    spec.cached = True
    spec.cache_fraction = frac
    spec.reuse_prob, spec.reuse_window = 0.7, 4
    stream = wl.BatchStream(spec)
    K = 10
    host_batches = [stream.next() for _ in range(K)]
    grads = [to_dev(wl.gen_grad(spec, k)) for k in range(K)]
    W0 = wl.all_weights_numpy(spec)
    results = []
    # sequential with the kernels fetching the missed rows; pipelined the same way; pipelined and
    # sequential with the rows gathered by host threads and moved by the copy engine
    # ... and both places of the tag step: between the training steps, or on a stream of its own
    # ... and the copy-engine path starting from pinned buffers of two rows, which have to grow with the lists
    # ... and the caches' data paths on the library's mover threads (native) or on Python threads
    for pipelined, host_gather, tag_on_main, stage_bytes, native in (
            (False, False, True, None, None), (True, False, True, None, None), (True, True, True, None, True),
            (False, True, True, None, None), (True, False, False, None, None), (True, True, False, None, True),
            (True, True, False, None, False), (True, True, True, None, False),
            (True, True, False, 512, False), (True, True, False, 512, True), (False, True, True, 512, None)):
        m = DeviceModel(spec, weights=W0, lock_depth=lock)
        if stage_bytes is not None:
            m.FETCH_STAGE_BYTES = stage_bytes
        m.reserve(max(len(b[0]) for b in host_batches))
        batches = [(to_dev(i), to_dev(o), o) for i, o in host_batches]
        tr = CachedTrainer(m, pipelined=pipelined, host_gather=host_gather, tag_on_main=tag_on_main, native_mover=native)
        tr.run(batches, grads)
        m.flush()
        torch.cuda.synchronize()
        if stage_bytes is not None and not (pipelined and native):
            assert max(m.fetch_rows) > stage_bytes // 128        # the buffers did grow
        if pipelined and host_gather and native:
            assert sum(mv.stats()["gather_bytes"] for mv in tr._movers) > 0      # the movers did the work
        tr.close()
        results.append((m.weights_numpy(), m.momentum.cpu().numpy(), np.stack(tr.history)))
        m.close()
    (Wa, ma, ha), (Wb, mb_, hb) = results[0], results[1]
    for Wx, mx, hx in results[1:]:
        assert (ha == hx).all()
        assert (Wa.view(np.uint16) == Wx.view(np.uint16)).all()
        assert (ma.view(np.uint32) == mx.view(np.uint32)).all()
    # the oracle's tag-only simulation makes the same decisions (the backward dirties every placed slot)
    groups = spec.dim_groups()
    B = spec.batch
    overflow = 0
    for g, (dim, t0, t1) in enumerate(groups):
        rows_g = int(spec.row_offset[t1] - spec.row_offset[t0])
        oc = oracle.Cache(wl.cache_sets_for(rows_g, frac), 32, dim, spec.dtype, 0, lock, with_data=False)
        for k, (idx, off) in enumerate(host_batches):
            keys = np.concatenate([spec.row_offset[t] - spec.row_offset[t0] + idx[off[t * B]:off[(t + 1) * B]]
                                   for t in range(t0, t1)])
            res = oc.lookup_insert(keys, k)
            used = res["slot_of_lookup"][res["slot_of_lookup"] >= 0]
            oc.dirty[used] = 1
            assert dict(zip(mb.COUNTER_NAMES, hb[k, g].tolist())) == res["counters"], (g, k)
            overflow += res["counters"]["overflow"]
        oc.close()
    if frac < 0.01:
        assert overflow > 0


@pytest.mark.parametrize("host_gather", [False, True])
def test_overflow_repair_survives_slow_side_streams(host_gather):
    """Lock depth 2, a cache much smaller than a batch (rows overflow in every batch) and move / repair
    streams that idle for about a millisecond before each piece of work, so that the tag step two batches
    ahead and the training run as far ahead of them as the events allow: the result must still equal the
    sequential run bit for bit (the overflow lists stay intact until their repair has read them)."""
    rows, dims = [20000, 9000, 4000, 12000], [64, 64, 128, 128]
    spec = custom_spec(rows, dims, 256, wl.FP16, [8, 12, 20, 5], [1.05, 0.9, 1.2, 1.0], seed=78)
    spec.cached = True
    spec.cache_fraction = 0.004
    spec.reuse_prob, spec.reuse_window = 0.7, 4
    stream = wl.BatchStream(spec)
    K = 12
    host_batches = [stream.next() for _ in range(K)]
    grads = [to_dev(wl.gen_grad(spec, k)) for k in range(K)]
    W0 = wl.all_weights_numpy(spec)
    results = []
    for pipelined, delay, tag_on_main in ((False, 0, True), (True, 2_000_000, True), (True, 0, True),
                                          (True, 2_000_000, False)):
        m = DeviceModel(spec, weights=W0, lock_depth=2)
        m.reserve(max(len(b[0]) for b in host_batches))
        batches = [(to_dev(i), to_dev(o), o) for i, o in host_batches]
        tr = CachedTrainer(m, pipelined=pipelined, host_gather=host_gather, tag_on_main=tag_on_main)
        tr.debug_delay_cycles = delay
        tr.run(batches, grads)
        m.flush()
        torch.cuda.synchronize()
        results.append((m.weights_numpy(), m.momentum.cpu().numpy(), np.stack(tr.history)))
        m.close()
    Wa, ma, ha = results[0]
    assert ha[:, :, mb.COUNTER_NAMES.index("overflow")].sum() > 100
    for Wx, mx, hx in results[1:]:
        assert (ha == hx).all()
        assert (Wa.view(np.uint16) == Wx.view(np.uint16)).all()
        assert (ma.view(np.uint32) == mx.view(np.uint32)).all()
