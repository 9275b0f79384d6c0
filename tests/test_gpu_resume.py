"""Error path and resume of the cache, without faulting or hanging anything:
  - a bulk-copy fetch whose wait limit is set to zero polls gives up at once, reports MTS_ERR_TIMEOUT through
    mts_cache_status and leaves the cache usable: the same call repeated with the default limit completes and
    the run ends bit-identical to an undisturbed one;
  - flush -> export state -> new cache -> import state -> continue equals the uninterrupted run."""
import copy

import numpy as np
import pytest
import torch

from paper_2305_01515_b200 import binding as mb
from paper_2305_01515_b200 import workload as wl
from paper_2305_01515_b200.harness import DeviceModel
from helpers import custom_spec, to_dev

pytestmark = pytest.mark.gpu


def _spec():
    spec = custom_spec([5000, 2500], [128, 128], 128, wl.FP16, [8, 12], [1.05, 1.1], seed=35)
    spec.cached = True
    spec.cache_fraction = 0.05
    return spec


def _steps(model, spec, ks, hook=None):
    for k in ks:
        idx, off = wl.gen_batch(spec, k)
        N = len(idx)
        d_idx, d_off = to_dev(idx), to_dev(off)
        model.reserve(N)
        model.cache_lookup(d_idx, d_off, off, k)
        if hook is not None:
            hook(k)
        model.cache_move()
        model.forward(d_idx, d_off, N)
        model.backward(d_idx, d_off, N, to_dev(wl.gen_grad(spec, k)))


def test_fetch_that_gives_up_reports_timeout_and_the_call_can_be_repeated():
    spec = _spec()
    W0 = wl.all_weights_numpy(spec)
    ref = DeviceModel(spec, weights=W0)
    _steps(ref, spec, range(6))
    ref.flush()
    m = DeviceModel(spec, weights=W0)
    seen = []

    def give_up_once(k):
        if k != 3:
            return
        c = m.caches[0]
        mb.cache_set_fetch_wait_limit(c, 0)            # the first wait of every tile runs out at once
        m.cache_fetch(0)
        torch.cuda.synchronize()
        with pytest.raises(mb.MtsError) as e:
            c.status()
        seen.append(e.value.code)
        assert c.status() == 0                         # the status word was cleared by the read
        mb.cache_set_fetch_wait_limit(c, 1 << 22)      # the step then repeats the fetch with the default limit

    _steps(m, spec, range(6), hook=give_up_once)
    m.flush()
    torch.cuda.synchronize()
    assert seen == [mb.ERR_TIMEOUT]
    assert m.caches[0].status() == 0
    assert (m.weights_numpy().view(np.uint16) == ref.weights_numpy().view(np.uint16)).all()
    assert torch.equal(m.momentum, ref.momentum)
    with pytest.raises(mb.MtsError):
        mb.cache_set_fetch_wait_limit(m.caches[0], -1)
    m.close(); ref.close()


@pytest.mark.parametrize("policy", [mb.POLICY_LRU, mb.POLICY_LFU])
def test_flush_export_import_continue_equals_uninterrupted_run(policy):
    spec = _spec()
    W0 = wl.all_weights_numpy(spec)
    ref = DeviceModel(spec, weights=W0, policy=policy, lock_depth=1)
    _steps(ref, spec, range(10))
    ref.flush()
    a = DeviceModel(spec, weights=W0, policy=policy, lock_depth=1)
    _steps(a, spec, range(5))
    a.flush()
    torch.cuda.synchronize()
    c = a.caches[0]
    n = c.num_sets * 32
    d = "cuda:0"
    tags = torch.empty(n, dtype=torch.int64, device=d); ts = torch.empty_like(tags); fr = torch.empty_like(tags)
    dirty = torch.empty(n, dtype=torch.uint8, device=d)
    mb.cache_export_state(c, tags, ts, fr, dirty)
    torch.cuda.synchronize()
    assert int(dirty.sum().item()) == 0 and int((tags >= 0).sum().item()) > 100
    W_mid = a.weights_numpy()
    m_mid = a.momentum.clone()
    a.close()
    b = DeviceModel(spec, weights=W_mid, policy=policy, lock_depth=1)      # a new process would start like this
    b.momentum.copy_(m_mid)
    mb.cache_import_state(b.caches[0], tags, ts, fr, dirty, b.host_rows_ptr(0))
    _steps(b, spec, range(5, 10))
    b.flush()
    torch.cuda.synchronize()
    assert (b.weights_numpy().view(np.uint16) == ref.weights_numpy().view(np.uint16)).all()
    assert torch.equal(b.momentum, ref.momentum)
    # the cache made the same decisions: same final state
    for x, y in zip(_state(b.caches[0]), _state(ref.caches[0])):
        assert torch.equal(x, y)
    b.close(); ref.close()


def _state(c):
    n = c.num_sets * 32
    d = "cuda:0"
    tags = torch.empty(n, dtype=torch.int64, device=d); ts = torch.empty_like(tags); fr = torch.empty_like(tags)
    dirty = torch.empty(n, dtype=torch.uint8, device=d)
    mb.cache_export_state(c, tags, ts, fr, dirty)
    torch.cuda.synchronize()
    return tags, ts, fr, dirty
