"""Schedule of the cached train step: the cache work of batch t+1 (tag lookup, miss prefetch,
dirty writeback) runs on a side stream while batch t trains on the main stream (Section 5.7 of
the paper: prefetch into the cache ahead of training; Section 6.1: cache kernels on their own
streams, synchronised with the next batch's lookups).  Only events order the two streams.

Why this is safe with lock_depth >= 1: the replacement of batch t+1 may only take ways whose
timestamp is older than t, so it never touches a slot batch t reads or updates; its decisions depend
on tags and timestamps only, which batch t's forward/backward do not write.  The one data hazard is
a row that found no evictable way in batch t (served from host memory directly) and is fetched from
host memory for batch t+1: when batch t reported such overflow, the data movement of batch t+1 waits
for batch t's backward.
"""
from __future__ import annotations

from typing import Callable, List, Optional

import numpy as np
import torch

from . import binding as mb
from .harness import DeviceModel


class CachedTrainer:
    def __init__(self, model: DeviceModel, pipelined: bool = True):
        assert model.cached
        self.m = model
        self.pipelined = pipelined
        self.dev = model.device
        self.main = torch.cuda.current_stream(self.dev)
        self.side = torch.cuda.Stream(self.dev) if pipelined else self.main
        n_c = len(model.caches)
        self.host_counters = [torch.zeros((n_c, mb.NUM_COUNTERS), dtype=torch.int64).pin_memory() for _ in range(2)]
        self.history: List[np.ndarray] = []           # per batch [n_caches, NUM_COUNTERS]

    def _prepare(self, t, batch, ctx, ev_tags, ev_ready, wait_bwd_prev, wait_bwd_cur_if_overflow):
        """Cache work of batch t into context ctx on the side stream."""
        m, s = self.m, self.side
        idx, off, off_host = batch[0], batch[1], batch[2]
        if wait_bwd_prev is not None:
            s.wait_event(wait_bwd_prev)                 # victims' rows and dirty bytes are final
        m.cache_lookup(idx, off, off_host, t, stream=s, ctx=ctx)
        for g in range(len(m.caches)):
            self.host_counters[ctx][g].copy_(m.ctx[ctx]["lists"][g]["counters"], non_blocking=True)
        ev_tags.record(s)
        if wait_bwd_cur_if_overflow is not None:
            s.wait_event(wait_bwd_cur_if_overflow)
        m.cache_move(stream=s, ctx=ctx)
        ev_ready.record(s)

    def run(self, batches, grads, out: Optional[torch.Tensor] = None,
            on_step: Optional[Callable[[int], None]] = None, first_step: int = 0) -> None:
        """Train on `batches` = [(indices_dev, offsets_dev, offsets_host)], `grads` = [grad_out_dev]."""
        m = self.m
        K = len(batches)
        if K == 0:
            return
        with torch.cuda.stream(self.side):
            pass
        ev_tags = [torch.cuda.Event() for _ in range(K)]
        ev_ready = [torch.cuda.Event() for _ in range(K)]
        ev_bwd = [torch.cuda.Event() for _ in range(K)]
        if out is None:
            out = torch.empty((m.spec.batch, m.spec.total_dim), dtype=torch.float32, device=self.dev)
        prev_overflow = False
        # side stream must see the inputs produced on the main stream
        start = torch.cuda.Event()
        start.record(self.main)
        self.side.wait_event(start)
        if self.pipelined:
            with torch.cuda.stream(self.side):
                self._prepare(first_step, batches[0], 0, ev_tags[0], ev_ready[0], None, None)
        for t in range(K):
            ctx = t & 1
            idx, off, _ = batches[t]
            N = idx.numel()
            if not self.pipelined:
                self._prepare(first_step + t, batches[t], ctx, ev_tags[t], ev_ready[t], None, None)
            else:
                self.main.wait_event(ev_ready[t])
            m.forward(idx, off, N, out=out, stream=self.main, ctx=ctx)
            m.backward(idx, off, N, grads[t], stream=self.main, ctx=ctx)
            ev_bwd[t].record(self.main)
            ev_tags[t].synchronize()                     # counters of batch t are on the host
            cnt = self.host_counters[ctx].numpy().copy()
            self.history.append(cnt)
            overflow_t = bool(cnt[:, 9].sum() > 0)
            if self.pipelined and t + 1 < K:
                with torch.cuda.stream(self.side):
                    self._prepare(first_step + t + 1, batches[t + 1], (t + 1) & 1, ev_tags[t + 1], ev_ready[t + 1],
                                  ev_bwd[t - 1] if t >= 1 else None, ev_bwd[t] if overflow_t else None)
            if on_step is not None:
                on_step(t)
        self.main.wait_stream(self.side)
