"""Schedule of the cached train step (Section 5.7 of the paper: prefetch into the cache ahead of
training; Section 6.1: cache kernels on their own streams, synchronised with the next batch's
lookups).  Streams, ordered by events only:

    main    : forward(t), backward(t)
    move[g] : cache g: save victims / fetch missed rows / write victims back for batch t+1   (host link)
    fix     : repair of rows that overflowed in batch t and were placed in batch t+1 (after backward(t))
    tag     : tag lookup and replacement for batch t+2                              (HBM, small)

so the host-link traffic of the next batch and the tag work of the one after it overlap the
training of the current batch.

Why this is safe with lock_depth >= 1.  The tag step of batch t+2 may only take ways stamped before
t+2-lock_depth; it waits for the backward of the newest such batch (batch t for lock_depth 1, batch
t-1 for lock_depth 2, which takes the tag step off the critical path), so it only evicts rows whose
batches have trained, and never a way of a batch that is still waiting to train.  Its decisions read and write tags, timestamps
and the dirty bytes of its victims only; forward/backward write none of the first two and only the
dirty bytes of their own batch's slots.  The data movement of batch t+1 touches victim slots (trained
at t-1 or earlier, complete because the tag step waited for backward(t-1)) and the slots of missed
rows, which no batch in flight uses.  One hazard is left: a row that found no evictable way in batch
t (it is read and updated in host memory directly) and is fetched from host memory for batch t+1,
possibly before backward(t) has updated it.  When batch t reported such overflow, the data movement
of batch t+1 still runs at once, and after backward(t) the rows of batch t's overflow list that batch
t+1 placed are copied from host memory again (mts_cache_refetch_overflowed with placed_step = the step
of batch t+1: the tag step of batch t+2 may already have placed other keys of that list, in slots that
hold their victims' rows until batch t+2's data movement, and those must not be touched).  A row that
overflowed in batch t-1 and is first placed by batch t+1 is covered by ordering: the data movement of
batch t+1 waits for backward(t-1).
"""
from __future__ import annotations

from typing import Callable, List, Optional

import numpy as np
import torch

from . import binding as mb
from .harness import DeviceModel


class CachedTrainer:
    def __init__(self, model: DeviceModel, pipelined: bool = True, host_gather: bool = False):
        """host_gather: missed rows are gathered by host threads into a pinned buffer and moved by the
        copy engine, instead of being read over the host link by a kernel."""
        assert model.cached
        self.m = model
        self.host_gather = host_gather
        if host_gather:
            model.enable_host_gather()
        self._ev_prev_ready = None
        self.pipelined = pipelined
        self.dev = model.device
        self.main = torch.cuda.current_stream(self.dev)
        self.tag = torch.cuda.Stream(self.dev, priority=-1) if pipelined else self.main
        # the data movement needs few thread blocks but must not queue behind the training kernels' blocks;
        # one stream per cache, so that the caches' row fetches share the host link instead of taking turns
        n_c = len(model.caches)
        self.moves = [torch.cuda.Stream(self.dev, priority=-1) if pipelined else self.main for _ in range(n_c)]
        self.fix = torch.cuda.Stream(self.dev, priority=-1) if pipelined else self.main
        self.copy = torch.cuda.Stream(self.dev, priority=-1)       # miss keys to the host (host_gather)
        self.host_counters = [torch.zeros((n_c, mb.NUM_COUNTERS), dtype=torch.int64).pin_memory()
                              for _ in range(DeviceModel.N_CTX)]
        self.history: List[np.ndarray] = []           # per batch [n_caches, NUM_COUNTERS]
        self.record_timeline = False                  # set to True to time every phase with events
        self._marks = []

    def _mark(self, name, t, stream):
        if self.record_timeline:
            e = torch.cuda.Event(enable_timing=True)
            e.record(stream)
            self._marks.append((name, t, e))

    def timeline(self):
        """[(phase, batch, ms since the first mark)] after a run with record_timeline = True."""
        if not self._marks:
            return []
        torch.cuda.synchronize(self.dev)
        base = self._marks[0][2]
        return [(n, t, base.elapsed_time(e)) for n, t, e in self._marks]

    def _lookup(self, t, step, batch, ev_tags, wait_event):
        """Tag path of batch t on the tag stream (into context t mod 3)."""
        m, s, ctx = self.m, self.tag, t % DeviceModel.N_CTX
        if wait_event is not None:
            s.wait_event(wait_event)
        self._mark("tag_begin", t, s)
        m.cache_lookup(batch[0], batch[1], batch[2], step, stream=s, ctx=ctx)
        self._mark("tag_end", t, s)
        with torch.cuda.stream(s):
            for g in range(len(m.caches)):
                self.host_counters[ctx][g].copy_(m.ctx[ctx]["lists"][g]["counters"], non_blocking=True)
        ev_tags.record(s)

    def _move(self, t, ev_tags, ev_ready, prev_overflow, prev_bwd):
        """Data path of batch t, each cache on its own move stream.  prev_overflow: number of rows of
        batch t-1 that found no way (0 = none), prev_bwd: event after batch t-1's backward."""
        ctx = t % DeviceModel.N_CTX
        refetch = wait_bwd = False
        if prev_overflow:
            cap = min(L["capacity"] for L in self.m.ctx[(t - 1) % DeviceModel.N_CTX]["lists"])
            if prev_overflow <= cap:
                refetch = True                       # move now, repair the few stale rows afterwards
            else:
                wait_bwd = True                      # the list was cut: wait for the backward first
        ends = []
        for g, s in enumerate(self.moves):
            s.wait_event(ev_tags)
            if wait_bwd:
                s.wait_event(prev_bwd)
            self._mark(f"move{g}_begin", t, s)
            # fetch, then write back, in stream order: the next batch's fetch of this cache, which may
            # miss a row written back now, comes after it on the same stream
            done = False
            if self.host_gather:
                # the host reads the rows itself: the tag step of this batch is over (its counters are on
                # the host), and every write-back of earlier batches has reached host memory (the
                # previous batch's data movement is over)
                if g == 0:
                    ev_tags.synchronize()
                    if self._ev_prev_ready is not None:
                        self._ev_prev_ready.synchronize()
                    if wait_bwd:
                        prev_bwd.synchronize()
                n_miss = int(self.host_counters[ctx][g][mb.COUNTER_NAMES.index("inserted")])
                done = self.m.cache_fetch_via_host(g, n_miss, self.copy, s, ctx,
                                                   mark=(lambda name, s=s: self._mark(name, t, s)) if self.record_timeline else None)
            if not done:
                self.m.cache_fetch(g, stream=s, ctx=ctx)
            self._mark(f"placed{g}", t, s)
            self.m.cache_writeback(g, stream=s, ctx=ctx)
            self._mark(f"move{g}_end", t, s)
            e = torch.cuda.Event()
            e.record(s)
            ends.append(e)
        # the repair of stale rows waits for the previous backward; on its own stream it does not hold
        # up the next batch's data movement
        s = self.fix
        for e in ends:
            s.wait_event(e)
        if refetch:
            s.wait_event(prev_bwd)
            self._mark("refetch_begin", t, s)
            self.m.cache_refetch((t - 1) % DeviceModel.N_CTX, placed_step=self._first_step + t, stream=s)
        self._mark("ready", t, s)
        ev_ready.record(s)
        self._ev_prev_ready = ev_ready

    def _counters(self, t, ev_tags) -> int:
        ev_tags.synchronize()                        # counters of batch t are on the host
        cnt = self.host_counters[t % DeviceModel.N_CTX].numpy().copy()
        self.history.append(cnt)
        return int(cnt[:, mb.COUNTER_NAMES.index("overflow")].max())

    def run(self, batches, grads, out: Optional[torch.Tensor] = None,
            on_step: Optional[Callable[[int], None]] = None, first_step: int = 0) -> None:
        """Train on `batches` = [(indices_dev, offsets_dev, offsets_host)], `grads` = [grad_out_dev]."""
        m = self.m
        K = len(batches)
        if K == 0:
            return
        self._first_step = first_step
        ev_tags = [torch.cuda.Event() for _ in range(K)]
        ev_ready = [torch.cuda.Event() for _ in range(K)]
        ev_bwd = [torch.cuda.Event() for _ in range(K)]
        if out is None:
            out = torch.empty((m.spec.batch, m.spec.total_dim), dtype=torch.float32, device=self.dev)
        if not self.pipelined:
            for t in range(K):
                idx, off, _ = batches[t]
                self._lookup(t, first_step + t, batches[t], ev_tags[t], None)
                self._move(t, ev_tags[t], ev_ready[t], 0, None)
                m.forward(idx, off, idx.numel(), out=out, stream=self.main, ctx=t % DeviceModel.N_CTX)
                m.backward(idx, off, idx.numel(), grads[t], stream=self.main, ctx=t % DeviceModel.N_CTX)
                self._counters(t, ev_tags[t])
                if on_step is not None:
                    on_step(t)
            return
        # the side streams must see the inputs produced on the main stream
        start = torch.cuda.Event()
        start.record(self.main)
        self.tag.wait_event(start)
        for s in self.moves + [self.fix]:
            s.wait_event(start)
        overflow = {}
        self._lookup(0, first_step, batches[0], ev_tags[0], None)
        self._move(0, ev_tags[0], ev_ready[0], 0, None)
        overflow[0] = self._counters(0, ev_tags[0])
        if K > 1:
            self._lookup(1, first_step + 1, batches[1], ev_tags[1], None)
        for t in range(K):
            idx, off, _ = batches[t]
            self.main.wait_event(ev_ready[t])
            self._mark("fwd_begin", t, self.main)
            m.forward(idx, off, idx.numel(), out=out, stream=self.main, ctx=t % DeviceModel.N_CTX)
            self._mark("fwd_end", t, self.main)
            m.backward(idx, off, idx.numel(), grads[t], stream=self.main, ctx=t % DeviceModel.N_CTX)
            self._mark("bwd_end", t, self.main)
            ev_bwd[t].record(self.main)
            if t + 2 < K:
                # the tag step of batch t+2 may evict rows stamped before t+2-lock_depth: the backward
                # of the last such batch must be over (with lock_depth 1 that is batch t, with 2 batch
                # t-1); the context it writes was last used by batch t-1.  Enqueued before the data movement
                # of batch t+1, whose host part (counters, row gather) blocks this thread
                last = min(t, t + 1 - m.lock_depth)
                # it rewrites the context of batch t-1, whose overflow list and counters the repair step
                # inside the data movement of batch t still reads: after that
                self.tag.wait_event(ev_ready[t])
                self._lookup(t + 2, first_step + t + 2, batches[t + 2], ev_tags[t + 2],
                             ev_bwd[last] if last >= 0 else None)
            if t + 1 < K:
                overflow[t + 1] = self._counters(t + 1, ev_tags[t + 1])
                if t >= 1:
                    # a row that overflowed in batch t-1 (updated in host memory by its backward) and is
                    # placed only now is fetched from host memory: after that backward
                    for s in self.moves:
                        s.wait_event(ev_bwd[t - 1])
                    if self.host_gather:
                        ev_bwd[t - 1].synchronize()
                self._move(t + 1, ev_tags[t + 1], ev_ready[t + 1], overflow[t], ev_bwd[t])
            if on_step is not None:
                on_step(t)
        self.main.wait_stream(self.tag)
        for s in self.moves + [self.fix]:
            self.main.wait_stream(s)
