"""Schedule of the cached train step (Section 5.7 of the paper: prefetch into the cache ahead of
training; Section 6.1: cache kernels on their own streams, synchronised with the next batch's
lookups).  Streams, ordered by events only:

    main    : forward(t), backward(t)
    tag     : tag lookup and replacement, two batches ahead of the training
    move[g] : cache g: save victims / fetch missed rows / write victims back for the batches ahead  (host link)
    save[g] : cache g, copy-engine path: victims saved and copied to the host beside the fetch on move[g]
    fix     : repair of rows that overflowed in batches t and t-1 and were placed by batch t+1

so the tag step and the host-link traffic of the batches ahead overlap the training of the current batch; the
launching thread never waits for the device.  The tag step is a train of some forty kernels, most of them
bound by latency; beside the training kernels (bound by the L1 / L2 data paths) both slow down, but the pair
finishes sooner than one after the other (configuration 4: 5.4 ms per batch against 5.9).  tag_on_main = True
runs the tag step of batch t + lock_depth + 1 after the backward of batch t on the training stream instead:
both run at their own speed and the data movement gets lock_depth batches of time, which is the better
schedule when the data movement, not the GPU, sets the pace.

Why this is safe with lock_depth >= 1.  The tag step of batch t may only take ways stamped before
t - lock_depth; it waits for the backward of the newest such batch (t - 1 - lock_depth), so it only
evicts rows whose batches have trained and never a way of a batch that is still waiting to train.
Its decisions read and write tags, timestamps and the dirty bytes of its victims only;
forward/backward write none of the first two and only the dirty bytes of their own batch's slots.
The data movement of batch t touches victim slots (complete, because the tag step waited for their
batches) and the slots of missed rows, which no batch in flight uses; a cache's movements follow
one another on one stream, so a row written back by one batch is in host memory before a later
batch fetches it.

Rows that found no evictable way ("overflow": read and updated in host memory directly) need one
more rule.  Batch t's data movement may run before the backward passes of batches t-1 ... t-lock_depth
have updated such rows in host memory; if batch t places one of them, its copy in the cache can be
stale.  After the backward of batch t-1 (and the data movement of batch t), the keys of the overflow
lists of batches t-1 ... t-lock_depth that are resident in a way stamped t are therefore copied from
host memory again (mts_cache_refetch_overflowed with placed_step = t; the stamp keeps the repair away
from keys that a tag step running further ahead has placed in slots that still hold their victims'
rows).  Older overflowed rows need nothing: the tag step of batch t already waited for their backward.

Batch contexts (DeviceModel.N_CTX = 6): the tag step of batch t rewrites the context batch t-6 used,
whose overflow list the repair before batch t-4 was the last to read, so it also waits for that repair
(long over in practice: the contexts are many so that this wait never holds the tag step back).

With host_gather the missed rows do not cross the host link at the request of SMs (small reads that
slow every kernel beside them): one worker thread per cache reads the miss list, gathers the rows with
the host's threads into a pinned buffer and enqueues one contiguous copy and the placing kernel, without
waiting for them: while they run it already handles the next batch.  The victims of a batch are final when
its tag step ends, so they are saved and copied out on save[g] at once (the placing kernel waits for the
save); the worker puts them into their host rows before its next gather, which may read one of them.  One more
thread enqueues the repair once all caches of a batch have moved.  The workers run ahead of the launching
thread; host-side flags tell each side which events the other has recorded.  By default the worker of a
cache is a thread of the library (mts_mover: the same calls in the same order, without the interpreter and
its lock in the loop: 1.9 -> 1.7 ms per batch on configuration 5, 0.43 -> 0.28 ms at batch 1024); the Python
worker below makes the same calls and is used when the phases are timed with events.
"""
from __future__ import annotations

import queue
import threading
import time
from typing import Callable, List, Optional

import numpy as np
import torch

from . import binding as mb
from .harness import DeviceModel


class CachedTrainer:
    def __init__(self, model: DeviceModel, pipelined: bool = True, host_gather: bool = False, tag_on_main: bool = False,
                 native_mover: Optional[bool] = None):
        """host_gather: missed rows are gathered by host threads into a pinned buffer and moved by the
        copy engine, instead of being read over the host link by a kernel.
        tag_on_main: the tag step of batch t + lock_depth + 1 follows the backward of batch t on the training
        stream, instead of running two batches ahead on a stream of its own (see the module docstring).
        native_mover (pipelined with host_gather): the caches' data paths run on threads of the library
        (mts_mover) instead of Python threads; None = yes, unless the phases are timed (record_timeline)."""
        self.native_mover = native_mover
        self._movers = None
        self._mover_seen = [{} for _ in model.caches]
        self._native = False
        self._submitted = []
        assert model.cached
        # the side streams run two batches ahead and keep two overflow lists alive: lock depths 1 and 2
        assert not pipelined or 1 <= model.lock_depth <= 2, "the pipelined schedule needs lock_depth 1 or 2"
        assert not (model.l2 and (pipelined or host_gather)), "two cache levels: sequential schedule, kernel data movement"
        self.m = model
        self.host_gather = host_gather
        if host_gather:
            model.enable_host_gather()
        self.pipelined = pipelined
        self.dev = model.device
        self.main = torch.cuda.current_stream(self.dev)
        self.tag_on_main = tag_on_main
        self.tag = torch.cuda.Stream(self.dev, priority=-1) if (pipelined and not tag_on_main) else self.main
        # the data movement needs few thread blocks but must not queue behind the training kernels' blocks;
        # one stream per cache, so that the caches' row traffic shares the host link instead of taking turns
        n_c = len(model.caches)
        self.moves = [torch.cuda.Stream(self.dev, priority=-1) if pipelined else self.main for _ in range(n_c)]
        self.fix = torch.cuda.Stream(self.dev, priority=-1) if pipelined else self.main
        self.copies = [torch.cuda.Stream(self.dev, priority=-1) for _ in range(n_c)]    # miss keys to the host (host_gather)
        # victims to the host (host_gather), beside the cache's fetch
        self.saves = [torch.cuda.Stream(self.dev, priority=-1) if pipelined else self.main for _ in range(n_c)]
        self.history: List[np.ndarray] = []           # per batch [n_caches, NUM_COUNTERS], filled when run() returns
        self.record_timeline = False                  # set to True to time every phase with events
        self._marks = []
        self._host_marks = []
        self._mark_lock = threading.Lock()
        self.debug_delay_cycles = 0                   # > 0: the move and repair streams idle that long before their work

    def close(self):
        """Stops the library's mover threads (after run() has returned)."""
        if self._movers is not None:
            for mv in self._movers:
                mv.close()
            self._movers = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _delay(self, stream):
        """Test aid: hold a side stream back so that the training and the tag step run far ahead of it."""
        if self.debug_delay_cycles > 0:
            with torch.cuda.stream(stream):
                torch.cuda._sleep(int(self.debug_delay_cycles))

    def _mark(self, name, t, stream):
        if self.record_timeline:
            e = torch.cuda.Event(enable_timing=True)
            e.record(stream)
            with self._mark_lock:
                self._marks.append((name, t, e))

    def _host_mark(self, name, t, g):
        if self.record_timeline:
            with self._mark_lock:
                self._host_marks.append((name, t, g, time.perf_counter()))

    def host_phases(self):
        """{phase: mean ms} a cache's worker thread spent between consecutive host marks (record_timeline = True)."""
        by = {}
        for name, t, g, at in self._host_marks:
            by.setdefault((t, g), []).append((at, name))
        tot, cnt = {}, {}
        for marks in by.values():
            marks.sort()
            for (a0, _), (a1, n1) in zip(marks, marks[1:]):
                tot[n1] = tot.get(n1, 0.0) + (a1 - a0) * 1e3
                cnt[n1] = cnt.get(n1, 0) + 1
        return {n: tot[n] / cnt[n] for n in tot}

    def timeline(self):
        """[(phase, batch, ms since the first mark)] after a run with record_timeline = True."""
        if not self._marks:
            return []
        torch.cuda.synchronize(self.dev)
        base = self._marks[0][2]
        return [(n, t, base.elapsed_time(e)) for n, t, e in self._marks]

    # ------------------------------------------------------------------ the three phases of a batch
    def _lookup(self, t, batch):
        """Tag path of batch t on the tag stream (into context t mod N_CTX); its counters go to row t of the
        pinned history buffer."""
        m, s, ctx = self.m, self.tag, t % DeviceModel.N_CTX
        if self.pipelined:
            if t - DeviceModel.N_CTX + 2 >= 0:                  # the last repair that read this context's lists
                s.wait_event(self.ev_ready[t - DeviceModel.N_CTX + 2])
            last = t - 1 - m.lock_depth                         # newest batch whose rows may be evicted now
            if last >= 0:
                s.wait_event(self.ev_bwd[last])
        self._mark("tag_begin", t, s)
        m.cache_lookup(batch[0], batch[1], batch[2], self._first_step + t, stream=s, ctx=ctx)
        self._mark("tag_end", t, s)
        with torch.cuda.stream(s):
            for g in range(len(m.caches)):
                L = m.ctx[ctx]["lists"][g]
                self._host_counters[t, g].copy_(L["counters2"] if m.l2 else L["counters"], non_blocking=True)
        self.ev_tags[t].record(s)

    def _move_cache(self, t, g, via_host):
        """Data path of batch t for cache g.  Kernel path: fetch, then write back, on the cache's move stream
        (the next batch's fetch of this cache, which may miss a row written back now, follows on the same
        stream).  Copy-engine path: the victims are saved and copied out on the cache's second stream as soon
        as the tag step is over, while this thread puts the previous batch's victims into their host rows and
        gathers the missed rows; the copy of the gathered rows and the placing kernel are only enqueued, so
        the thread goes on to the next batch while they run."""
        s, ctx = self.moves[g], t % DeviceModel.N_CTX
        s.wait_event(self.ev_tags[t])
        self._delay(s)
        self._mark(f"move{g}_begin", t, s)
        done = False
        if via_host:
            # the host reads the rows itself: the tag step of this batch is over (its counters are on the host)
            self._host_mark("job_begin", t, g)
            self.ev_tags[t].synchronize()
            self._host_mark("tag_waited", t, g)
            n_miss = int(self._host_counters[t, g, mb.COUNTER_NAMES.index("inserted")])
            n_evict = int(self._host_counters[t, g, mb.COUNTER_NAMES.index("evicted")])
            if not self.m.host_lists_fit(g, n_miss, n_evict) and self.m.host_buffers_can_hold(g, max(n_miss, n_evict)):
                # longer lists than any before: larger buffers, once nothing of this cache is in flight
                self._finish_writeback(g)
                for q in (self.copies[g], self.saves[g], s):
                    q.synchronize()
                self.m.grow_host_buffers(g, max(n_miss, n_evict) * 5 // 4)
            if self.m.host_lists_fit(g, n_miss, n_evict):
                self.m.cache_request_miss_keys(g, n_miss, self.copies[g], ctx)      # ahead of the victims' copies
                w = self.saves[g]
                w.wait_event(self.ev_tags[t])
                self._delay(w)
                saved = self.m.cache_save_victims_via_host(g, n_evict, w, ctx)
                copied = torch.cuda.Event()
                copied.record(w)
                self._host_mark("victims_enqueued", t, g)
                # this cache's write-backs of earlier batches reach host memory before the gather reads it
                self._finish_writeback(g)
                self._host_mark("scattered", t, g)
                self._pending_wb[g] = (copied, n_evict, ctx)
                self.m.cache_fetch_via_host(
                    g, n_miss, self.copies[g], s, ctx, saved,
                    mark=(lambda name, s=s: self._mark(name, t, s)) if self.record_timeline else None)
                self._host_mark("gathered_enqueued", t, g)
                if not self.pipelined:
                    self._finish_writeback(g)
                done = True
        if not done:
            if via_host:
                self._finish_writeback(g)
            self.m.cache_fetch(g, stream=s, ctx=ctx)
            self.m.cache_writeback(g, stream=s, ctx=ctx)
        self._mark(f"placed{g}", t, s)
        self._mark(f"move{g}_end", t, s)
        self.ev_moved[t][g].record(s)
        if via_host:
            self._host_mark("job_end", t, g)
        if via_host and not done:
            self.ev_moved[t][g].synchronize()       # the kernels' write-back is in host memory before the next gather

    def _finish_writeback(self, g):
        """Cache g: the victims whose copy to the host was enqueued by an earlier batch go into their rows."""
        pend = self._pending_wb[g]
        if pend is not None:
            e, n_evict, ctx = pend
            e.synchronize()
            self.m.cache_writeback_via_host_finish(g, n_evict, ctx)
            self._pending_wb[g] = None

    def _finish_move(self, t, waited=False):
        """After the data movement of batch t: repair the rows that overflowed in the batches whose backward may
        have run after their copy was taken, then batch t is ready to train.  waited: the repair stream already
        waits for the batch's data movement (the library's movers arranged that)."""
        s = self.fix
        if not waited:
            for e in self.ev_moved[t]:
                s.wait_event(e)
        if self.pipelined and t >= 1:
            s.wait_event(self.ev_bwd[t - 1])
            self._delay(s)
            self._mark("refetch_begin", t, s)
            for k in range(1, self.m.lock_depth + 1):
                if t - k >= 0:
                    self.m.cache_refetch((t - k) % DeviceModel.N_CTX, placed_step=self._first_step + t, stream=s)
        self._mark("ready", t, s)
        self.ev_ready[t].record(s)

    def _move(self, t):
        for g in range(len(self.moves)):
            self._move_cache(t, g, self.host_gather)
        self._finish_move(t)

    # ------------------------------------------------------------------ worker threads (host_gather, pipelined)
    def _fail(self, e):
        self._worker_error = e
        for f in self._ready_recorded:
            f.set()
        for f in self._submitted:
            f.set()
        for row in self._moved_recorded:
            for f in row:
                f.set()

    def _cache_worker(self, g):
        """Batch after batch, the data path of cache g."""
        try:
            torch.cuda.set_device(self.dev)
            while True:
                t = self._jobs[g].get()
                if t is None:
                    self._finish_writeback(g)
                    return
                self._move_cache(t, g, True)
                self._moved_recorded[t][g].set()
        except BaseException as e:                              # surface the failure in the launching thread
            self._fail(e)

    def _finisher(self, K):
        """Batch after batch: once every cache has enqueued its data path and the launching thread has recorded
        the previous backward, enqueue the repair and the batch's ready event."""
        try:
            torch.cuda.set_device(self.dev)
            for t in range(K):
                if self._native:
                    self._submitted[t].wait()
                    if self._stop.is_set() or self._worker_error is not None:
                        return
                    # blocks until each mover has recorded the batch's "moved" event, then the repair stream waits for it
                    for g, mv in enumerate(self._movers):
                        mv.stream_wait_moved(self._job_of[t][g], self.fix)
                else:
                    for f in self._moved_recorded[t]:
                        f.wait()
                if t >= 1:
                    self._bwd_recorded[t - 1].wait()            # the repair waits for that event on the device
                if self._stop.is_set() or self._worker_error is not None:
                    return
                self._finish_move(t, waited=self._native)
                self._ready_recorded[t].set()
        except BaseException as e:
            self._fail(e)

    def _submit_move(self, t):
        """Batch t to the library's movers (one per cache), which run its data path on their own threads."""
        m, ctx = self.m, t % DeviceModel.N_CTX
        tag_done = self.ev_tags[t].cuda_event
        for g, mv in enumerate(self._movers):
            self._delay(self.moves[g])
            self._delay(self.saves[g])
            L = m.ctx[ctx]["lists"][g]
            self._job_of[t][g] = mv.submit(L["miss_keys"], L["miss_slots"], L["evict_keys"], L["evict_slots"],
                                           L["evict_dirty"], L["capacity"], L["counters"], self._host_counters[t, g],
                                           L["staging"], tag_done, self.moves[g], self.saves[g], self.copies[g])
        self._submitted[t].set()

    def _wait_ready_recorded(self, t):
        if self._threads:
            self._ready_recorded[t].wait()
            if self._worker_error is not None:
                raise self._worker_error

    def run(self, batches, grads, out: Optional[torch.Tensor] = None,
            on_step: Optional[Callable[[int], None]] = None, first_step: int = 0,
            after_backward: Optional[Callable[[int], None]] = None, pause_gc: bool = True) -> None:
        """Train on `batches` = [(indices_dev, offsets_dev, offsets_host)], `grads` = [grad_out_dev].
        after_backward(t) is called when batch t's backward has been enqueued and before any later work that
        may reuse its context; on_step(t) at the end of iteration t.
        pause_gc: the launching thread and the workers are Python threads, and a collection of the interpreter's
        oldest generation stalls all of them for milliseconds (measured: 5.5 -> 6.9 ms per batch on configuration 4
        in a process that had run other workloads before); the cyclic collector is off while the batches run."""
        import gc
        paused = pause_gc and gc.isenabled()
        if paused:
            gc.collect()
            gc.disable()
        try:
            self._run(batches, grads, out, on_step, first_step, after_backward)
        finally:
            if paused:
                gc.enable()

    def _run(self, batches, grads, out, on_step, first_step, after_backward) -> None:
        m = self.m
        K = len(batches)
        if K == 0:
            return
        self._first_step = first_step
        n_c = len(m.caches)
        self.ev_tags = [torch.cuda.Event() for _ in range(K)]
        self.ev_ready = [torch.cuda.Event() for _ in range(K)]
        self.ev_bwd = [torch.cuda.Event() for _ in range(K)]
        self.ev_moved = [[torch.cuda.Event() for _ in range(n_c)] for _ in range(K)]
        n_cnt = mb.NUM_COUNTERS2 if m.l2 else mb.NUM_COUNTERS
        self._host_counters = torch.zeros((K, n_c, n_cnt), dtype=torch.int64).pin_memory()
        self._threads = []
        self._native = False
        self._worker_error = None
        self._pending_wb = [None] * n_c
        if out is None:
            out = torch.empty((m.spec.batch, m.spec.total_dim), dtype=torch.float32, device=self.dev)

        def train(t):
            idx, off, _ = batches[t]
            ctx = t % DeviceModel.N_CTX
            self._mark("fwd_begin", t, self.main)
            m.forward(idx, off, idx.numel(), out=out, stream=self.main, ctx=ctx)
            self._mark("fwd_end", t, self.main)
            m.backward(idx, off, idx.numel(), grads[t], stream=self.main, ctx=ctx)
            self._mark("bwd_end", t, self.main)
            if after_backward is not None:
                after_backward(t)

        if not self.pipelined:
            for t in range(K):
                self._lookup(t, batches[t])
                self._move(t)
                train(t)
                if on_step is not None:
                    on_step(t)
            torch.cuda.synchronize(self.dev)
            self.history.extend(self._host_counters.numpy().copy())
            return

        # the side streams must see the inputs produced on the main stream
        start = torch.cuda.Event()
        start.record(self.main)
        for s in [self.tag, self.fix] + self.copies + self.moves + self.saves:
            s.wait_event(start)
        if self.host_gather:
            self._jobs = [queue.Queue() for _ in range(n_c)]
            self._ready_recorded = [threading.Event() for _ in range(K)]
            self._bwd_recorded = [threading.Event() for _ in range(K)]
            self._moved_recorded = [[threading.Event() for _ in range(n_c)] for _ in range(K)]
            self._stop = threading.Event()
            # the caches' data paths: threads of the library (movers), or Python threads when the phases are
            # to be timed with events (record_timeline) or the caller asked for them
            self._native = self.native_mover if self.native_mover is not None else not self.record_timeline
            self._submitted = [threading.Event() for _ in range(K)]
            self._job_of = [[0] * n_c for _ in range(K)]
            if self._native:
                if self._movers is None:
                    self._movers = [mb.Mover(c, m.host_rows_ptr(g), c.dim * m.spec.elem_bytes, m.gather_threads,
                                             DeviceModel.N_CTX, m.FETCH_STAGE_BYTES, max(m.FETCH_STAGE_MAX_BYTES, m.FETCH_STAGE_BYTES))
                                    for g, c in enumerate(m.caches)]
                self._threads = []
            else:
                self._threads = [threading.Thread(target=self._cache_worker, args=(g,), daemon=True) for g in range(n_c)]
            self._threads.append(threading.Thread(target=self._finisher, args=(K,), daemon=True))
            for th in self._threads:
                th.start()

        def start_move(t):
            """The data path of batch t, as soon as its tag step is enqueued."""
            if self._threads and self._native:
                self._submit_move(t)       # ev_tags[t] has been recorded by this thread already
            elif self._threads:
                for q in self._jobs:
                    q.put(t)
            else:
                for g in range(n_c):
                    self._move_cache(t, g, False)

        def finish_move(t):
            """The repair and the ready event of batch t; needs the event of the backward of batch t-1."""
            if not self._threads:          # with worker threads the finisher thread does this
                self._finish_move(t)

        # batches the tag step runs ahead of the training: it may evict rows of batches up to its own minus
        # lock_depth + 1, and those must have trained
        ahead = m.lock_depth + 1 if self.tag_on_main else 2
        try:
            for t in range(min(ahead, K)):
                self._lookup(t, batches[t])
                start_move(t)
            finish_move(0)
            for t in range(K):
                self._wait_ready_recorded(t)
                self.main.wait_event(self.ev_ready[t])
                train(t)
                self.ev_bwd[t].record(self.main)
                if self._threads:
                    self._bwd_recorded[t].set()
                if t + 1 < K:
                    finish_move(t + 1)
                if t + ahead < K:
                    self._lookup(t + ahead, batches[t + ahead])
                    start_move(t + ahead)
                if on_step is not None:
                    on_step(t)
        finally:
            if self._threads:
                if any(not f.is_set() for f in self._ready_recorded):      # an error in this thread: release the others
                    self._stop.set()
                for f in self._bwd_recorded:
                    f.set()
                for q in self._jobs:
                    q.put(None)
                for row in self._moved_recorded:
                    for f in row:
                        f.set()
                for f in self._submitted:
                    f.set()
                for th in self._threads:
                    th.join()
                if self._native and self._worker_error is None:
                    for g, mv in enumerate(self._movers):
                        mv.drain()             # the last victims into their host rows
                        st, cur = m.host_copy_stats[g], mv.stats()
                        for k in ("gather_s", "gather_bytes", "scatter_s", "scatter_bytes"):
                            st[k] += cur[k] - self._mover_seen[g].get(k, 0.0)
                        self._mover_seen[g] = cur
                self._threads = []
                if self._worker_error is not None:
                    raise self._worker_error
        for s in [self.tag, self.fix] + self.copies + self.moves + self.saves:
            self.main.wait_stream(s)
        torch.cuda.synchronize(self.dev)
        self.history.extend(self._host_counters.numpy().copy())
