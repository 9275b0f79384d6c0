"""Torch plumbing around the C ABI: device buffers for one model, one call per step of the path.

Nothing here computes anything on its own; every step is a call into libmtrains_b200.so.
"""
from __future__ import annotations

import os
import threading
import time
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as mb
from . import workload as wl


class DeviceModel:
    """Weights, optimizer state and scratch of one ModelSpec on one GPU.

    Tables are either HBM resident (one flat device buffer) or host resident (one flat pinned host
    buffer, device-visible through unified addressing) behind one cache per embedding dim.  By default
    an uncached spec keeps every table in HBM and a cached spec every table in the host tier;
    `host_tables` (one bool per table) mixes the two in one model."""

    N_CTX = 6        # batch contexts: batch t trains, the rows of t+1 move, the tags of t+2 are looked up, the
    #                  overflow lists of t-1 and t-2 are still needed for repairs; two more so that the tag step
    #                  never has to wait for the repair that last read the context it rewrites

    def __init__(self, spec: wl.ModelSpec, device="cuda:0", max_lookups: int = 0, weights: Optional[np.ndarray] = None,
                 lock_depth: int = 0, policy: int = mb.POLICY_LRU, cache_sets: Optional[List[int]] = None,
                 host_tables: Optional[Sequence[bool]] = None, l2_fraction: float = 0.0):
        """l2_fraction > 0: every cache gets a second, exclusive level in pinned host memory holding that share
        of its table group's rows (two-level hierarchy; sequential schedule only)."""
        self.spec = spec
        self.lock_depth = lock_depth
        self.l2_fraction = float(l2_fraction)
        self.l2: List[mb.Cache] = []
        self.device = torch.device(device)
        self.tdtype = torch.float32 if spec.dtype == wl.FP32 else torch.float16
        n_elem = int(spec.weight_offset[-1])
        if host_tables is None:
            host_tables = [bool(spec.cached)] * spec.T
        self.host_tables = [bool(x) for x in host_tables]
        self.cached = any(self.host_tables)
        self.all_cached = all(self.host_tables)
        self.host_weights = torch.empty(n_elem, dtype=self.tdtype, pin_memory=True) if self.cached else None
        self.dev_weights = None if self.all_cached else torch.empty(n_elem, dtype=self.tdtype, device=self.device)
        for t in range(spec.T):
            a, b = int(spec.weight_offset[t]), int(spec.weight_offset[t + 1])
            store = self.host_weights if self.host_tables[t] else self.dev_weights
            if weights is not None:
                store[a:b].copy_(torch.from_numpy(weights[a:b]))
                continue
            dst = store[a:b].view(-1, int(spec.dims[t]))
            step = 1 << 22
            for r0 in range(0, int(spec.rows[t]), step):
                r1 = min(r0 + step, int(spec.rows[t]))
                dst[r0:r1].copy_(wl.weights_torch(spec, t, self.device, r0, r1))
        self.momentum = torch.zeros(int(spec.row_offset[-1]), dtype=torch.float32, device=self.device)
        self.caches: List[mb.Cache] = []
        # one cache per run of consecutive host-tier tables of one dim
        self.groups = []
        t = 0
        while t < spec.T:
            if not self.host_tables[t]:
                t += 1
                continue
            t1 = t
            while t1 < spec.T and self.host_tables[t1] and spec.dims[t1] == spec.dims[t]:
                t1 += 1
            self.groups.append((int(spec.dims[t]), t, t1))
            t = t1
        cache_id = None
        if self.cached:
            cache_id = np.full(spec.T, -1, np.int32)
            for g, (dim, t0, t1) in enumerate(self.groups):
                cache_id[t0:t1] = g
                rows_g = int(spec.row_offset[t1] - spec.row_offset[t0])
                sets = cache_sets[g] if cache_sets is not None else wl.cache_sets_for(rows_g, spec.cache_fraction)
                self.caches.append(mb.cache_create(sets, rows_g, dim, spec.dtype, policy, lock_depth))
                if self.l2_fraction > 0.0:
                    sets2 = wl.cache_sets_for(rows_g, self.l2_fraction)
                    esz = 4 if spec.dtype == wl.FP32 else 2
                    rows2 = torch.zeros(sets2 * 32 * dim * esz, dtype=torch.uint8).pin_memory()
                    self.l2.append(mb.Cache(sets2, rows_g, dim, spec.dtype, policy, lock_depth, host_rows=rows2))
        self.tables = mb.tables_create(spec.dtype, spec.rows, spec.dims, spec.weight_offset[:-1], cache_id,
                                       self.dev_weights, self.host_weights, self.momentum)
        self.cache_data = [c.data_ptr for c in self.caches] if self.cached else None
        self.cache_dirty = [c.dirty_ptr for c in self.caches] if self.cached else None
        self.max_lookups = 0
        self.workspace = None
        self.ws_bytes = 0
        self.fetch_rows = None
        if max_lookups:
            self.reserve(max_lookups)

    # ------------------------------------------------------------------ scratch
    def reserve(self, max_lookups: int) -> None:
        max_lookups = max(int(max_lookups), 1)
        if max_lookups <= self.max_lookups:
            return
        self.max_lookups = max_lookups
        B = self.spec.batch
        self.ws_bytes = mb.tbe_backward_workspace_bytes(self.tables, B, max_lookups)
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=self.device)
        # the cache calls may run on a side stream while backward runs: scratch of their own
        self.cache_ws_bytes = max([mb.cache_workspace_bytes(c, max_lookups) for c in self.caches] + [256])
        if self.l2:
            self.cache_ws_bytes = max(mb.cache2_workspace_bytes(a, b, max_lookups, max_lookups) for a, b in zip(self.caches, self.l2))
            esz = 4 if self.spec.dtype == wl.FP32 else 2
            self.fetch_staging2 = torch.empty(max_lookups * max(c.dim for c in self.caches) * esz, dtype=torch.uint8,
                                              device=self.device)
        self.cache_ws = torch.empty(self.cache_ws_bytes, dtype=torch.uint8, device=self.device)
        if self.cached:
            # the victim staging buffer is only used inside one data movement call sequence, so one per
            # cache serves all batch contexts
            esz = 4 if self.spec.dtype == wl.FP32 else 2
            self.staging = [torch.empty(min(max_lookups, c.num_sets * c.ways) * c.dim * esz, dtype=torch.uint8,
                                        device=self.device) for c in self.caches]
            self.ctx = [self._new_context(max_lookups) for _ in range(self.N_CTX)]
            self.cur = 0

    def _new_context(self, n: int):
        dev = self.device
        lists = []
        for g, c in enumerate(self.caches):
            cap = min(n, c.num_sets * c.ways)        # a call can place at most one row per slot
            lists.append(dict(
                miss_keys=torch.empty(cap, dtype=torch.int64, device=dev),
                miss_slots=torch.empty(cap, dtype=torch.int32, device=dev),
                evict_keys=torch.empty(cap, dtype=torch.int64, device=dev),
                evict_slots=torch.empty(cap, dtype=torch.int32, device=dev),
                evict_dirty=torch.empty(cap, dtype=torch.uint8, device=dev),
                overflow_keys=torch.empty(n, dtype=torch.int64, device=dev),      # never cut: n distinct keys at most
                overflow_capacity=n,
                counters=torch.zeros(mb.NUM_COUNTERS, dtype=torch.int64, device=dev),
                staging=self.staging[g],
                capacity=cap))
        if self.l2:
            # two levels: the lists of mts_cache2_lookup_insert, a key array, a staging buffer for the rows
            # on their way into the first level; the first ten counters are the one-level counters
            esz = 4 if self.spec.dtype == wl.FP32 else 2
            for g, (c, L) in enumerate(zip(self.caches, lists)):
                cap = L["capacity"] = n
                two = {name: torch.zeros(cap, dtype=t, device=dev) for name, t in (
                    ("fetch_keys", torch.int64), ("fetch_slots", torch.int32), ("fetch_src", torch.int32),
                    ("ev1_keys", torch.int64), ("ev1_slots", torch.int32), ("ev1_dirty", torch.uint8),
                    ("ev1_dst", torch.int32), ("ev2_keys", torch.int64), ("ev2_slots", torch.int32),
                    ("ev2_dirty", torch.uint8), ("drop_keys", torch.int64), ("drop_slots", torch.int32),
                    ("drop_dirty", torch.uint8))}
                L["two"] = two
                L["counters2"] = torch.zeros(mb.NUM_COUNTERS2, dtype=torch.int64, device=dev)
                L["counters"] = L["counters2"][:mb.NUM_COUNTERS]
                L["keys"] = torch.empty(n, dtype=torch.int64, device=dev)
        # the lookups ordered by row (uint32 bit patterns), written by the tag step and reused by the backward
        return dict(slot=torch.full((n,), -1, dtype=torch.int32, device=dev),
                    sorted_rows=torch.empty(n, dtype=torch.int32, device=dev),
                    sorted_bag=torch.empty(n, dtype=torch.int32, device=dev),
                    sorted_slot=torch.empty(n, dtype=torch.int32, device=dev), lists=lists)

    @property
    def slot_of_lookup(self):
        return self.ctx[self.cur]["slot"]

    @property
    def lists(self):
        return self.ctx[self.cur]["lists"]

    def _ctx(self, ctx: Optional[int]):
        return self.ctx[self.cur if ctx is None else ctx]

    # ------------------------------------------------------------------ steps of the path
    def forward(self, indices, offsets, N: int, out=None, pooling_mode: int = mb.POOL_SUM, stream=None,
                ctx: Optional[int] = None):
        if out is None:
            out = torch.empty((self.spec.batch, self.spec.total_dim), dtype=torch.float32, device=self.device)
        slot = self._ctx(ctx)["slot"] if self.cached else None
        mb.tbe_forward(self.tables, self.spec.batch, indices, offsets, N, pooling_mode, slot, self.cache_data, out,
                       out.shape[1], stream, f16=out.dtype == torch.float16, bf16=out.dtype == torch.bfloat16)
        return out

    def backward(self, indices, offsets, N: int, grad_out, lr: Optional[float] = None, eps: Optional[float] = None,
                 pooling_mode: int = mb.POOL_SUM, uniq_rows_out=None, n_unique_out=None, stream=None,
                 ctx: Optional[int] = None, reuse_tag_order: bool = True) -> None:
        """reuse_tag_order: when every table is cached, the backward takes the lookups ordered by row from
        the tag step of the same batch instead of sorting them again."""
        self.reserve(N)
        lr = self.spec.lr if lr is None else lr
        eps = self.spec.eps if eps is None else eps
        if self.all_cached and reuse_tag_order and uniq_rows_out is None and not self.l2:
            cx = self._ctx(ctx)
            mb.tbe_backward_apply_presorted(
                self.tables, self.spec.batch, offsets, N, pooling_mode, grad_out, grad_out.shape[1], lr, eps,
                cx["sorted_rows"], cx["sorted_bag"], cx["sorted_slot"], self.cache_data,
                self.cache_dirty, self.workspace, self.ws_bytes, stream, f16=grad_out.dtype == torch.float16)
            return
        if grad_out.dtype == torch.float16:      # fp16 gradients: the two-call form
            self.backward_sort(indices, offsets, N, uniq_rows_out, n_unique_out, stream)
            self.backward_apply(offsets, N, grad_out, lr, eps, pooling_mode, stream, ctx)
            return
        slot = self._ctx(ctx)["slot"] if self.cached else None
        mb.tbe_backward_rowwise_adagrad(
            self.tables, self.spec.batch, indices, offsets, N, pooling_mode, grad_out, grad_out.shape[1], lr, eps,
            slot, self.cache_data, self.cache_dirty, self.workspace, self.ws_bytes, uniq_rows_out, n_unique_out, stream)

    def backward_sort(self, indices, offsets, N: int, uniq_rows_out=None, n_unique_out=None, stream=None) -> None:
        """Index-only half of the backward; may run on another stream than the forward pass."""
        self.reserve(N)
        mb.tbe_backward_sort(self.tables, self.spec.batch, indices, offsets, N, self.workspace, self.ws_bytes,
                             uniq_rows_out, n_unique_out, stream)

    def backward_apply(self, offsets, N: int, grad_out, lr: Optional[float] = None, eps: Optional[float] = None,
                       pooling_mode: int = mb.POOL_SUM, stream=None, ctx: Optional[int] = None) -> None:
        """Gradient half of the backward, after backward_sort of the same batch."""
        slot = self._ctx(ctx)["slot"] if self.cached else None
        mb.tbe_backward_apply(
            self.tables, self.spec.batch, offsets, N, pooling_mode, grad_out, grad_out.shape[1],
            self.spec.lr if lr is None else lr, self.spec.eps if eps is None else eps,
            slot, self.cache_data, self.cache_dirty, self.workspace, self.ws_bytes, stream,
            f16=grad_out.dtype == torch.float16)

    def group_range(self, g: int, offsets_host: np.ndarray):
        """Lookup range [begin, begin + n) of cache group g in one batch (host-side CSR)."""
        _, t0, t1 = self.groups[g]
        B = self.spec.batch
        begin = int(offsets_host[t0 * B])
        return begin, int(offsets_host[t1 * B]) - begin

    def host_rows_ptr(self, g: int) -> int:
        _, t0, _ = self.groups[g]
        esz = 4 if self.spec.dtype == wl.FP32 else 2
        return self.host_weights.data_ptr() + int(self.spec.weight_offset[t0]) * esz

    def cache_lookup(self, indices, offsets, offsets_host: np.ndarray, step: int, stream=None,
                     ctx: Optional[int] = None) -> None:
        """Tag path of one batch: lookup_insert of every cache (slots, miss / evict / overflow lists, and the
        batch's lookups ordered by row for the backward)."""
        B = self.spec.batch
        cx = self._ctx(ctx)
        for g, c in enumerate(self.caches):
            _, t0, t1 = self.groups[g]
            begin, n = self.group_range(g, offsets_host)
            L = cx["lists"][g]
            if self.l2:
                keys = L["keys"][:n]
                mb.linearize_keys(self.tables, t0, t1, B, indices, offsets, begin, n, keys if n else None, stream)
                mb.cache2_lookup_insert(c, self.l2[g], keys if n else None, n, step,
                                        cx["slot"][begin:begin + n] if n else None, L["two"], L["capacity"],
                                        L["counters2"], self.cache_ws, self.cache_ws_bytes, stream)
                continue
            mb.cache_lookup_insert_tables(
                c, self.tables, t0, t1, B, indices, offsets, begin, n, step, cx["slot"], L["miss_keys"],
                L["miss_slots"], L["evict_keys"], L["evict_slots"], L["evict_dirty"], L["capacity"],
                L["overflow_keys"], L["overflow_capacity"], L["counters"], self.cache_ws, self.cache_ws_bytes, stream,
                sorted_rows_out=cx["sorted_rows"], sorted_bag_out=cx["sorted_bag"],
                sorted_slot_out=cx["sorted_slot"])

    def cache_move(self, stream=None, ctx: Optional[int] = None) -> None:
        """Data path of one batch: save dirty victims, pull missed rows from the host tier, write victims back."""
        for g in range(len(self.caches)):
            self.cache_fetch(g, stream, ctx)
            self.cache_writeback(g, stream, ctx)

    def cache_fetch(self, g: int, stream=None, ctx: Optional[int] = None) -> None:
        """Cache g: dirty victims into the staging buffer, then the missed rows from the host tier into their slots."""
        L = self._ctx(ctx)["lists"][g]
        if self.l2:
            # two levels: the whole data movement between the levels and the store is one call
            mb.cache2_move(self.caches[g], self.l2[g], self.host_rows_ptr(g), L["two"], L["capacity"], L["counters2"],
                           self.fetch_staging2, stream)
            return
        mb.cache_prefetch_misses(self.caches[g], self.host_rows_ptr(g), L["miss_keys"], L["miss_slots"],
                                 L["evict_slots"], L["evict_dirty"], L["capacity"], L["counters"], L["staging"], stream)

    # ---- missed rows gathered by host threads and moved by the copy engine
    FETCH_STAGE_BYTES = 96 << 20         # first size of the pinned buffers, per cache and batch context; they grow on demand
    FETCH_STAGE_MAX_BYTES = 256 << 20    # ... up to this size; longer lists (a cold cache's first batches) take the kernels

    def enable_host_gather(self, threads: Optional[int] = None) -> None:
        """Pinned host buffers (keys and gathered rows, per cache and batch context) and one device
        buffer per cache for the copy-engine path of the missed rows."""
        if self.fetch_rows is not None:
            return
        esz = 4 if self.spec.dtype == wl.FP32 else 2
        # every gather / scatter uses all cores; the caches' workers take turns at it (one lock), so that a cache
        # with many wide rows is not left with a third of the cores while the others idle
        self.gather_threads = threads or os.cpu_count() or 1
        self.host_copy_lock = threading.Lock()
        # seconds and bytes the host threads spent on gathers / scatters (and waiting for their turn), per cache
        self.host_copy_stats = [{"gather_s": 0.0, "gather_bytes": 0, "scatter_s": 0.0, "scatter_bytes": 0, "wait_s": 0.0}
                                for _ in self.caches]
        n_c = len(self.caches)
        self.fetch_rows = [0] * n_c
        self.fetch_dev = [None] * n_c
        self.fetch_host = [[None] * n_c for _ in range(self.N_CTX)]
        self.fetch_keys = [[None] * n_c for _ in range(self.N_CTX)]
        # the way back: dirty victims, their keys and dirty bytes
        self.wb_host = [[None] * n_c for _ in range(self.N_CTX)]
        self.wb_keys = [[None] * n_c for _ in range(self.N_CTX)]
        self.wb_dirty = [[None] * n_c for _ in range(self.N_CTX)]
        for g, c in enumerate(self.caches):
            self.grow_host_buffers(g, self.FETCH_STAGE_BYTES // (c.dim * esz))

    def grow_host_buffers(self, g: int, rows: int) -> None:
        """Cache g: buffers of the copy-engine path for lists of up to `rows` rows (never more than the list
        capacity).  The caller makes sure that no copy of this cache is in flight and no list waits in them."""
        cap = self.ctx[0]["lists"][g]["capacity"]
        rb = self.caches[g].dim * (4 if self.spec.dtype == wl.FP32 else 2)
        rows = max(1, min(cap, int(rows), max(self.FETCH_STAGE_MAX_BYTES, self.FETCH_STAGE_BYTES) // rb))
        if rows <= self.fetch_rows[g]:
            return
        pinned = lambda n, dt: torch.empty(n, dtype=dt, pin_memory=True)
        self.fetch_dev[g] = None
        self.fetch_dev[g] = torch.empty(rows * rb, dtype=torch.uint8, device=self.device)
        for x in range(self.N_CTX):
            self.fetch_host[x][g] = pinned(rows * rb, torch.uint8)
            self.fetch_keys[x][g] = pinned(rows, torch.int64)
            self.wb_host[x][g] = pinned(rows * rb, torch.uint8)
            self.wb_keys[x][g] = pinned(rows, torch.int64)
            self.wb_dirty[x][g] = pinned(rows, torch.uint8)
        self.fetch_rows[g] = rows

    def host_lists_fit(self, g: int, n_miss: int, n_evict: int) -> bool:
        """Whether the miss and evict lists of a batch fit the pinned buffers of the copy-engine path."""
        return n_miss <= self.fetch_rows[g] and n_evict <= self.fetch_rows[g]

    def host_buffers_can_hold(self, g: int, rows: int) -> bool:
        """Whether grow_host_buffers may size cache g's buffers for lists of `rows` rows."""
        rb = self.caches[g].dim * (4 if self.spec.dtype == wl.FP32 else 2)
        return rows <= self.ctx[0]["lists"][g]["capacity"] and rows * rb <= self.FETCH_STAGE_MAX_BYTES

    def cache_save_victims_via_host(self, g: int, n_evict: int, stream, ctx: int):
        """Cache g, copy-engine path of the write-back: the dirty victims are saved to the staging buffer and
        the first n_evict entries of the evict list (keys, dirty bytes) and of the staging buffer go to pinned
        host buffers, all on `stream`.  A victim's row is final once its batch's tag step is over, so this
        needs nothing of the batch's fetch.  Returns the event recorded after the saving kernel (the placing
        kernel, which overwrites the victims' slots, has to wait for it)."""
        L = self.ctx[ctx]["lists"][g]
        mb.cache_save_victims(self.caches[g], L["evict_slots"], L["evict_dirty"], L["capacity"], L["counters"],
                              L["staging"], stream)
        saved = torch.cuda.Event()
        saved.record(stream)
        if n_evict > 0:
            rb = self.caches[g].dim * (4 if self.spec.dtype == wl.FP32 else 2)
            with torch.cuda.stream(stream):
                self.wb_keys[ctx][g][:n_evict].copy_(L["evict_keys"][:n_evict], non_blocking=True)
                self.wb_dirty[ctx][g][:n_evict].copy_(L["evict_dirty"][:n_evict], non_blocking=True)
                self.wb_host[ctx][g][:n_evict * rb].copy_(L["staging"][:n_evict * rb], non_blocking=True)
        return saved

    def cache_request_miss_keys(self, g: int, n_miss: int, copy_stream, ctx: int) -> None:
        """Cache g, copy-engine path: the first n_miss keys of the miss list start their way to the host on
        `copy_stream` (the caller made sure the tag step is over).  Called before the victims' copies are
        enqueued: the same copy engine serves both, and the gather waits for the keys only."""
        if n_miss > 0:
            with torch.cuda.stream(copy_stream):
                self.fetch_keys[ctx][g][:n_miss].copy_(self.ctx[ctx]["lists"][g]["miss_keys"][:n_miss], non_blocking=True)

    def cache_fetch_via_host(self, g: int, n_miss: int, copy_stream, stream, ctx: int, saved, mark=None) -> None:
        """Cache g, copy-engine path, after cache_request_miss_keys: host threads gather the rows, one
        contiguous copy and the placing kernel (after the event `saved` of cache_save_victims_via_host) follow
        on `stream`.  Blocks the calling thread for the key copy and the gather, not for the copy of the rows."""
        L = self.ctx[ctx]["lists"][g]
        c = self.caches[g]
        esz = 4 if self.spec.dtype == wl.FP32 else 2
        rb = c.dim * esz
        if n_miss > 0:
            keys_h = self.fetch_keys[ctx][g]
            copy_stream.synchronize()
            rows_h = self.fetch_host[ctx][g]
            t0 = time.perf_counter()
            with self.host_copy_lock:
                t1 = time.perf_counter()
                mb.host_gather_rows(self.host_rows_ptr(g), keys_h.numpy(), n_miss, rb, rows_h, self.gather_threads)
                st = self.host_copy_stats[g]
                st["gather_s"] += time.perf_counter() - t1
                st["gather_bytes"] += n_miss * rb
                st["wait_s"] += t1 - t0
            with torch.cuda.stream(stream):
                if mark is not None:
                    mark(f"copy{g}_begin")
                self.fetch_dev[g][:n_miss * rb].copy_(rows_h[:n_miss * rb], non_blocking=True)
                if mark is not None:
                    mark(f"copy{g}_end")
        stream.wait_event(saved)
        mb.cache_place_fetched(c, self.fetch_dev[g], L["miss_slots"], None, None, L["capacity"], L["counters"], None, stream)

    def cache_writeback_via_host_finish(self, g: int, n_evict: int, ctx: int) -> None:
        """Host threads put the dirty victims into their rows of the host tier (after the copies of
        cache_writeback_via_host_begin have completed)."""
        if n_evict > 0:
            rb = self.caches[g].dim * (4 if self.spec.dtype == wl.FP32 else 2)
            t0 = time.perf_counter()
            with self.host_copy_lock:
                t1 = time.perf_counter()
                mb.host_scatter_rows(self.host_rows_ptr(g), self.wb_keys[ctx][g].numpy(), self.wb_dirty[ctx][g].numpy(),
                                     n_evict, rb, self.wb_host[ctx][g], self.gather_threads)
                st = self.host_copy_stats[g]
                st["scatter_s"] += time.perf_counter() - t1
                st["scatter_bytes"] += n_evict * rb
                st["wait_s"] += t1 - t0

    def cache_writeback(self, g: int, stream=None, ctx: Optional[int] = None) -> None:
        """Cache g: the staged dirty victims back to the host tier (after cache_fetch of the same batch)."""
        L = self._ctx(ctx)["lists"][g]
        if self.l2:
            return                               # part of the two-level data movement
        mb.cache_writeback_evicted(self.caches[g], self.host_rows_ptr(g), L["evict_keys"], L["evict_dirty"],
                                   L["capacity"], L["counters"], L["staging"], stream)

    def cache_refetch(self, prev_ctx: int, placed_step: int = -1, stream=None) -> None:
        """After the backward of the batch in context `prev_ctx`: refresh rows that overflowed there
        and were placed by the batch whose lookup had step `placed_step`."""
        for g, c in enumerate(self.caches):
            L = self.ctx[prev_ctx]["lists"][g]
            mb.cache_refetch_overflowed(c, self.host_rows_ptr(g), L["overflow_keys"], L["overflow_capacity"],
                                        L["counters"], placed_step, stream)

    def cache_step(self, indices, offsets, offsets_host: np.ndarray, step: int, stream=None,
                   do_prefetch: bool = True, ctx: Optional[int] = None) -> None:
        """lookup_insert + prefetch + writeback of every cache for one batch."""
        self.cache_lookup(indices, offsets, offsets_host, step, stream, ctx)
        if do_prefetch:
            self.cache_move(stream, ctx)

    def flush(self, stream=None) -> None:
        for g, c in enumerate(self.caches):
            mb.cache_flush(c, self.host_rows_ptr(g), stream)
            if self.l2:
                mb.cache_flush(self.l2[g], self.host_rows_ptr(g), stream)

    def weights_numpy(self) -> np.ndarray:
        """All tables back to back, each from the memory that holds it (host-tier tables: call flush first)."""
        torch.cuda.synchronize(self.device)
        if not self.cached:
            return self.dev_weights.cpu().numpy().copy()
        out = self.host_weights.numpy().copy()
        if not self.all_cached:
            dev = self.dev_weights.cpu().numpy()
            for t in range(self.spec.T):
                if not self.host_tables[t]:
                    a, b = int(self.spec.weight_offset[t]), int(self.spec.weight_offset[t + 1])
                    out[a:b] = dev[a:b]
        return out

    def close(self) -> None:
        self.tables.destroy()
        for c in self.caches + self.l2:
            c.destroy()
