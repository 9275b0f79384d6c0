"""Thin ctypes binding of libmtrains_b200.so: same names as include/mtrains_b200.h, argument
marshalling only.  Every step of the path runs in the library's CUDA kernels; there is no
fallback: a missing library or a failing call raises.

Pointer arguments accept a torch tensor (its data_ptr is passed), an int address, or None.
`stream` accepts a torch.cuda.Stream, an int handle or None (legacy default stream).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("MTRAINS_B200_LIB", os.path.join(HERE, "libmtrains_b200.so"))

OK = 0
ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CAPACITY, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED = (
    -1, -2, -3, -4, -5, -6, -7)
DTYPE_FP32, DTYPE_FP16 = 0, 1
POOL_SUM, POOL_MEAN, POOL_MAX = 0, 1, 2
POLICY_LRU, POLICY_LFU = 0, 1
MAX_CACHES, CACHE_WAYS, NUM_COUNTERS, NUM_COUNTERS2 = 8, 32, 10, 20
COUNTER_NAMES2 = ("lookups", "unique", "hit_lookups", "miss_lookups", "unique_hits", "unique_misses", "inserted",
                  "evicted", "evicted_dirty", "overflow", "l2_hit_lookups", "l2_unique_hits", "promoted", "demoted",
                  "l2_evicted", "l2_evicted_dirty", "l2_bypass", "l2_bypass_dirty", "l2_dropped", "l2_dropped_dirty")
COUNTER_NAMES = ("lookups", "unique", "hit_lookups", "miss_lookups", "unique_hits",
                 "unique_misses", "inserted", "evicted", "evicted_dirty", "overflow")

EXPORTS = (
    "mts_last_error_string", "mts_launch_count", "mts_trace_enable", "mts_trace_kernel_count",
    "mts_trace_kernel_name", "mts_trace_report", "mts_tables_create", "mts_tables_destroy", "mts_tables_status",
    "mts_tbe_forward", "mts_tbe_backward_workspace_bytes", "mts_tbe_backward_rowwise_adagrad",
    "mts_tbe_backward_rowwise_adagrad_static", "mts_tbe_backward_sort", "mts_tbe_backward_apply",
    "mts_tbe_forward_f16", "mts_tbe_forward_bf16", "mts_tbe_backward_apply_f16",
    "mts_cache_create", "mts_cache_destroy", "mts_cache_status", "mts_cache_data", "mts_cache_dirty",
    "mts_linearize_keys", "mts_cache_workspace_bytes", "mts_cache_lookup_insert", "mts_cache_lookup_insert_tables",
    "mts_tbe_backward_apply_presorted", "mts_cache_create_host_level", "mts_cache2_workspace_bytes",
    "mts_cache2_lookup_insert", "mts_cache2_move", "mts_cache_import_state", "mts_cache_set_fetch_wait_limit",
    "mts_place_tables",
    "mts_cache_prefetch_misses", "mts_host_gather_rows", "mts_host_scatter_rows", "mts_cache_place_fetched", "mts_cache_save_victims", "mts_mover_create", "mts_mover_submit", "mts_mover_stream_wait_moved", "mts_mover_drain", "mts_mover_stats", "mts_mover_destroy", "mts_cache_writeback_evicted", "mts_cache_refetch_overflowed", "mts_cache_flush",
    "mts_cache_export_state",
)


class MtsError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"mtrains_b200 error {code}: {msg}")
        self.code = code


class TableDesc(C.Structure):
    _fields_ = [("T", C.c_int32), ("dtype", C.c_int32),
                ("host_rows", C.POINTER(C.c_int64)), ("host_dim", C.POINTER(C.c_int32)),
                ("host_weight_offset", C.POINTER(C.c_int64)), ("host_cache_id", C.POINTER(C.c_int32)),
                ("dev_weights", C.c_void_p), ("host_weights_mapped", C.c_void_p),
                ("momentum", C.c_void_p)]


_lib = None


def lib():
    """The loaded library.  Raises if it has not been built (python __graft_entry__.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python __graft_entry__.py` "
                "(nvcc, sm_100a); there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
        L.mts_last_error_string.restype = C.c_char_p
        L.mts_last_error_string.argtypes = []
        L.mts_launch_count.restype = i64
        L.mts_launch_count.argtypes = []
        L.mts_trace_enable.argtypes = [i32]
        L.mts_trace_kernel_count.restype = i32
        L.mts_trace_kernel_count.argtypes = []
        L.mts_trace_kernel_name.restype = C.c_char_p
        L.mts_trace_kernel_name.argtypes = [i32]
        L.mts_trace_report.argtypes = [C.POINTER(C.c_double), C.POINTER(i64), i32]
        L.mts_tables_create.argtypes = [C.POINTER(TableDesc), C.POINTER(vp)]
        L.mts_tables_destroy.argtypes = [vp]
        L.mts_tables_status.argtypes = [vp, C.POINTER(i32), vp]
        L.mts_tbe_forward.argtypes = [vp, i32, vp, vp, i64, i32, vp, C.POINTER(vp), i32, vp, i64, vp]
        L.mts_tbe_backward_workspace_bytes.restype = sz
        L.mts_tbe_backward_workspace_bytes.argtypes = [vp, i32, i64]
        L.mts_tbe_backward_rowwise_adagrad.argtypes = [vp, i32, vp, vp, i64, i32, vp, i64, f32, f32, vp,
                                                       C.POINTER(vp), C.POINTER(vp), i32, vp, sz, vp, vp, vp]
        L.mts_tbe_backward_rowwise_adagrad_static.argtypes = [vp, i32, vp, vp, i64, i32, vp, i64, f32, f32, vp,
                                                              C.POINTER(vp), C.POINTER(vp), i32, vp, vp, vp]
        L.mts_tbe_backward_sort.argtypes = [vp, i32, vp, vp, i64, vp, sz, vp, vp, vp]
        L.mts_tbe_backward_apply.argtypes = [vp, i32, vp, i64, i32, vp, i64, f32, f32, vp, C.POINTER(vp),
                                             C.POINTER(vp), i32, vp, sz, vp]
        L.mts_tbe_forward_f16.argtypes = L.mts_tbe_forward.argtypes
        L.mts_tbe_forward_bf16.argtypes = L.mts_tbe_forward.argtypes
        L.mts_tbe_backward_apply_f16.argtypes = L.mts_tbe_backward_apply.argtypes
        L.mts_cache_create.argtypes = [C.POINTER(vp), i64, i64, i32, i32, i32, i32, i32]
        L.mts_cache_destroy.argtypes = [vp]
        L.mts_cache_status.argtypes = [vp, C.POINTER(i32), vp]
        L.mts_cache_data.restype = vp
        L.mts_cache_data.argtypes = [vp]
        L.mts_cache_dirty.restype = vp
        L.mts_cache_dirty.argtypes = [vp]
        L.mts_linearize_keys.argtypes = [vp, i32, i32, i32, vp, vp, i64, i64, vp, vp]
        L.mts_cache_workspace_bytes.restype = sz
        L.mts_cache_workspace_bytes.argtypes = [vp, i64]
        L.mts_cache_lookup_insert.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, sz, vp]
        L.mts_cache_lookup_insert_tables.argtypes = [vp, vp, i32, i32, i32, vp, vp, i64, i64, i64, vp, vp, vp, vp, vp, vp,
                                                     i64, vp, i64, vp, vp, vp, vp, vp, sz, vp]
        L.mts_tbe_backward_apply_presorted.argtypes = [vp, i32, vp, i64, i32, vp, i32, i64, f32, f32, vp, vp, vp,
                                                       C.POINTER(vp), C.POINTER(vp), i32, vp, sz, vp]
        L.mts_cache_create_host_level.argtypes = [C.POINTER(vp), i64, i64, i32, i32, i32, i32, i32, vp]
        L.mts_cache2_workspace_bytes.restype = sz
        L.mts_cache2_workspace_bytes.argtypes = [vp, vp, i64, i64]
        L.mts_cache2_lookup_insert.argtypes = [vp, vp, vp, i64, i64] + [vp] * 14 + [i64, vp, vp, sz, vp]
        L.mts_cache2_move.argtypes = [vp, vp, vp] + [vp] * 13 + [i64, vp, vp, vp]
        L.mts_cache_refetch_overflowed.argtypes = [vp, vp, vp, i64, vp, i64, vp]
        L.mts_cache_prefetch_misses.argtypes = [vp, vp, vp, vp, vp, vp, i64, vp, vp, vp]
        L.mts_cache_writeback_evicted.argtypes = [vp, vp, vp, vp, i64, vp, vp, vp]
        L.mts_host_gather_rows.argtypes = [vp, vp, i64, i64, vp, i32]
        L.mts_host_scatter_rows.argtypes = [vp, vp, vp, i64, i64, vp, i32]
        L.mts_cache_place_fetched.argtypes = [vp, vp, vp, vp, vp, i64, vp, vp, vp]
        L.mts_cache_save_victims.argtypes = [vp, vp, vp, i64, vp, vp, vp]
        L.mts_mover_create.argtypes = [C.POINTER(vp), vp, vp, i64, i32, i32, i64, i64]
        L.mts_mover_submit.argtypes = [vp, C.POINTER(MoveJob)]
        L.mts_mover_stream_wait_moved.argtypes = [vp, i64, vp]
        L.mts_mover_drain.argtypes = [vp]
        L.mts_mover_stats.argtypes = [vp, C.POINTER(C.c_double)]
        L.mts_mover_destroy.argtypes = [vp]
        L.mts_cache_flush.argtypes = [vp, vp, vp]
        L.mts_cache_export_state.argtypes = [vp, vp, vp, vp, vp, vp]
        L.mts_cache_import_state.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.mts_cache_set_fetch_wait_limit.argtypes = [vp, i64]
        L.mts_place_tables.argtypes = [i32, C.POINTER(i64), C.POINTER(C.c_double), i64, C.c_double, C.c_double,
                                       C.POINTER(i32), C.POINTER(C.c_double), C.POINTER(i32)]
        for name in EXPORTS:
            getattr(L, name)            # raises AttributeError when a declared symbol is missing
        _lib = L
    return _lib


def last_error_string() -> str:
    return lib().mts_last_error_string().decode()


def launch_count() -> int:
    return int(lib().mts_launch_count())


def trace_enable(enable: bool) -> None:
    _check(lib().mts_trace_enable(1 if enable else 0))


def trace_report() -> dict:
    """{kernel name: (total device ms, launches)} since the last enable/report; synchronises."""
    n = int(lib().mts_trace_kernel_count())
    ms = (C.c_double * n)()
    cnt = (C.c_int64 * n)()
    _check(lib().mts_trace_report(ms, cnt, n))
    return {lib().mts_trace_kernel_name(k).decode(): (float(ms[k]), int(cnt[k])) for k in range(n) if cnt[k]}


def _check(rc: int) -> None:
    if rc != OK:
        raise MtsError(rc, last_error_string())


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(s):
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _ptr_array(items: Optional[Sequence], n: int):
    if items is None:
        return None
    arr = (C.c_void_p * max(n, 1))()
    for i, it in enumerate(items):
        arr[i] = _ptr(it)
    return arr


class Tables:
    """Handle returned by mts_tables_create; keeps the host arrays of the description alive."""

    def __init__(self, dtype: int, rows, dim, weight_offset, cache_id, dev_weights, host_weights_mapped,
                 momentum):
        T = len(rows)
        self._rows = (C.c_int64 * T)(*[int(r) for r in rows])
        self._dim = (C.c_int32 * T)(*[int(d) for d in dim])
        self._woff = (C.c_int64 * T)(*[int(w) for w in weight_offset])
        self._cid = (C.c_int32 * T)(*[int(c) for c in cache_id]) if cache_id is not None else None
        self._keep = (dev_weights, host_weights_mapped, momentum)
        d = TableDesc(T, dtype, self._rows, self._dim, self._woff,
                      self._cid if self._cid is not None else C.POINTER(C.c_int32)(),
                      _ptr(dev_weights), _ptr(host_weights_mapped), _ptr(momentum))
        h = C.c_void_p()
        _check(lib().mts_tables_create(C.byref(d), C.byref(h)))
        self.handle = h
        self.T = T
        self.total_dim = int(sum(int(x) for x in dim))

    def status(self, stream=None) -> int:
        st = C.c_int32(0)
        _check(lib().mts_tables_status(self.handle, C.byref(st), _stream(stream)))
        return int(st.value)

    def destroy(self):
        if self.handle:
            _check(lib().mts_tables_destroy(self.handle))
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def tables_create(dtype, rows, dim, weight_offset, cache_id, dev_weights, host_weights_mapped, momentum) -> Tables:
    return Tables(dtype, rows, dim, weight_offset, cache_id, dev_weights, host_weights_mapped, momentum)


def tbe_forward(tables: Tables, B: int, indices, offsets, N: int, pooling_mode: int, slot_of_lookup,
                cache_data: Optional[Sequence], out, out_stride: int, stream=None, f16: bool = False,
                bf16: bool = False) -> None:
    """f16 / bf16: `out` holds IEEE binary16 / bfloat16 (mts_tbe_forward_f16 / _bf16), else fp32."""
    n_caches = len(cache_data) if cache_data is not None else 0
    fn = lib().mts_tbe_forward_bf16 if bf16 else lib().mts_tbe_forward_f16 if f16 else lib().mts_tbe_forward
    _check(fn(tables.handle, B, _ptr(indices), _ptr(offsets), N, pooling_mode,
                                 _ptr(slot_of_lookup), _ptr_array(cache_data, n_caches), n_caches, _ptr(out),
                                 out_stride, _stream(stream)))


def tbe_backward_workspace_bytes(tables: Tables, B: int, N: int) -> int:
    return int(lib().mts_tbe_backward_workspace_bytes(tables.handle, B, N))


def tbe_backward_rowwise_adagrad(tables: Tables, B: int, indices, offsets, N: int, pooling_mode: int, grad_out,
                                 grad_stride: int, lr: float, eps: float, slot_of_lookup,
                                 cache_data: Optional[Sequence], cache_dirty: Optional[Sequence], workspace,
                                 workspace_bytes: int, uniq_rows_out=None, n_unique_out=None, stream=None) -> None:
    n_caches = len(cache_data) if cache_data is not None else 0
    _check(lib().mts_tbe_backward_rowwise_adagrad(
        tables.handle, B, _ptr(indices), _ptr(offsets), N, pooling_mode, _ptr(grad_out), grad_stride, lr, eps,
        _ptr(slot_of_lookup), _ptr_array(cache_data, n_caches), _ptr_array(cache_dirty, n_caches), n_caches,
        _ptr(workspace), workspace_bytes, _ptr(uniq_rows_out), _ptr(n_unique_out), _stream(stream)))


def tbe_backward_sort(tables: Tables, B: int, indices, offsets, N: int, workspace, workspace_bytes: int,
                      uniq_rows_out=None, n_unique_out=None, stream=None) -> None:
    """First half of the backward (indices only): lookups ordered by row, left in the workspace."""
    _check(lib().mts_tbe_backward_sort(tables.handle, B, _ptr(indices), _ptr(offsets), N, _ptr(workspace),
                                       workspace_bytes, _ptr(uniq_rows_out), _ptr(n_unique_out), _stream(stream)))


def tbe_backward_apply(tables: Tables, B: int, offsets, N: int, pooling_mode: int, grad_out, grad_stride: int,
                       lr: float, eps: float, slot_of_lookup, cache_data: Optional[Sequence],
                       cache_dirty: Optional[Sequence], workspace, workspace_bytes: int, stream=None,
                       f16: bool = False) -> None:
    """Second half: per-row gradient sums and the optimizer, on the workspace tbe_backward_sort left.
    f16: `grad_out` holds IEEE binary16 (mts_tbe_backward_apply_f16), else fp32."""
    n_caches = len(cache_data) if cache_data is not None else 0
    fn = lib().mts_tbe_backward_apply_f16 if f16 else lib().mts_tbe_backward_apply
    _check(fn(
        tables.handle, B, _ptr(offsets), N, pooling_mode, _ptr(grad_out), grad_stride, lr, eps,
        _ptr(slot_of_lookup), _ptr_array(cache_data, n_caches), _ptr_array(cache_dirty, n_caches), n_caches,
        _ptr(workspace), workspace_bytes, _stream(stream)))


def tbe_backward_apply_presorted(tables: Tables, B: int, offsets, N: int, pooling_mode: int, grad_out,
                                 grad_stride: int, lr: float, eps: float, sorted_rows, sorted_bag, sorted_slot,
                                 cache_data: Optional[Sequence], cache_dirty: Optional[Sequence],
                                 workspace, workspace_bytes: int, stream=None, f16: bool = False) -> None:
    """Gradient half of the backward on lookups already ordered by row (mts_cache_lookup_insert_tables)."""
    n_caches = len(cache_data) if cache_data is not None else 0
    _check(lib().mts_tbe_backward_apply_presorted(
        tables.handle, B, _ptr(offsets), N, pooling_mode, _ptr(grad_out), DTYPE_FP16 if f16 else DTYPE_FP32,
        grad_stride, lr, eps, _ptr(sorted_rows), _ptr(sorted_bag), _ptr(sorted_slot),
        _ptr_array(cache_data, n_caches), _ptr_array(cache_dirty, n_caches), n_caches, _ptr(workspace),
        workspace_bytes, _stream(stream)))


STATIC_SCRATCH_BYTES = 8 << 20


def tbe_backward_rowwise_adagrad_static(tables: Tables, B: int, indices, offsets, N: int, pooling_mode: int,
                                        grad_out, grad_stride: int, lr: float, eps: float, slot_of_lookup=None,
                                        cache_data: Optional[Sequence] = None,
                                        cache_dirty: Optional[Sequence] = None, uniq_rows_out=None,
                                        n_unique_out=None, stream=None) -> None:
    """Backward for callers that cannot allocate device memory: the scratch is an 8 MiB array
    inside the library, shared by all calls (keep them on one stream).  Batches whose scratch need
    exceeds it raise MtsError(ERR_CAPACITY).  First call per device: outside stream capture."""
    n_caches = len(cache_data) if cache_data is not None else 0
    _check(lib().mts_tbe_backward_rowwise_adagrad_static(
        tables.handle, B, _ptr(indices), _ptr(offsets), N, pooling_mode, _ptr(grad_out), grad_stride, lr, eps,
        _ptr(slot_of_lookup), _ptr_array(cache_data, n_caches), _ptr_array(cache_dirty, n_caches), n_caches,
        _ptr(uniq_rows_out), _ptr(n_unique_out), _stream(stream)))


class Cache:
    """Handle returned by mts_cache_create."""

    def __init__(self, num_sets: int, key_space: int, dim: int, dtype: int, policy: int = POLICY_LRU,
                 lock_depth: int = 0, ways: int = CACHE_WAYS, host_rows=None):
        """host_rows: pinned host tensor (or address) that holds the rows of this level (a second level);
        None = the rows live in HBM, allocated by the library."""
        h = C.c_void_p()
        if host_rows is None:
            _check(lib().mts_cache_create(C.byref(h), num_sets, key_space, ways, dim, dtype, policy, lock_depth))
        else:
            _check(lib().mts_cache_create_host_level(C.byref(h), num_sets, key_space, ways, dim, dtype, policy,
                                                     lock_depth, _ptr(host_rows)))
        self._host_rows = host_rows            # keep the storage alive
        self.handle = h
        self.num_sets, self.ways, self.dim, self.dtype = num_sets, ways, dim, dtype
        self.data_ptr = int(lib().mts_cache_data(h))
        self.dirty_ptr = int(lib().mts_cache_dirty(h))

    def status(self, stream=None) -> int:
        st = C.c_int32(0)
        _check(lib().mts_cache_status(self.handle, C.byref(st), _stream(stream)))
        return int(st.value)

    def destroy(self):
        if self.handle:
            _check(lib().mts_cache_destroy(self.handle))
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def cache_create(num_sets, key_space, dim, dtype, policy=POLICY_LRU, lock_depth=0) -> Cache:
    return Cache(num_sets, key_space, dim, dtype, policy, lock_depth)


def linearize_keys(tables: Tables, t_begin: int, t_end: int, B: int, indices, offsets, lookup_begin: int, n: int,
                   keys_out, stream=None) -> None:
    _check(lib().mts_linearize_keys(tables.handle, t_begin, t_end, B, _ptr(indices), _ptr(offsets), lookup_begin,
                                    n, _ptr(keys_out), _stream(stream)))


def cache_workspace_bytes(cache: Cache, N: int) -> int:
    return int(lib().mts_cache_workspace_bytes(cache.handle, N))


def cache_lookup_insert(cache: Cache, keys, N: int, step: int, slot_of_lookup, miss_keys, miss_slots, evict_keys,
                        evict_slots, evict_dirty, list_capacity: int, counters, workspace, workspace_bytes: int,
                        stream=None, overflow_keys=None) -> None:
    _check(lib().mts_cache_lookup_insert(cache.handle, _ptr(keys), N, step, _ptr(slot_of_lookup), _ptr(miss_keys),
                                         _ptr(miss_slots), _ptr(evict_keys), _ptr(evict_slots), _ptr(evict_dirty),
                                         _ptr(overflow_keys), list_capacity, _ptr(counters), _ptr(workspace),
                                         workspace_bytes, _stream(stream)))


def cache_lookup_insert_tables(cache: Cache, tables: Tables, t_begin: int, t_end: int, B: int, indices, offsets,
                               lookup_begin: int, n: int, step: int, slot_of_lookup, miss_keys, miss_slots,
                               evict_keys, evict_slots, evict_dirty, list_capacity: int, overflow_keys,
                               overflow_capacity: int, counters, workspace, workspace_bytes: int, stream=None,
                               sorted_rows_out=None, sorted_bag_out=None, sorted_slot_out=None) -> None:
    """Tag lookup of one cache fed from the batch's sparse input; slot_of_lookup and the three optional
    outputs are batch-wide arrays."""
    _check(lib().mts_cache_lookup_insert_tables(
        cache.handle, tables.handle, t_begin, t_end, B, _ptr(indices), _ptr(offsets), lookup_begin, n, step,
        _ptr(slot_of_lookup), _ptr(miss_keys), _ptr(miss_slots), _ptr(evict_keys), _ptr(evict_slots),
        _ptr(evict_dirty), list_capacity, _ptr(overflow_keys), overflow_capacity, _ptr(counters),
        _ptr(sorted_rows_out), _ptr(sorted_bag_out), _ptr(sorted_slot_out), _ptr(workspace), workspace_bytes,
        _stream(stream)))


def cache2_workspace_bytes(l1: Cache, l2: Cache, N: int, list_capacity: int) -> int:
    return int(lib().mts_cache2_workspace_bytes(l1.handle, l2.handle, N, list_capacity))


def cache2_lookup_insert(l1: Cache, l2: Cache, keys, N: int, step: int, slot_of_lookup, lists: dict, list_capacity: int,
                         counters2, workspace, workspace_bytes: int, stream=None) -> None:
    """lists: the thirteen list arrays by name (fetch_keys, fetch_slots, fetch_src, ev1_keys, ev1_slots, ev1_dirty,
    ev1_dst, ev2_keys, ev2_slots, ev2_dirty, drop_keys, drop_slots, drop_dirty)."""
    L = lists
    _check(lib().mts_cache2_lookup_insert(
        l1.handle, l2.handle, _ptr(keys), N, step, _ptr(slot_of_lookup), _ptr(L["fetch_keys"]), _ptr(L["fetch_slots"]),
        _ptr(L["fetch_src"]), _ptr(L["ev1_keys"]), _ptr(L["ev1_slots"]), _ptr(L["ev1_dirty"]), _ptr(L["ev1_dst"]),
        _ptr(L["ev2_keys"]), _ptr(L["ev2_slots"]), _ptr(L["ev2_dirty"]), _ptr(L["drop_keys"]), _ptr(L["drop_slots"]),
        _ptr(L["drop_dirty"]), list_capacity, _ptr(counters2), _ptr(workspace), workspace_bytes, _stream(stream)))


def cache2_move(l1: Cache, l2: Cache, host_store_mapped, lists: dict, list_capacity: int, counters2, fetch_staging,
                stream=None) -> None:
    L = lists
    _check(lib().mts_cache2_move(
        l1.handle, l2.handle, _ptr(host_store_mapped), _ptr(L["fetch_keys"]), _ptr(L["fetch_slots"]), _ptr(L["fetch_src"]),
        _ptr(L["ev1_keys"]), _ptr(L["ev1_slots"]), _ptr(L["ev1_dirty"]), _ptr(L["ev1_dst"]), _ptr(L["ev2_keys"]),
        _ptr(L["ev2_slots"]), _ptr(L["ev2_dirty"]), _ptr(L["drop_keys"]), _ptr(L["drop_slots"]), _ptr(L["drop_dirty"]),
        list_capacity, _ptr(counters2), _ptr(fetch_staging), _stream(stream)))


def cache_refetch_overflowed(cache: Cache, host_rows_mapped, overflow_keys, list_capacity: int, counters,
                             placed_step: int = -1, stream=None) -> None:
    _check(lib().mts_cache_refetch_overflowed(cache.handle, _ptr(host_rows_mapped), _ptr(overflow_keys),
                                              list_capacity, _ptr(counters), placed_step, _stream(stream)))


def cache_prefetch_misses(cache: Cache, host_rows_mapped, miss_keys, miss_slots, evict_slots, evict_dirty,
                          list_capacity: int, counters, evict_staging, stream=None) -> None:
    _check(lib().mts_cache_prefetch_misses(cache.handle, _ptr(host_rows_mapped), _ptr(miss_keys), _ptr(miss_slots),
                                           _ptr(evict_slots), _ptr(evict_dirty), list_capacity, _ptr(counters),
                                           _ptr(evict_staging), _stream(stream)))


def host_gather_rows(host_rows_ptr: int, host_keys, n: int, row_bytes: int, host_out, threads: int) -> None:
    """host_keys: host int64 array (numpy); host_rows_ptr / host_out: host addresses (pinned buffers)."""
    assert host_keys.dtype.itemsize == 8 and host_keys.flags.c_contiguous and len(host_keys) >= n
    _check(lib().mts_host_gather_rows(int(host_rows_ptr), int(host_keys.ctypes.data), n, row_bytes,
                                      _ptr(host_out), threads))


def host_scatter_rows(host_rows_ptr: int, host_keys, host_mask, n: int, row_bytes: int, host_in, threads: int) -> None:
    """host_keys int64 / host_mask uint8 (or None): host numpy arrays; host_rows_ptr / host_in: host addresses."""
    assert host_keys.dtype.itemsize == 8 and host_keys.flags.c_contiguous and len(host_keys) >= n
    _check(lib().mts_host_scatter_rows(int(host_rows_ptr), int(host_keys.ctypes.data),
                                       None if host_mask is None else int(host_mask.ctypes.data), n, row_bytes,
                                       _ptr(host_in), threads))


def cache_place_fetched(cache: Cache, fetched, miss_slots, evict_slots, evict_dirty, list_capacity: int, counters,
                        evict_staging, stream=None) -> None:
    _check(lib().mts_cache_place_fetched(cache.handle, _ptr(fetched), _ptr(miss_slots), _ptr(evict_slots),
                                         _ptr(evict_dirty), list_capacity, _ptr(counters), _ptr(evict_staging),
                                         _stream(stream)))


class MoveJob(C.Structure):
    """mts_move_job of the header."""
    _fields_ = [("miss_keys", C.c_void_p), ("miss_slots", C.c_void_p), ("evict_keys", C.c_void_p),
                ("evict_slots", C.c_void_p), ("evict_dirty", C.c_void_p), ("list_capacity", C.c_int64),
                ("counters", C.c_void_p), ("host_counters", C.c_void_p), ("evict_staging", C.c_void_p),
                ("tag_done", C.c_void_p), ("move_stream", C.c_void_p), ("save_stream", C.c_void_p),
                ("copy_stream", C.c_void_p)]


class Mover:
    """mts_mover: the copy-engine data movement of one cache on a host thread of the library."""

    def __init__(self, cache: Cache, host_rows: int, row_bytes: int, threads: int, n_contexts: int,
                 first_buffer_bytes: int, max_buffer_bytes: int):
        h = C.c_void_p()
        _check(lib().mts_mover_create(C.byref(h), cache.handle, host_rows, row_bytes, threads, n_contexts,
                                      first_buffer_bytes, max_buffer_bytes))
        self.handle = h
        self.submitted = 0

    def submit(self, miss_keys, miss_slots, evict_keys, evict_slots, evict_dirty, list_capacity: int, counters,
               host_counters, evict_staging, tag_done: int, move_stream, save_stream, copy_stream) -> int:
        """Hands the batch to the mover's thread; returns its job index."""
        job = MoveJob(_ptr(miss_keys), _ptr(miss_slots), _ptr(evict_keys), _ptr(evict_slots), _ptr(evict_dirty),
                      list_capacity, _ptr(counters), _ptr(host_counters), _ptr(evict_staging), tag_done,
                      _stream(move_stream), _stream(save_stream), _stream(copy_stream))
        _check(lib().mts_mover_submit(self.handle, C.byref(job)))
        self.submitted += 1
        return self.submitted - 1

    def stream_wait_moved(self, job_index: int, stream) -> None:
        _check(lib().mts_mover_stream_wait_moved(self.handle, job_index, _stream(stream)))

    def drain(self) -> None:
        _check(lib().mts_mover_drain(self.handle))

    def stats(self) -> dict:
        v = (C.c_double * 5)()
        _check(lib().mts_mover_stats(self.handle, v))
        return {"gather_s": v[0], "gather_bytes": v[1], "scatter_s": v[2], "scatter_bytes": v[3], "kernel_batches": v[4]}

    def close(self) -> None:
        if self.handle:
            lib().mts_mover_destroy(self.handle)
            self.handle = None


def cache_save_victims(cache: Cache, evict_slots, evict_dirty, list_capacity: int, counters, evict_staging,
                       stream=None) -> None:
    _check(lib().mts_cache_save_victims(cache.handle, _ptr(evict_slots), _ptr(evict_dirty), list_capacity,
                                        _ptr(counters), _ptr(evict_staging), _stream(stream)))


def cache_writeback_evicted(cache: Cache, host_rows_mapped, evict_keys, evict_dirty, list_capacity: int, counters,
                            evict_staging, stream=None) -> None:
    _check(lib().mts_cache_writeback_evicted(cache.handle, _ptr(host_rows_mapped), _ptr(evict_keys),
                                             _ptr(evict_dirty), list_capacity, _ptr(counters), _ptr(evict_staging),
                                             _stream(stream)))


def cache_flush(cache: Cache, host_rows_mapped, stream=None) -> None:
    _check(lib().mts_cache_flush(cache.handle, _ptr(host_rows_mapped), _stream(stream)))


def place_tables(size_bytes, bytes_per_sample, hbm_budget_bytes: int, bw_hbm: float, bw_host: float):
    """mts_place_tables on host sequences: ([placement per table: 0 HBM / 1 host tier], time per sample, optimal)."""
    T = len(size_bytes)
    sz = (C.c_int64 * T)(*[int(x) for x in size_bytes])
    cost = (C.c_double * T)(*[float(x) for x in bytes_per_sample])
    out = (C.c_int32 * T)()
    t, opt = C.c_double(0.0), C.c_int32(0)
    _check(lib().mts_place_tables(T, sz, cost, int(hbm_budget_bytes), float(bw_hbm), float(bw_host), out,
                                  C.byref(t), C.byref(opt)))
    return list(out), float(t.value), bool(opt.value)


def cache_import_state(cache: Cache, tags, timestamps, counts, dirty, host_rows_mapped, stream=None) -> None:
    _check(lib().mts_cache_import_state(cache.handle, _ptr(tags), _ptr(timestamps), _ptr(counts), _ptr(dirty),
                                        _ptr(host_rows_mapped), _stream(stream)))


def cache_set_fetch_wait_limit(cache: Cache, polls: int) -> None:
    _check(lib().mts_cache_set_fetch_wait_limit(cache.handle, polls))


def cache_export_state(cache: Cache, tags, timestamps, counts, dirty, stream=None) -> None:
    _check(lib().mts_cache_export_state(cache.handle, _ptr(tags), _ptr(timestamps), _ptr(counts), _ptr(dirty),
                                        _stream(stream)))
