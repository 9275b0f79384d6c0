"""ctypes front end of the CPU oracle (oracle/mtrains_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the timed CPU
baseline of bench.py.  The product package never imports this module, and this module
never imports the product package.  All arguments are numpy arrays; nothing here computes
anything itself, it only marshals pointers for the C functions.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mtrains_oracle.c")
_LIB = os.path.join(_HERE, "libmtrains_oracle.so")

NCOUNTERS = 10
NCOUNTERS2 = 20
COUNTER_NAMES2 = ("lookups", "unique", "hit_lookups", "miss_lookups", "unique_hits", "unique_misses", "inserted",
                  "evicted", "evicted_dirty", "overflow", "l2_hit_lookups", "l2_unique_hits", "promoted", "demoted",
                  "l2_evicted", "l2_evicted_dirty", "l2_bypass", "l2_bypass_dirty", "l2_dropped", "l2_dropped_dirty")
COUNTER_NAMES = ("lookups", "unique", "hit_lookups", "miss_lookups", "unique_hits",
                 "unique_misses", "inserted", "evicted", "evicted_dirty", "overflow")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP for the outer loops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_half_to_double.restype = C.c_double
        _lib.orc_half_to_double.argtypes = [C.c_uint16]
        _lib.orc_double_to_half.restype = C.c_uint16
        _lib.orc_double_to_half.argtypes = [C.c_double]
        _lib.orc_cache_set_of.restype = C.c_int64
        _lib.orc_cache_set_of.argtypes = [C.c_int64, C.c_int64]
        _lib.orc_tbe_backward_rowwise_adagrad.restype = C.c_int64
        _lib.orc_cache_create.restype = C.c_void_p
        _lib.orc_cache_lookup_insert.restype = C.c_int64
        _lib.orc_cache_flush.restype = C.c_int64
        _lib.orc_cache2_lookup_insert.restype = C.c_int64
        _lib.orc_place_tables.restype = C.c_double
        for name in ("orc_cache_tags", "orc_cache_ts", "orc_cache_freq", "orc_cache_dirty",
                     "orc_cache_data"):
            getattr(_lib, name).restype = C.c_void_p
            getattr(_lib, name).argtypes = [C.c_void_p]
        _lib.orc_eq3_bandwidth.restype = C.c_double
        _lib.orc_eq3_bandwidth.argtypes = [C.c_double] * 5
        _lib.orc_eq4_iops.restype = C.c_double
        _lib.orc_eq4_iops.argtypes = [C.c_double] * 4
    return _lib


def set_threads(n: int) -> None:
    lib().orc_set_threads(C.c_int(int(n)))


def max_threads() -> int:
    return int(lib().orc_max_threads())


def _p(a: Optional[np.ndarray]):
    if a is None:
        return C.c_void_p(0)
    assert a.flags["C_CONTIGUOUS"]
    return C.c_void_p(a.ctypes.data)


def _ptr_array(items: Optional[Sequence[Optional[np.ndarray]]]):
    if items is None:
        return C.c_void_p(0), None
    arr = (C.c_void_p * len(items))()
    for i, it in enumerate(items):
        arr[i] = None if it is None else it.ctypes.data
    return arr, arr


def half_to_double(h: int) -> float:
    return float(lib().orc_half_to_double(C.c_uint16(int(h))))


def double_to_half(x: float) -> int:
    return int(lib().orc_double_to_half(C.c_double(float(x))))


def cache_set_of(key: int, S: int) -> int:
    return int(lib().orc_cache_set_of(C.c_int64(int(key)), C.c_int64(int(S))))


def place_tables(size_bytes, bytes_per_sample, fast_capacity_bytes: int, bw_fast: float, bw_slow: float):
    """Brute-force placement of T <= 24 tables over a fast and a slow memory (Eq. 6, one GPU).
    Returns (placement int32 [T]: 0 fast / 1 slow, minimal time per sample)."""
    size_bytes = _i64(size_bytes)
    cost = np.ascontiguousarray(bytes_per_sample, dtype=np.float64)
    T = len(size_bytes)
    assert T <= 24
    out = np.zeros(T, np.int32)
    t = lib().orc_place_tables(C.c_int32(T), _p(size_bytes), _p(cost), C.c_int64(int(fast_capacity_bytes)),
                               C.c_double(bw_fast), C.c_double(bw_slow), _p(out))
    return out, float(t)


def eq3_bandwidth(qps, T, D, p, L) -> float:
    return float(lib().orc_eq3_bandwidth(qps, T, D, p, L))


def eq4_iops(qps, TB, LB, alpha) -> float:
    return float(lib().orc_eq4_iops(qps, TB, LB, alpha))


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def tbe_forward(dtype: int, dim, out_offset, weight_offset, weights: np.ndarray, B: int,
                indices, offsets, pooling_mode: int = 0, slot_of_lookup=None,
                cache_data: Optional[Sequence[Optional[np.ndarray]]] = None,
                want_mag: bool = False):
    """Pooled lookup; returns out fp32 [B, sum(dim)] (and sum|W| in fp64 when asked)."""
    dim = _i32(dim); out_offset = _i32(out_offset); weight_offset = _i64(weight_offset)
    indices = _i64(indices); offsets = _i64(offsets)
    T = len(dim)
    total = int(dim.sum())
    if slot_of_lookup is not None:
        slot_of_lookup = _i32(slot_of_lookup)
    out = np.zeros((B, total), dtype=np.float32)
    mag = np.zeros((B, total), dtype=np.float64) if want_mag else None
    cd, _keep = _ptr_array(cache_data)
    lib().orc_tbe_forward(C.c_int32(T), C.c_int32(dtype), _p(dim), _p(out_offset), _p(weight_offset),
                          _p(weights), C.c_int32(B), _p(indices), _p(offsets), C.c_int32(pooling_mode),
                          _p(slot_of_lookup), cd, _p(out), C.c_int64(total), _p(mag))
    return (out, mag) if want_mag else out


def tbe_backward_rowwise_adagrad(dtype: int, dim, out_offset, weight_offset, row_offset,
                                 weights: np.ndarray, momentum: np.ndarray, B: int, indices, offsets,
                                 grad_out: np.ndarray, lr: float, eps: float, pooling_mode: int = 0,
                                 slot_of_lookup=None, cache_data=None, cache_dirty=None,
                                 step_mag: Optional[np.ndarray] = None) -> np.ndarray:
    """In-place update of `weights` (or cache data) and `momentum`; returns the ascending
    distinct linear row ids the batch touched.  step_mag (fp64, one entry per weight element)
    receives the cancellation-free step size of every touched element."""
    dim = _i32(dim); out_offset = _i32(out_offset); weight_offset = _i64(weight_offset)
    row_offset = _i64(row_offset); indices = _i64(indices); offsets = _i64(offsets)
    assert grad_out.dtype == np.float32 and grad_out.flags["C_CONTIGUOUS"]
    assert momentum.dtype == np.float32
    T = len(dim)
    N = int(offsets[T * B])
    if slot_of_lookup is not None:
        slot_of_lookup = _i32(slot_of_lookup)
    uniq = np.zeros(max(N, 1), dtype=np.int64)
    if step_mag is not None:
        assert step_mag.dtype == np.float64 and step_mag.size == weights.size
    cd, _k1 = _ptr_array(cache_data)
    cdirty, _k2 = _ptr_array(cache_dirty)
    U = lib().orc_tbe_backward_rowwise_adagrad(
        C.c_int32(T), C.c_int32(dtype), _p(dim), _p(out_offset), _p(weight_offset), _p(row_offset),
        _p(weights), _p(momentum), C.c_int32(B), _p(indices), _p(offsets), C.c_int32(pooling_mode),
        _p(grad_out), C.c_int64(grad_out.shape[1]), C.c_float(lr), C.c_float(eps),
        _p(slot_of_lookup), cd, cdirty, _p(uniq), _p(step_mag))
    return uniq[:U].copy()


class Cache:
    """One cache level of the oracle: tags, timestamps, use counts, dirty bytes, row data."""

    def __init__(self, num_sets: int, ways: int, dim: int, dtype: int, policy: int = 0,
                 lock_depth: int = 0, with_data: bool = True):
        self.S, self.ways, self.dim, self.dtype = int(num_sets), int(ways), int(dim), int(dtype)
        self.policy, self.lock_depth = int(policy), int(lock_depth)
        self._h = C.c_void_p(lib().orc_cache_create(
            C.c_int64(self.S), C.c_int32(self.ways), C.c_int32(self.dim), C.c_int32(self.dtype),
            C.c_int32(self.policy), C.c_int32(self.lock_depth), C.c_int32(1 if with_data else 0)))
        n = self.S * self.ways
        self.tags = self._view(lib().orc_cache_tags(self._h), np.int64, (self.S, self.ways))
        self.ts = self._view(lib().orc_cache_ts(self._h), np.int64, (self.S, self.ways))
        self.freq = self._view(lib().orc_cache_freq(self._h), np.int64, (self.S, self.ways))
        self.dirty = self._view(lib().orc_cache_dirty(self._h), np.uint8, (n,))
        self.data = None
        if with_data:
            et = np.float32 if dtype == 0 else np.float16
            self.data = self._view(lib().orc_cache_data(self._h), et, (n, self.dim))

    @staticmethod
    def _view(addr, dtype, shape):
        count = int(np.prod(shape))
        buf = (C.c_char * (count * np.dtype(dtype).itemsize)).from_address(addr)
        return np.frombuffer(buf, dtype=dtype).reshape(shape)

    def close(self):
        if self._h:
            self.tags = self.ts = self.freq = self.dirty = self.data = None
            lib().orc_cache_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def lookup_insert(self, keys, step: int, list_capacity: Optional[int] = None):
        """list_capacity: entries the miss list may hold (default: no limit)."""
        keys = _i64(keys)
        N = len(keys)
        cap = max(N, 1)
        list_capacity = cap if list_capacity is None else int(list_capacity)
        slot = np.full(cap, -1, dtype=np.int32)
        mk = np.zeros(cap, np.int64); msl = np.zeros(cap, np.int32)
        ek = np.zeros(cap, np.int64); esl = np.zeros(cap, np.int32); ed = np.zeros(cap, np.uint8)
        cnt = np.zeros(NCOUNTERS, np.int64)
        lib().orc_cache_lookup_insert(self._h, _p(keys), C.c_int64(N), C.c_int64(step), _p(slot),
                                      _p(mk), _p(msl), _p(ek), _p(esl), _p(ed), C.c_int64(list_capacity), _p(cnt))
        nm, ne = int(cnt[6]), int(cnt[7])
        return dict(slot_of_lookup=slot[:N], miss_keys=mk[:nm], miss_slots=msl[:nm],
                    evict_keys=ek[:ne], evict_slots=esl[:ne], evict_dirty=ed[:ne],
                    counters=dict(zip(COUNTER_NAMES, (int(x) for x in cnt))))

    def prefetch_misses(self, host: np.ndarray, res) -> np.ndarray:
        """Save dirty victims to a staging buffer, then fetch missed rows into their slots."""
        ne = len(res["evict_keys"])
        staging = np.zeros((max(ne, 1), self.dim), dtype=self.data.dtype)
        lib().orc_cache_prefetch_misses(self._h, _p(host), _p(res["miss_keys"]), _p(res["miss_slots"]),
                                        C.c_int64(len(res["miss_keys"])), _p(res["evict_slots"]),
                                        _p(res["evict_dirty"]), C.c_int64(ne), _p(staging))
        return staging

    def writeback_evicted(self, host: np.ndarray, res, staging: np.ndarray) -> None:
        lib().orc_cache_writeback_evicted(self._h, _p(host), _p(res["evict_keys"]), _p(res["evict_dirty"]),
                                          C.c_int64(len(res["evict_keys"])), _p(staging))

    def flush(self, host: np.ndarray) -> int:
        return int(lib().orc_cache_flush(self._h, _p(host)))


class Cache2:
    """Two-level exclusive cache of the oracle: `l1` and `l2` are Cache objects of one row shape."""

    def __init__(self, l1: Cache, l2: Cache):
        assert l1.dim == l2.dim and l1.dtype == l2.dtype
        self.l1, self.l2 = l1, l2

    def lookup_insert(self, keys, step: int):
        keys = _i64(keys)
        N = len(keys)
        cap = max(N, 1)
        slot = np.full(cap, -1, dtype=np.int32)
        fk = np.zeros(cap, np.int64); fs = np.zeros(cap, np.int32); fsrc = np.zeros(cap, np.int32)
        e1k = np.zeros(cap, np.int64); e1s = np.zeros(cap, np.int32); e1d = np.zeros(cap, np.uint8)
        e1dst = np.zeros(cap, np.int32)
        e2k = np.zeros(cap, np.int64); e2s = np.zeros(cap, np.int32); e2d = np.zeros(cap, np.uint8)
        dk = np.zeros(cap, np.int64); ds = np.zeros(cap, np.int32); dd = np.zeros(cap, np.uint8)
        cnt = np.zeros(NCOUNTERS2, np.int64)
        lib().orc_cache2_lookup_insert(self.l1._h, self.l2._h, _p(keys), C.c_int64(N), C.c_int64(step), _p(slot),
                                       _p(fk), _p(fs), _p(fsrc), _p(e1k), _p(e1s), _p(e1d), _p(e1dst),
                                       _p(e2k), _p(e2s), _p(e2d), _p(dk), _p(ds), _p(dd), _p(cnt))
        c = dict(zip(COUNTER_NAMES2, (int(x) for x in cnt)))
        nf, n1, n2, nd = c["inserted"], c["evicted"], c["l2_evicted"], c["l2_dropped"]
        return dict(slot_of_lookup=slot[:N], fetch_keys=fk[:nf], fetch_slots=fs[:nf], fetch_src=fsrc[:nf],
                    ev1_keys=e1k[:n1], ev1_slots=e1s[:n1], ev1_dirty=e1d[:n1], ev1_dst=e1dst[:n1],
                    ev2_keys=e2k[:n2], ev2_slots=e2s[:n2], ev2_dirty=e2d[:n2],
                    drop_keys=dk[:nd], drop_slots=ds[:nd], drop_dirty=dd[:nd], counters=c)

    def move(self, store: np.ndarray, res) -> None:
        """Data movement of one lookup_insert result between the two levels and the backing store."""
        lib().orc_cache2_move(
            self.l1._h, self.l2._h, _p(store), _p(res["fetch_keys"]), _p(res["fetch_slots"]), _p(res["fetch_src"]),
            C.c_int64(len(res["fetch_keys"])), _p(res["ev1_keys"]), _p(res["ev1_slots"]), _p(res["ev1_dirty"]),
            _p(res["ev1_dst"]), C.c_int64(len(res["ev1_keys"])), _p(res["ev2_keys"]), _p(res["ev2_slots"]),
            _p(res["ev2_dirty"]), C.c_int64(len(res["ev2_keys"])), _p(res["drop_keys"]), _p(res["drop_slots"]),
            _p(res["drop_dirty"]), C.c_int64(len(res["drop_keys"])))

    def flush(self, store: np.ndarray) -> int:
        """Every dirty row of either level goes to the store (a row is in one level only)."""
        return self.l1.flush(store) + self.l2.flush(store)
