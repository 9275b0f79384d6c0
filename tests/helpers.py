"""Shared test plumbing: small random problems and tolerance checks (no method arithmetic)."""
import numpy as np

from paper_2305_01515_b200 import workload as wl


def small_spec(T=3, rows=(7, 5, 11), dims=(8, 4, 8), B=4, pooling=3.0, dtype=wl.FP32,
               bag_dist="poisson", alpha=0.0, seed=1):
    tabs = [wl.TableSpec(rows=int(r), dim=int(d), pooling=pooling, alpha=alpha)
            for r, d in zip(rows, dims)][:T]
    rng = np.random.default_rng([seed, 99])
    tabs = wl._finish_tables(tabs, rng)
    return wl.ModelSpec("small", tabs, dtype, B, bag_dist, seed=seed)


def storage_dtype(spec):
    return np.float32 if spec.dtype == wl.FP32 else np.float16


PARITY_LOG = []     # (what, plain max|diff| / max|ref|, largest |diff| / bound, rtol, elements); printed at session end


def assert_close_mag(got, ref, mag, rtol, what=""):
    """|got - ref| <= rtol * (|ref| + mag), element by element.  Also records the plain
    max|diff| / max|ref| and how much of the bound the worst element used."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    bound = rtol * (np.abs(ref) + np.asarray(mag, dtype=np.float64))
    err = np.abs(got - ref)
    if err.size:
        with np.errstate(divide="ignore", invalid="ignore"):
            used = np.where(bound > 0, err / bound, np.where(err > 0, np.inf, 0.0))
        PARITY_LOG.append((what, float(err.max() / max(np.abs(ref).max(), 1e-300)), float(used.max()), rtol,
                           int(err.size)))
    bad = err > bound
    if bad.any():
        k = np.argmax(err - bound)
        raise AssertionError(
            f"{what}: {int(bad.sum())} of {bad.size} elements out of tolerance; worst at flat index "
            f"{k}: got {got.flat[k]!r} ref {ref.flat[k]!r} err {err.flat[k]:.3e} bound {bound.flat[k]:.3e}")


# ---------------------------------------------------------------------------- GPU-side plumbing
FWD_RTOL = {0: 1e-5, 1: 2e-3}      # storage dtype -> tolerance of |got - ref| <= rtol * (|ref| + mag)


def to_dev(a, device="cuda:0"):
    import torch

    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def oracle_args(spec):
    return (spec.dtype, spec.dims, spec.out_offset[:-1], spec.weight_offset[:-1])


def custom_spec(rows, dims, B, dtype, poolings=None, alphas=None, bag_dist="poisson", seed=0, name="custom"):
    poolings = poolings or [4.0] * len(rows)
    alphas = alphas or [0.0] * len(rows)
    tabs = [wl.TableSpec(rows=int(r), dim=int(d), pooling=float(p), alpha=float(a))
            for r, d, p, a in zip(rows, dims, poolings, alphas)]
    tabs = wl._finish_tables(tabs, np.random.default_rng([seed, 17]))
    return wl.ModelSpec(name, tabs, dtype, B, bag_dist, seed=seed)


def as_tensor(ptr, n, dtype):
    """A torch view of device memory owned by the library (test plumbing only)."""
    import torch

    class _Holder:
        pass

    h = _Holder()
    itemsize = torch.empty((), dtype=dtype).element_size()
    h.__cuda_array_interface__ = {"shape": (n,), "typestr": {1: "|u1", 2: "<f2", 4: "<f4"}[itemsize],
                                  "data": (ptr, False), "version": 2}
    t = torch.as_tensor(h, device="cuda:0")
    return t.view(dtype) if t.dtype != dtype else t
