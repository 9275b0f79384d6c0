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


def assert_close_mag(got, ref, mag, rtol, what=""):
    """|got - ref| <= rtol * (|ref| + mag), element by element."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    bound = rtol * (np.abs(ref) + np.asarray(mag, dtype=np.float64))
    err = np.abs(got - ref)
    bad = err > bound
    if bad.any():
        k = np.argmax(err - bound)
        raise AssertionError(
            f"{what}: {int(bad.sum())} of {bad.size} elements out of tolerance; worst at flat index "
            f"{k}: got {got.flat[k]!r} ref {ref.flat[k]!r} err {err.flat[k]:.3e} bound {bound.flat[k]:.3e}")
