import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); deselect with -m 'not gpu'")


def pytest_collection_modifyitems(config, items):
    import torch

    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _built_libraries():
    """Build the CUDA library (nvcc cross-compiles without a GPU) and the C oracle once."""
    import shutil

    import oracle
    from paper_2305_01515_b200 import build

    oracle.build()
    if shutil.which("nvcc") or os.path.exists("/usr/local/cuda/bin/nvcc"):
        build.build_library()
    yield


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """Floating-point parity actually observed: the plain max|diff| / max|ref| of every tolerance check,
    and the share of its per-element bound rtol * (|ref| + mag) the worst element used."""
    try:
        from helpers import PARITY_LOG
    except ImportError:
        return
    if not PARITY_LOG:
        return
    worst = {}
    for what, plain, used, rtol, n in PARITY_LOG:
        key = (what.rstrip("0123456789 ").strip() or "(unnamed)", rtol)
        w = worst.setdefault(key, [0.0, 0.0, 0, 0])
        w[0], w[1], w[2], w[3] = max(w[0], plain), max(w[1], used), w[2] + 1, w[3] + n
    terminalreporter.write_line("floating-point parity (worst over the checks of a kind):")
    terminalreporter.write_line("  kind | rtol | checks | elements | max|diff|/max|ref| | worst |diff|/bound")
    for (what, rtol), (plain, used, checks, n) in sorted(worst.items()):
        terminalreporter.write_line(f"  {what} | {rtol:g} | {checks} | {n} | {plain:.3e} | {used:.3f}")
