"""The library keeps fallback code paths behind build-time switches (the generic forward and reduce kernels that
the lean forms replace for rows of up to 256 columns, plain loads instead of bulk copies in the fetch kernel, no
row requests ahead in the reduce step).  They are compiled into a second library here and have to pass the same
parity tests against the oracle as the default build."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
VARIANT = ["MTS_BWD_USE_LEAN=0", "MTS_FWD_LEAN=0", "MTS_FETCH_PLAIN_LOADS", "MTS_BWD_PREFETCH_ROWS=0"]


def test_fallback_code_paths_pass_the_parity_tests(tmp_path):
    from paper_2305_01515_b200 import build

    lib = build.build_library(out=str(tmp_path / "libmtrains_b200_variant.so"), defines=VARIANT)
    env = dict(os.environ, MTRAINS_B200_LIB=lib)
    cmd = [sys.executable, "-m", "pytest", "-m", "gpu", "-x", "-q", "-p", "no:cacheprovider",
           "tests/test_gpu_forward.py", "tests/test_gpu_backward.py", "tests/test_gpu_cache.py"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=2400)
    assert r.returncode == 0, r.stdout[-4000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
