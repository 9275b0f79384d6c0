"""Host-side halves of the copy-engine data movement (no GPU call): mts_host_gather_rows and
mts_host_scatter_rows against numpy indexing, for row sizes that take the 16-byte streaming path and one
that does not, with one and with several threads."""
import numpy as np
import pytest

from paper_2305_01515_b200 import binding as mb


@pytest.mark.parametrize("row_bytes", [16, 128, 256, 512, 4096, 24])
@pytest.mark.parametrize("threads", [1, 5])
def test_gather_and_scatter_match_numpy(row_bytes, threads):
    rng = np.random.default_rng(row_bytes + threads)
    table = rng.integers(0, 255, (5000, row_bytes), dtype=np.uint8)
    keys = rng.integers(0, 5000, 3000).astype(np.int64)               # with repeats
    out = np.zeros((3000, row_bytes), np.uint8)
    mb.host_gather_rows(table.ctypes.data, keys, 3000, row_bytes, out.ctypes.data, threads)
    assert (out == table[keys]).all()
    mb.host_gather_rows(table.ctypes.data, keys, 0, row_bytes, out.ctypes.data, threads)      # n = 0 is a no-op
    t2 = table.copy()
    ukeys = rng.permutation(5000)[:3000].astype(np.int64)
    mask = (rng.random(3000) < 0.5).astype(np.uint8)
    mb.host_scatter_rows(t2.ctypes.data, ukeys, mask, 3000, row_bytes, out.ctypes.data, threads)
    exp = table.copy()
    exp[ukeys[mask == 1]] = out[mask == 1]
    assert (t2 == exp).all()
    t3 = table.copy()
    mb.host_scatter_rows(t3.ctypes.data, ukeys, None, 3000, row_bytes, out.ctypes.data, threads)
    exp[ukeys] = out
    assert (t3 == exp).all()
