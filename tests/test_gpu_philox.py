"""The device Philox-4x32-10 equals the oracle's, word for word."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def test_raw_stream_equality():
    import paper_2502_06352_b200 as L
    n = 1 << 20
    seed = 0xDEADBEEF12345678
    got = L.philox_raw(seed, 5, 11, 22, 33, n).cpu().numpy()
    ctr = np.empty((n, 4), dtype=np.uint64)
    ctr[:, 0] = (np.arange(n) + 5) & 0xFFFFFFFF
    ctr[:, 1], ctr[:, 2], ctr[:, 3] = 11, 22, 33
    want = oracle.philox4x32_10(ctr, (seed & 0xFFFFFFFF, seed >> 32)).astype(np.int64)
    assert np.array_equal(got, want)
    zero = L.philox_raw(0, 0, 0, 0, 0, 1).cpu().numpy()[0]
    want0 = oracle.philox4x32_10(np.zeros((1, 4), dtype=np.uint64), (0, 0))[0]
    assert [int(v) for v in zero] == [int(v) for v in want0]
