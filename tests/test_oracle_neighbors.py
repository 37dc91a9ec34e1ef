"""Pins for the oracle's latent-neighbour table (Sec. 2.2, Sec. 4: k nearest
codebook entries): an independent all-pairs sort, closed forms on integer
codebooks, duplicate rows."""
import itertools

import numpy as np

import oracle


def _all_pairs_sorted(cb, k):
    """Second, independent brute force: build every (dist, j) pair with Python
    floats, sort, drop self."""
    L = len(cb)
    out = []
    for i in range(L):
        pairs = []
        for j in range(L):
            if j == i:
                continue
            d = 0.0
            for t in range(len(cb[i])):
                d += (float(cb[i][t]) - float(cb[j][t])) ** 2
            pairs.append((d, j))
        pairs.sort()
        out.append([j for _, j in pairs[:k]])
    return np.array(out)


def test_matches_all_pairs_sort_tiny():
    rng = np.random.default_rng(0)
    for L, d, k in [(5, 1, 4), (17, 3, 6), (64, 8, 10), (33, 5, 32)]:
        cb = rng.standard_normal((L, d)).astype(np.float32)
        idx, dist = oracle.neighbor_table(cb, k)
        assert np.array_equal(idx, _all_pairs_sorted(cb, k))
        assert np.all(np.diff(dist, axis=1) >= 0)
        assert not np.any(idx == np.arange(L)[:, None])


def test_integer_line_closed_form():
    # codes 0..9 on a line: neighbours of i are i-1, i+1, i-2, i+2, ... with the
    # lower index first among equal distances
    cb = np.arange(10, dtype=np.float32)[:, None]
    idx, dist = oracle.neighbor_table(cb, 4)
    assert list(idx[5]) == [4, 6, 3, 7]
    assert list(dist[5]) == [1, 1, 4, 4]
    assert list(idx[0]) == [1, 2, 3, 4]
    assert list(idx[9]) == [8, 7, 6, 5]
    assert list(idx[1]) == [0, 2, 3, 4]


def test_duplicates_tie_by_index():
    rng = np.random.default_rng(4)
    cb = rng.standard_normal((12, 4)).astype(np.float32)
    cb[7] = cb[2]
    cb[9] = cb[2]
    idx, dist = oracle.neighbor_table(cb, 5)
    assert list(idx[2][:2]) == [7, 9] and list(dist[2][:2]) == [0, 0]
    assert list(idx[7][:2]) == [2, 9]
    assert list(idx[9][:2]) == [2, 7]
    # a third row sees the three copies at one distance, lowest index first
    for i in (0, 1, 3):
        pos = [list(idx[i]).index(j) for j in (2, 7, 9) if j in idx[i]]
        assert pos == sorted(pos)
        if len(pos) == 3:
            assert pos[2] - pos[0] == 2
    # permutation of rows permutes the table consistently (metric is symmetric,
    # nothing depends on storage order except the tie rule)
    full_idx, full_dist = oracle.neighbor_table(cb, 11)
    D = ((cb[:, None, :].astype(np.float64) - cb[None, :, :]) ** 2).sum(-1)
    for i in range(12):
        assert np.allclose(full_dist[i], D[i][full_idx[i]])
        assert sorted(full_idx[i]) == [j for j in range(12) if j != i]


def test_rows_subset_and_limits():
    rng = np.random.default_rng(5)
    cb = rng.standard_normal((40, 6))
    idx, _ = oracle.neighbor_table(cb, 7)
    sub, _ = oracle.neighbor_table(cb, 7, rows=[3, 39])
    assert np.array_equal(sub, idx[[3, 39]])
    idx0, _ = oracle.neighbor_table(cb, 0)
    assert idx0.shape == (40, 0)
    try:
        oracle.neighbor_table(cb, 40)
        assert False
    except ValueError:
        pass
