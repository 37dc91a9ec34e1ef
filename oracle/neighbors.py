"""Latent neighbourhood B_k (oracle; test infrastructure).

Sec. 2.2 / Sec. 4: B_k(x) is the set of the k nearest neighbours of the draft
token's codebook vector c_x in latent space (App. A.1: codebook
C = {c_1..c_L}, c_i in R^d).  The metric is read as squared Euclidean distance
on the raw codebook rows; the token itself is not listed (it always belongs to
the relaxed set A), and the list is ordered by (distance, index) ascending.
"""

import numpy as np


def neighbor_row(codebook64, i, k):
    """Indices and squared distances of the k nearest rows j != i to row i."""
    diff = codebook64 - codebook64[i]
    dist = (diff * diff).sum(axis=1)
    order = np.lexsort((np.arange(dist.shape[0]), dist))   # by dist, then index
    order = order[order != i][:k]
    return order.astype(np.int32), dist[order]


def neighbor_table(codebook, k, rows=None):
    """Brute-force table: idx [R][k] int32 and dist [R][k] float64 for the query
    rows `rows` (default: all), codebook widened exactly to double."""
    cb = np.asarray(codebook, dtype=np.float64)
    L = cb.shape[0]
    if not 0 <= k <= L - 1:
        raise ValueError("k must be in [0, L-1]")
    rows = range(L) if rows is None else rows
    idx = np.empty((len(rows), k), dtype=np.int32)
    dist = np.empty((len(rows), k), dtype=np.float64)
    for r, i in enumerate(rows):
        idx[r], dist[r] = neighbor_row(cb, int(i), k)
    return idx, dist
