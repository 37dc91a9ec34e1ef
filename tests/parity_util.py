"""Comparison of CUDA results with the oracle under the near-tie rule.

Integers (accepted child, sampled token, neighbour index) must be equal.  A
difference is tolerated, and counted, only where the oracle's own double
values show that the deciding comparison was closer than TIE:
  accept   |u - thr| < TIE            subset cut   |running sum - bound| < TIE
  resample |u - cdf_j| < TIE          (relative to the total mass)
Probabilities (m, thr) must agree within ATOL.
"""
import numpy as np

import oracle

ATOL = 1e-5
TIE = 1e-6
KEY_TIE = 2e-5      # sampler: gap between adjacent Gumbel keys (float32 keys of magnitude < 100)


def compare_verify(gpu, orc, parent, u_accept, seq_ids=None):
    """gpu: dict of numpy arrays [B][N] (node_next, node_token, node_mass, node_thresh);
    orc: list of oracle.verify_sequence results for the sequences seq_ids.
    Returns counts of tolerated near-ties; raises AssertionError otherwise."""
    children = oracle.tree_children(parent)
    N = len(parent)
    stats = dict(nodes=0, tested=0, tie_accept=0, tie_cut=0, tie_resample=0, dirty_sequences=set())
    seq_ids = range(len(orc)) if seq_ids is None else seq_ids
    for o, b in zip(orc, seq_ids):
        for n in range(N):
            stats["nodes"] += 1
            diverged = False
            for c in children[n]:
                om, oth = o["node_mass"][c], o["node_thresh"][c]
                gm, gth = float(gpu["node_mass"][b, c]), float(gpu["node_thresh"][b, c])
                if om < 0:
                    assert gm == -1.0 and gth == -1.0, ("untested child has values", b, c, gm, gth)
                    continue
                stats["tested"] += 1
                if abs(gm - om) > ATOL or abs(gth - oth) > ATOL:
                    assert o["cut_margin"][c] < TIE, ("mass mismatch", b, c, gm, om, gth, oth, o["cut_margin"][c])
                    stats["tie_cut"] += 1
                    diverged = True
                    break
                o_acc = o["node_next"][n] == c
                g_acc = int(gpu["node_next"][b, n]) == c
                if o_acc != g_acc:
                    assert abs(float(u_accept[b, c]) - oth) < TIE, ("accept mismatch", b, c, float(u_accept[b, c]), oth, gth)
                    stats["tie_accept"] += 1
                    diverged = True
                    break
                if o_acc:
                    break
            if diverged:
                stats["dirty_sequences"].add(b)
                continue
            assert int(gpu["node_next"][b, n]) == o["node_next"][n], ("node_next", b, n)
            if o["node_next"][n] < 0:
                gt, ot = int(gpu["node_token"][b, n]), int(o["node_token"][n])
                if gt != ot:
                    assert o["resample_margin"][n] < TIE, ("token mismatch", b, n, gt, ot, o["resample_margin"][n])
                    stats["tie_resample"] += 1
                    stats["dirty_sequences"].add(b)
            else:
                assert int(gpu["node_token"][b, n]) == -1
    return stats


def check_walk(gpu, tokens, max_depth, orc=None, dirty=(), seq_ids=None):
    """The walk is integer work: out_* must equal the walk over the GPU's own per-node results,
    and the oracle's walk for sequences without tolerated near-ties."""
    B = gpu["accept_len"].shape[0]
    for b in range(B):
        ln, toks, nodes = oracle.walk(gpu["node_next"][b], gpu["node_token"][b], tokens[b])
        assert ln == int(gpu["accept_len"][b]) and ln <= max_depth
        assert list(gpu["out_tokens"][b][: ln + 1]) == toks
        assert list(gpu["out_nodes"][b][: ln + 1]) == nodes
        assert np.all(gpu["out_tokens"][b][ln + 1:] == -1) and np.all(gpu["out_nodes"][b][ln + 1:] == -1)
    if orc is not None:
        seq_ids = range(len(orc)) if seq_ids is None else seq_ids
        for o, b in zip(orc, seq_ids):
            if b in dirty:
                continue
            assert int(gpu["accept_len"][b]) == o["accept_len"]
            assert list(gpu["out_tokens"][b][: o["accept_len"] + 1]) == o["out_tokens"]


def compare_neighbors(gpu_idx, gpu_dist, codebook64, rows, k):
    """Exact equality of neighbour lists with the oracle rows; a difference is tolerated only
    where the two distances involved differ by less than TIE.  Returns the number tolerated."""
    oidx, odist = oracle.neighbor_table(codebook64, k, rows=rows)
    ties = 0
    for r, i in enumerate(rows):
        g = gpu_idx[i]
        if np.array_equal(g, oidx[r]):
            if gpu_dist is not None:
                assert np.allclose(gpu_dist[i], odist[r], rtol=1e-6, atol=1e-30)
            continue
        assert len(set(g.tolist())) == k and i not in g
        for pos in np.nonzero(g != oidx[r])[0]:
            dg = ((codebook64[i] - codebook64[g[pos]]) ** 2).sum()
            assert abs(dg - odist[r][pos]) < TIE, ("neighbour mismatch", i, pos, g[pos], oidx[r][pos], dg, odist[r][pos])
            ties += 1
    return ties
