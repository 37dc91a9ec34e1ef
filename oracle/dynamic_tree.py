"""Dynamic-tree drafting (Sec. 2.1, "Tree Drafting and Verification", the dynamic variant; Sec. 3,
"Shallow draft trees").  TEST INFRASTRUCTURE, like the rest of this package.

Every draft node t_i carries a global accept value V_i = prod of the drafter's confidences c_j along
the path from the root to t_i.  A depth of drafting takes the current frontier, gives every
frontier node its top-K tokens by drafter confidence (the confidence of a token is its
probability in the drafter's post-processed row), and keeps the E candidates with the largest V
as the next frontier.  After the last depth all candidates drafted so far are ranked by V and the
best m - 1 of them, with the root, are the draft tree that goes to verification.

Everything is kept as log V in double precision.  Order of equal values (stated so that both
sides agree): tokens of one row by (z descending, token id ascending); candidates by (log V
descending, pool index ascending), a pool index being the position at which the candidate was
created (depth by depth, frontier slot by frontier slot, rank by rank).  With that order a
parent always ranks before its children (c <= 1), so the trimmed set is a tree.
"""
import numpy as np

from .postprocess import postprocess_row


def top_children(z, P, K):
    """The K tokens of one row with the largest z (ties: lower id) and the log of their confidence."""
    V = z.shape[0]
    order = np.lexsort((np.arange(V), -z.astype(np.float64)))      # primary: z descending, then id
    tok = order[:K]
    with np.errstate(divide="ignore"):
        return tok.astype(np.int64), np.log(P[tok])


def expand_frontier(rows, frontier_logv, K, E, margins=None):
    """One depth.  rows: list over frontier slots of (P, z) or None for an empty slot;
    frontier_logv[f] = log V of the node in slot f.  Returns (cand_token [F*K], cand_logv [F*K],
    chosen [E] candidate indices f*K + r in rank order; -1 where fewer than E exist)."""
    F = len(rows)
    cand_token = np.full(F * K, -1, dtype=np.int64)
    cand_logv = np.full(F * K, -np.inf)
    for f in range(F):
        if rows[f] is None:
            continue
        P, z = rows[f]
        tok, lnc = top_children(z, P, K)
        cand_token[f * K:(f + 1) * K] = tok
        cand_logv[f * K:(f + 1) * K] = frontier_logv[f] + lnc
    order = np.lexsort((np.arange(F * K), -cand_logv))
    live = int(np.isfinite(cand_logv).sum())
    chosen = np.full(E, -1, dtype=np.int64)
    n = min(E, live)
    chosen[:n] = order[:n]
    if margins is not None and n < live:
        margins.append(float(cand_logv[order[n - 1]] - cand_logv[order[n]]))    # gap at the cut
    return cand_token, cand_logv, chosen


def trim(pool_parent, pool_logv, m, margins=None):
    """Indices (ascending) of the pool entries that form the final tree: the root (entry 0) and the
    m - 1 other entries with the largest log V (ties: lower pool index)."""
    Pn = len(pool_parent)
    idx = np.arange(1, Pn)
    live = idx[np.isfinite(pool_logv[1:])]
    order = live[np.lexsort((live, -pool_logv[live]))]
    n = min(m - 1, len(order))
    if margins is not None and n < len(order):
        margins.append(float(pool_logv[order[n - 1]] - pool_logv[order[n]]))
    return np.sort(np.concatenate(([0], order[:n])))


def breadth_first(pool_parent, pool_depth, keep):
    """Renumber the kept pool entries breadth first: by depth, then by the new id of the parent,
    then by pool index (= rank among siblings).  Returns (parent [n] in new ids, pool_index [n])."""
    keep = list(int(i) for i in keep)
    new_id = {0: 0}
    out = [0]
    max_depth = max(int(pool_depth[i]) for i in keep)
    for dep in range(1, max_depth + 1):
        level = [i for i in keep if int(pool_depth[i]) == dep]
        level.sort(key=lambda i: (new_id[int(pool_parent[i])], i))
        for i in level:
            new_id[i] = len(out)
            out.append(i)
    parent = np.array([-1] + [new_id[int(pool_parent[i])] for i in out[1:]], dtype=np.int64)
    return parent, np.array(out, dtype=np.int64)


def draft_dynamic_tree(row_of, depths, K, E, m, cfg_scale=None, temperature=1.0, allowed_begin=0, allowed_end=None,
                       margins=None):
    """Drafting of one sequence.  row_of(depth, slot) -> (cond, uncond) raw drafter rows of the node in
    frontier slot `slot` at depth `depth` (synthetic stand-ins for a drafter's forward pass).
    Returns dict(parent, token, logv, pool_index, depth) of the trimmed tree, breadth first, plus the
    whole pool (pool_parent, pool_token, pool_logv, pool_depth)."""
    pool_parent, pool_token, pool_logv, pool_depth = [-1], [-1], [0.0], [0]
    frontier = [0]                                              # pool indices, slot order
    for dep in range(depths):
        rows, flv = [], []
        for slot, node in enumerate(frontier):
            if node < 0:
                rows.append(None)
                flv.append(-np.inf)
                continue
            cond, uncond = row_of(dep, slot)
            rows.append(postprocess_row(cond, uncond, cfg_scale, temperature, 0, allowed_begin, allowed_end))
            flv.append(pool_logv[node])
        cand_token, cand_logv, chosen = expand_frontier(rows, np.array(flv), K, E, margins)
        base = len(pool_parent)
        for c in range(len(cand_token)):
            pool_parent.append(frontier[c // K] if frontier[c // K] >= 0 else -1)
            pool_token.append(int(cand_token[c]))
            pool_logv.append(float(cand_logv[c]))
            pool_depth.append(dep + 1)
        frontier = [base + int(c) if c >= 0 else -1 for c in chosen]
    pool_parent = np.array(pool_parent)
    pool_logv = np.array(pool_logv)
    pool_depth = np.array(pool_depth)
    keep = trim(pool_parent, pool_logv, m, margins)
    parent, pool_index = breadth_first(pool_parent, pool_depth, keep)
    pool_token = np.array(pool_token)
    return {"parent": parent, "token": pool_token[pool_index], "logv": pool_logv[pool_index], "pool_index": pool_index,
            "depth": pool_depth[pool_index], "pool_parent": pool_parent, "pool_token": pool_token,
            "pool_logv": pool_logv, "pool_depth": pool_depth}
