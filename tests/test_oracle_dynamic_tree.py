"""Pins of oracle/dynamic_tree.py (Sec. 2.1, dynamic tree drafting: V_i = prod c_j, top-K expansion, trimming by V;
Sec. 3: low confidence gives shallow trees) against products written out with a library softmax, brute force on
tiny inputs, closed forms and invariants."""
import itertools

import numpy as np
import torch

from oracle import dynamic_tree as DT


def _rows(seed, depths, slots, V, scale):
    g = np.random.default_rng(seed)
    data = (g.standard_normal((depths, slots, V)) * scale).astype(np.float32)
    return data, (lambda d, s: (data[d, s], None))


def _check_tree(t, K, m):
    parent, depth, logv = t["parent"], t["depth"], t["logv"]
    n = len(parent)
    assert n <= m and parent[0] == -1 and depth[0] == 0 and logv[0] == 0.0
    assert all(0 <= parent[i] < i for i in range(1, n)) and all(parent[i] >= parent[i - 1] for i in range(1, n))
    assert all(depth[i] == depth[parent[i]] + 1 for i in range(1, n))
    assert all(logv[i] <= logv[parent[i]] for i in range(1, n))
    assert max(np.bincount(parent[1:], minlength=n)) <= K
    # children of one node keep their rank order (pool index ascending) and carry distinct tokens
    for p in range(n):
        ch = [i for i in range(1, n) if parent[i] == p]
        assert list(t["pool_index"][ch]) == sorted(t["pool_index"][ch])
        assert len(set(t["token"][ch])) == len(ch)


def test_values_are_products_of_library_softmax_confidences_along_the_path():
    data, row_of = _rows(3, 3, 4, 50, 2.0)
    t = DT.draft_dynamic_tree(row_of, 3, 3, 4, 12)
    _check_tree(t, 3, 12)
    pp, pt, pd = t["pool_parent"], t["pool_token"], t["pool_depth"]
    # slot of every expanded pool entry: position of the entry among the frontier of its depth
    kids = {}
    for i in range(1, len(pp)):
        if pp[i] >= 0:
            kids.setdefault(int(pp[i]), []).append(i)
    slot_of = {0: 0}
    base = 1
    for dep in range(3):
        level = [i for i in range(1, len(pp)) if pd[i] == dep + 1]
        expanded = sorted({int(pp[i]) for i in level if pp[i] >= 0}, key=lambda e: min(kids[e]))
        for s, e in enumerate(expanded):
            slot_of[e] = s
    for i in t["pool_index"][1:]:
        prod, node = 1.0, int(i)
        while node != 0:
            par = int(pp[node])
            conf = torch.softmax(torch.from_numpy(data[pd[par], slot_of[par]].astype(np.float64)), 0)
            prod *= float(conf[pt[node]])
            node = par
        assert abs(np.exp(t["pool_logv"][i]) - prod) <= 1e-12 * prod


def test_expand_frontier_against_brute_force_on_tiny_rows():
    g = np.random.default_rng(0)
    for trial in range(50):
        F, V, K, E = 3, 7, 2, 4
        z = g.standard_normal((F, V)).astype(np.float32)
        if trial % 5 == 0:
            z[1, 3] = z[1, 5]                                   # a tie inside a row
        P = np.exp(z.astype(np.float64))
        P /= P.sum(axis=1, keepdims=True)
        lv = np.log(g.uniform(0.05, 1.0, F))
        tok, logv, chosen = DT.expand_frontier([(P[f], z[f]) for f in range(F)], lv, K, E)
        # brute force: every (slot, token) pair valued by the product, best K per slot, best E overall
        cands = []
        for f in range(F):
            best = sorted(range(V), key=lambda j: (-float(z[f, j]), j))[:K]
            for r, j in enumerate(best):
                cands.append((np.exp(lv[f]) * P[f, j], f * K + r, j))
        assert [c[2] for c in cands] == list(tok)
        assert np.allclose(np.exp(logv), [c[0] for c in cands], rtol=1e-12)
        want = [c[1] for c in sorted(cands, key=lambda c: (-c[0], c[1]))[:E]]
        assert list(chosen) == want


def test_uniform_rows_give_the_first_tokens_and_the_first_slots():
    row_of = lambda d, s: (np.zeros(16, dtype=np.float32), None)
    t = DT.draft_dynamic_tree(row_of, 2, 3, 2, 6)
    # depth 1: tokens 0,1,2 with V = 1/16; frontier = candidates 0 and 1; depth 2: V = 1/256 each
    assert list(t["parent"]) == [-1, 0, 0, 0, 1, 1] and list(t["token"]) == [-1, 0, 1, 2, 0, 1]
    assert np.allclose(np.exp(t["logv"]), [1, 1 / 16, 1 / 16, 1 / 16, 1 / 256, 1 / 256])


def test_no_trimming_gives_the_full_k_ary_tree():
    _, row_of = _rows(5, 3, 9, 40, 1.0)
    t = DT.draft_dynamic_tree(row_of, 3, 3, 9, 1000)            # E >= F K at depths 0 and 1; depth 2 expands 9 of 9
    assert len(t["parent"]) == 1 + 3 + 9 + 27
    _check_tree(t, 3, 1000)


def test_a_dominant_chain_is_followed_to_the_last_depth_and_diffuse_rows_stay_shallow():
    V, depths = 64, 6
    sharp = np.full((depths, 4, V), -20.0, dtype=np.float32)
    sharp[:, :, 7] = 10.0
    t = DT.draft_dynamic_tree(lambda d, s: (sharp[d, s], None), depths, 4, 4, 10)
    assert t["depth"].max() == depths and t["token"][t["depth"].argmax()] == 7
    # Sec. 3: low confidence -> the product decays fast -> wide and shallow trees
    mean_depth = {}
    for scale in (0.25, 6.0):
        ds = []
        for seed in range(8):
            _, row_of = _rows(100 + seed, depths, 8, 256, scale)
            tt = DT.draft_dynamic_tree(row_of, depths, 8, 8, 40)
            _check_tree(tt, 8, 40)
            ds.append(tt["depth"].mean())
        mean_depth[scale] = float(np.mean(ds))
    assert mean_depth[6.0] > mean_depth[0.25] + 0.5


def test_trim_keeps_the_best_values_and_parents_before_children():
    g = np.random.default_rng(9)
    _, row_of = _rows(11, 4, 6, 30, 1.5)
    for m in (2, 5, 17, 60):
        margins = []
        t = DT.draft_dynamic_tree(row_of, 4, 3, 6, m, margins=margins)
        _check_tree(t, 3, m)
        kept = set(int(i) for i in t["pool_index"])
        lv = t["pool_logv"]
        worst_kept = min(lv[i] for i in kept if i != 0) if len(kept) > 1 else np.inf
        left = [lv[i] for i in range(1, len(lv)) if i not in kept and np.isfinite(lv[i])]
        assert not left or max(left) <= worst_kept
    # ties between equal values go to the lower pool index
    keep = DT.trim(np.array([-1, 0, 0, 0]), np.array([0.0, -1.0, -1.0, -1.0]), 3)
    assert list(keep) == [0, 1, 2]


def test_guidance_temperature_and_allowed_range_reach_the_confidences():
    g = np.random.default_rng(4)
    cond = g.standard_normal((1, 1, 32)).astype(np.float32)
    unc = g.standard_normal((1, 1, 32)).astype(np.float32)
    t = DT.draft_dynamic_tree(lambda d, s: (cond[d, s], unc[d, s]), 1, 4, 4, 5, cfg_scale=3.0, temperature=0.7,
                              allowed_begin=8, allowed_end=24)
    z = ((unc[0, 0] + 3.0 * (cond[0, 0] - unc[0, 0])) / 0.7).astype(np.float64)
    z[:8] = -np.inf
    z[24:] = -np.inf
    conf = torch.softmax(torch.from_numpy(z), 0).numpy()
    best = np.argsort(-conf, kind="stable")[:4]
    assert list(t["token"][1:]) == list(best) and np.allclose(np.exp(t["logv"][1:]), conf[best], rtol=1e-5)
