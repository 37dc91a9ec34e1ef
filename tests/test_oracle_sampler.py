"""Pins for the oracle's stochastic draft sampler (Sec. 2.1: s tokens drawn from
p at every node), read as Gumbel-top-s sampling without replacement."""
import itertools

import numpy as np

import oracle


def test_equal_uniforms_give_the_most_probable_tokens():
    p = np.array([0.1, 0.4, 0.05, 0.25, 0.2])
    toks, probs = oracle.sample_children(p, np.full(5, 0.37), 3)
    assert toks == [1, 3, 4] and probs == [0.4, 0.25, 0.2]


def test_ties_lower_id_first_and_small_support():
    p = np.array([0.5, 0.0, 0.5, 0.0])
    toks, probs = oracle.sample_children(p, np.full(4, 0.5), 3)
    assert toks == [0, 2, -1] and probs == [0.5, 0.5, 0.0]


def test_ordered_pairs_follow_successive_sampling_law():
    rng = np.random.default_rng(0)
    V, trials = 5, 40000
    p = np.array([0.35, 0.25, 0.0, 0.3, 0.1])
    counts = {}
    first = np.zeros(V)
    for t in range(trials):
        toks, _ = oracle.sample_children(p, rng.uniform(1e-12, 1, V), 2)
        assert toks[0] != toks[1] and 2 not in toks
        counts[tuple(toks)] = counts.get(tuple(toks), 0) + 1
        first[toks[0]] += 1
    chi2, dof = 0.0, -1
    for a, b in itertools.permutations([0, 1, 3, 4], 2):
        e = trials * p[a] * p[b] / (1 - p[a])
        chi2 += (counts.get((a, b), 0) - e) ** 2 / e
        dof += 1
    assert dof == 11 and chi2 < 39.0          # p ~ 1e-4
    e1 = trials * p[[0, 1, 3, 4]]
    assert ((first[[0, 1, 3, 4]] - e1) ** 2 / e1).sum() < 21.1   # 3 dof


def test_tree_fill_uses_row_of_the_parent_and_respects_range():
    rng = np.random.default_rng(1)
    parent = [-1, 0, 0, 1, 1, 2, 3]
    V = 24
    logits = rng.standard_normal((7, V)).astype(np.float32) * 3
    unc = rng.standard_normal((7, V)).astype(np.float32)
    gum = rng.uniform(0.01, 0.99, (7, V))
    kw = dict(cfg_scale=2.0, temperature=0.8, top_k_draft=6, allowed_begin=4, allowed_end=20)
    tokens, prob = oracle.sample_draft_tree(parent, logits, unc, gum, **kw)
    assert tokens[0] == -1 and np.all(tokens[1:] >= 4) and np.all(tokens[1:] < 20)
    for n, ch in enumerate(oracle.tree_children(parent)):
        if not ch:
            continue
        p, _ = oracle.postprocess_row(logits[n], unc[n], 2.0, 0.8, 6, 4, 20)
        want, wp = oracle.sample_children(p, gum[n], len(ch))
        assert [int(tokens[c]) for c in ch] == want
        assert np.allclose(prob[ch], wp)
        assert all(p[t] > 0 for t in want)
    # level-by-level expansion gives the same result as one call
    t2 = None
    for lo, hi in ((0, 1), (1, 3), (3, 7)):
        t2, _ = oracle.sample_draft_tree(parent, logits, unc, gum, t2, parent_begin=lo, parent_end=hi, **kw)
    assert np.array_equal(t2, tokens)
