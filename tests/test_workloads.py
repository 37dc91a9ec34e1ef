"""Host-side checks of the synthetic workload generators."""
import numpy as np
import torch

import workloads as W


def test_tree_level_sizes():
    want = {26: [4, 6, 9, 4, 2], 60: [4, 9, 18, 14, 7, 6, 1], 80: [4, 10, 19, 15, 20, 7, 3, 1]}
    for n, lv in want.items():
        parent = W.static_tree(n)
        assert len(parent) == n and W.tree_levels(parent) == lv
        assert parent[0] == -1 and all(0 <= parent[i] < i for i in range(1, n))
        assert all(parent[i] >= parent[i - 1] for i in range(1, n))
        fan = np.bincount(np.array(parent[1:]), minlength=n)
        assert fan.max() <= 4
        # left-heavy: the first child's subtree is at least as large as the second's
    assert sum(1 for c in np.bincount(np.array(W.static_tree(26)[1:]), minlength=26) if c) == 16


def test_generators_are_seeded_and_shaped():
    cfg = W.CONFIGS["c1_tiny"]
    a = W.make_logits(cfg, step=3)
    b = W.make_logits(cfg, step=3)
    c = W.make_logits(cfg, step=4)
    assert a["target_cond"].shape == (1, 26, 16384) and a["target_cond"].dtype == torch.float32
    assert torch.equal(a["draft_uncond"], b["draft_uncond"])
    assert not torch.equal(a["target_cond"], c["target_cond"])
    cb = W.make_codebook(400, 8, "bf16", seed=1, dup_frac=0.05)
    assert cb.dtype == torch.bfloat16
    uniq = torch.unique(cb.float(), dim=0).shape[0]
    assert 380 <= uniq < 400
    ua, ur = W.make_uniforms(3, 5, 7)
    assert ua.min() >= 0 and ua.max() < 1 and ur.shape == (3, 5)
    gu = W.make_gumbel_uniforms(1, 2, 100, 7)
    assert gu.min() > 0 and gu.max() < 1
    tok = W.random_sibling_tokens(W.static_tree(26), 4, 10, 14, 9)
    par = W.static_tree(26)
    for b_ in range(4):
        for n in range(26):
            ch = [i for i in range(26) if par[i] == n]
            assert len({int(tok[b_, c]) for c in ch}) == len(ch)
