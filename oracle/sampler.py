"""Stochastic static-tree drafting (oracle; test infrastructure).

Sec. 2.1: at a node with s children the drafter samples s tokens from
p(. | path).  Read as sampling without replacement, done with the Gumbel-top-s
construction: key_j = log p_j - log(-log U_j), U_j uniform in (0,1); the s
largest keys, in descending order, are the children's tokens.  This has the
law of s successive draws from p renormalised after removing earlier draws,
which is what the sibling loop of the verifier assumes.
"""

import numpy as np

from .postprocess import postprocess_row
from .tree import tree_children


def sample_children(p, uniforms, s, return_gaps=False):
    """Tokens of s children drawn from distribution p with uniforms U [V].

    Returns (tokens, probs): tokens by descending key (ties: lower id first);
    -1 where fewer than s tokens have positive probability.  With return_gaps
    also the key gap between rank r and rank r+1 for r < s (diagnostic)."""
    p = np.asarray(p, dtype=np.float64)
    U = np.asarray(uniforms, dtype=np.float64)
    support = np.nonzero(p > 0)[0]
    key = np.log(p[support]) - np.log(-np.log(U[support]))
    order = np.lexsort((support, -key))
    toks = [-1] * s
    probs = [0.0] * s
    for r in range(min(s, len(order))):
        toks[r] = int(support[order[r]])
        probs[r] = float(p[toks[r]])
    if return_gaps:
        ks = key[order[: s + 1]]
        gaps = [float(ks[r] - ks[r + 1]) if r + 1 < len(ks) else np.inf for r in range(s)]
        return toks, probs, gaps
    return toks, probs


def sample_draft_tree(parent, draft_cond, draft_uncond, gumbel_uniforms, tokens_in=None, *,
                      cfg_scale=1.0, temperature=1.0, top_k_draft=0, allowed_begin=0,
                      allowed_end=None, parent_begin=0, parent_end=None):
    """Fill tokens of the children of the parents in [parent_begin, parent_end).

    draft_* are [N][V] (row n = drafter logits at node n), gumbel_uniforms
    [N][V].  Returns (tokens [N] int64, draft_prob [N] double); entries of
    nodes not expanded keep tokens_in (or -1) and probability 0."""
    children = tree_children(parent)
    N = len(parent)
    parent_end = N if parent_end is None else parent_end
    tokens = np.full(N, -1, dtype=np.int64) if tokens_in is None else np.array(tokens_in, dtype=np.int64)
    prob = np.zeros(N)
    for n in range(parent_begin, parent_end):
        if not children[n]:
            continue
        p, _ = postprocess_row(draft_cond[n], None if draft_uncond is None else draft_uncond[n],
                               cfg_scale, temperature, top_k_draft, allowed_begin, allowed_end)
        toks, probs = sample_children(p, gumbel_uniforms[n], len(children[n]))
        for c, t, pr in zip(children[n], toks, probs):
            tokens[c], prob[c] = t, pr
    return tokens, prob
