"""Relaxed acceptance of one draft tree (oracle; test infrastructure).

Follows Sec. 4 (multiplicative bound, relaxed accept probability), App. A.2
Eq. 1-2 (accept test, residual resampling) and Sec. 2.1 (tree verification).
p = drafter, q = target.  All arithmetic in double on the distributions that
postprocess_row returns.

Readings where the paper is silent:
 * the neighbour list excludes the draft token x itself; x always belongs to A
 * A is the longest prefix of the distance-ordered list for which the running
   sum stays strictly below lambda * q(x)  (Sec. 4, display with "<")
 * siblings are tested one after another in stored order; after a rejection
   the mass of A is moved onto x (q~), the target becomes the normalised
   positive part of q~ - p (Eq. 2), and the drafter is renormalised without x
 * the token drawn when no child is accepted (or at a leaf) uses inverse-CDF
   sampling in token-id order
 * additive variant (Sec. 2.2, LANTERN's bound, delta > 0): neighbours join A
   while the mass they add to x, i.e. the total-variation distance between q
   and q~, stays strictly below delta; q(x) itself does not count against delta
"""

import numpy as np

from .postprocess import postprocess_row
from .tree import tree_children


def relaxed_mass(q_cur, x, nbr_idx, k, lam, code_offset, n_codes, margins=None, delta=0.0, force_members=None,
                 skip=False):
    """Sec. 4: m = sum of q over A_{k,lambda}(x) and the members of A besides x.
    With delta > 0 the additive bound of Sec. 2.2 replaces the multiplicative one:
    the neighbours' own running sum stays below delta (A_{k,delta}); lam is unused.

    If `margins` is a list, |running sum - bound| of every comparison made is
    appended to it (diagnostic for near-tie accounting; no effect on the result).
    `force_members` (diagnostic, used only when a comparison with another
    implementation continues past a near-tie): take exactly that many list entries
    instead of applying the bound.
    `skip` selects the other reading of "a subset of B_k that satisfies the bound"
    (Sec. 4 gives only the inequality): a neighbour that would break the bound is
    passed over and the list is searched on, instead of ending the search."""
    cum = q_cur[x]
    bound = q_cur[x] + delta if delta > 0 else lam * q_cur[x]
    members = []
    code = x - code_offset
    if 0 <= code < n_codes:
        for r in range(k):
            a = code_offset + int(nbr_idx[code][r])
            if margins is not None:
                margins.append(abs(cum + q_cur[a] - bound))
            take = cum + q_cur[a] < bound if force_members is None else r < force_members
            if take:
                cum = cum + q_cur[a]
                members.append(a)
            elif not skip or force_members is not None:
                break
    return cum, members


def moved_mass(q_cur, x, m, members):
    """q~: the target distribution with the mass of A concentrated on x."""
    q_t = np.array(q_cur, dtype=np.float64)
    q_t[x] = m
    for a in members:
        q_t[a] = 0.0
    return q_t


def sibling_loop(q, p, child_ids, tokens, u_accept, nbr_idx, k, lam, code_offset, n_codes, delta=0.0, forced=None,
                 skip=False, det_draft=False):
    """Test the children of one node in stored order (Sec. 4; App. A.2 Eq. 1-2).

    `skip`: greedy-skip reading of the subset (see relaxed_mass).
    `det_draft`: the draft tokens were chosen deterministically (Sec. 3, what dynamic-tree
    drafting does): the drafter puts probability 1 on each of them, so the accept probability
    is min(1, m) = m, p is not used, and the residual after a rejection is q~ without x.

    `forced` (diagnostic): {child: {"accept": bool, "n_members": int}} overrides the
    accept decision and / or the size of A of that child, so that a comparison can go
    on after a floating-point near-tie with the other side's decision imposed.

    Returns (accepted child or -1, q_cur, {child: (m, thr, cut_margin, |A| - 1)}): q_cur
    is the target distribution left after the rejections (q itself at a leaf);
    cut_margin is the smallest |running sum - bound| met while forming A."""
    q_cur = np.array(q, dtype=np.float64)
    p_cur = None if (p is None or det_draft) else np.array(p, dtype=np.float64)
    tested = {}
    for c in child_ids:
        x = int(tokens[c])
        if x < 0:
            continue
        margins = []
        f = (forced or {}).get(c, {})
        m, members = relaxed_mass(q_cur, x, nbr_idx, k, lam, code_offset, n_codes, margins, delta,
                                  force_members=f.get("n_members"), skip=skip)
        if det_draft:
            thr = min(1.0, m)                     # Sec. 3: p(x) = 1
        elif p_cur[x] > 0:
            thr = min(1.0, m / p_cur[x])          # Sec. 4, final accept probability
        else:
            thr = 1.0 if m > 0 else 0.0
        tested[c] = (m, thr, min(margins) if margins else np.inf, len(members))
        accept = float(u_accept[c]) < thr
        if "accept" in f:
            accept = bool(f["accept"])
        if accept:
            return c, q_cur, tested
        q_t = moved_mass(q_cur, x, m, members)
        if det_draft:
            r = q_t.copy()                         # Eq. 2 with p = the point mass at x
            r[x] = max(m - 1.0, 0.0)
            Z = r.sum()
            q_cur = r / Z if Z > 0 else q_t
            continue
        r = np.maximum(q_t - p_cur, 0.0)           # Eq. 2
        Z = r.sum()
        q_cur = r / Z if Z > 0 else q_t
        w = 1.0 - p_cur[x]
        p_cur[x] = 0.0
        if w > 0:
            p_cur = p_cur / w
    return -1, q_cur, tested


def inverse_cdf(dist, u, return_margin=False):
    """Smallest token j whose cumulative mass exceeds u * total.  With
    return_margin also min_j |u * total - cdf_j| / total (diagnostic)."""
    cdf = np.cumsum(dist)
    target = float(u) * cdf[-1]
    j = int(np.argmax(cdf > target))
    if return_margin:
        return j, float(np.abs(cdf - target).min() / cdf[-1])
    return j


def verify_node(q, p, child_ids, tokens, u_accept, u_resample, nbr_idx, k, lam,
                code_offset, n_codes, delta=0.0, forced=None, skip=False, det_draft=False):
    """Process one tree node.

    q: target distribution of the node; p: drafter distribution (None at a leaf)
    child_ids: its children in stored order; tokens[c]: draft token of node c
    (a negative token means "no draft" and is skipped).
    Returns (next_child or -1, sampled token or -1, {child: (m, thr, cut_margin, |A| - 1)});
    tested["resample_margin"] is set when a token was drawn.
    """
    nxt, q_cur, tested = sibling_loop(q, p, child_ids, tokens, u_accept, nbr_idx, k, lam,
                                      code_offset, n_codes, delta, forced, skip, det_draft)
    if nxt >= 0:
        return nxt, -1, tested
    j, margin = inverse_cdf(q_cur, u_resample, return_margin=True)
    tested["resample_margin"] = margin
    return -1, j, tested


def walk(node_next, node_token, tokens):
    """Sec. 2.1 / App. A.2: follow accepted children from the root; the accepted
    draft tokens are kept, then one token drawn at the node where the walk
    stops.  Returns (accept_len, out_tokens, out_nodes); the lists have
    accept_len + 1 entries."""
    cur = 0
    out_tokens, out_nodes = [], []
    while node_next[cur] >= 0:
        cur = int(node_next[cur])
        out_tokens.append(int(tokens[cur]))
        out_nodes.append(cur)
    out_tokens.append(int(node_token[cur]))
    out_nodes.append(cur)
    return len(out_tokens) - 1, out_tokens, out_nodes


def verify_sequence(parent, target_cond, target_uncond, draft_cond, draft_uncond, tokens,
                    u_accept, u_resample, nbr_idx, *, cfg_scale=1.0, temperature=1.0,
                    top_k_target=0, top_k_draft=0, lam=1.0, k=0, code_offset=0, n_codes=0,
                    allowed_begin=0, allowed_end=None, delta=0.0, skip=False, det_draft=False):
    """Verify one sequence's tree.  Logit arrays are [N][V]; uncond may be None.

    Returns a dict with node_next, node_token (int arrays [N]), node_mass,
    node_thresh (double [N], -1 where a node was not tested), accept_len,
    out_tokens, out_nodes.
    """
    children = tree_children(parent)
    N = len(parent)
    node_next = np.full(N, -1, dtype=np.int64)
    node_token = np.full(N, -1, dtype=np.int64)
    node_mass = np.full(N, -1.0)
    node_thresh = np.full(N, -1.0)
    cut_margin = np.full(N, np.inf)
    resample_margin = np.full(N, np.inf)
    for n in range(N):
        q, _ = postprocess_row(target_cond[n], None if target_uncond is None else target_uncond[n],
                               cfg_scale, temperature, top_k_target, allowed_begin, allowed_end)
        p = None
        if children[n] and not det_draft:
            p, _ = postprocess_row(draft_cond[n], None if draft_uncond is None else draft_uncond[n],
                                   cfg_scale, temperature, top_k_draft, allowed_begin, allowed_end)
        nxt, tok, tested = verify_node(q, p, children[n], tokens, u_accept, u_resample[n],
                                       nbr_idx, k, lam, code_offset, n_codes, delta, skip=skip, det_draft=det_draft)
        node_next[n], node_token[n] = nxt, tok
        resample_margin[n] = tested.pop("resample_margin", np.inf)
        for c, (m, thr, cm, _) in tested.items():
            node_mass[c], node_thresh[c], cut_margin[c] = m, thr, cm
    accept_len, out_tokens, out_nodes = walk(node_next, node_token, tokens)
    return dict(node_next=node_next, node_token=node_token, node_mass=node_mass,
                node_thresh=node_thresh, accept_len=accept_len, out_tokens=out_tokens,
                out_nodes=out_nodes, cut_margin=cut_margin, resample_margin=resample_margin)


def verify_batch(parent, target_cond, target_uncond, draft_cond, draft_uncond, tokens,
                 u_accept, u_resample, nbr_idx, **params):
    """verify_sequence over the leading batch dimension; returns a list of dicts."""
    out = []
    for b in range(len(tokens)):
        out.append(verify_sequence(
            parent, target_cond[b], None if target_uncond is None else target_uncond[b],
            None if draft_cond is None else draft_cond[b], None if draft_uncond is None else draft_uncond[b],
            tokens[b], u_accept[b], u_resample[b], nbr_idx, **params))
    return out
