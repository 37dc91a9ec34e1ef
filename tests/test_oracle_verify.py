"""Pins for the oracle's relaxed acceptance (Sec. 4), accept test and residual
(App. A.2 Eq. 1-2) and tree walk (Sec. 2.1)."""
import itertools

import numpy as np

import oracle


def _dists(rng, V, conc=0.5):
    q = rng.dirichlet(np.full(V, conc))
    p = rng.dirichlet(np.full(V, conc))
    return q, p


def _table(rng, L, k, d=3):
    idx, _ = oracle.neighbor_table(rng.standard_normal((L, d)), k)
    return idx


def test_reduces_to_speculative_sampling():
    """A = {x} (k = 0, or lambda = 1): accept prob min(1, q/p) (Eq. 1), residual
    norm([q - p]_+) (Eq. 2)."""
    rng = np.random.default_rng(0)
    V = 16
    nbr = _table(rng, V, 5)
    for trial in range(20):
        q, p = _dists(rng, V)
        for k, lam in ((0, 3.0), (5, 1.0)):
            for x in range(V):
                tokens = [0, x]
                u = [0.0, 1.0]      # force rejection to see the residual
                nxt, q_cur, tested = oracle.sibling_loop(q, p, [1], tokens, u, nbr, k, lam, 0, V)
                m, thr = tested[1][:2]
                assert m == q[x]
                assert thr == min(1.0, q[x] / p[x])
                res = np.maximum(q - p, 0)
                assert nxt == -1 and np.allclose(q_cur, res / res.sum(), atol=1e-15)


def test_relaxed_set_second_way():
    """A = longest prefix of the neighbour list whose running sum (including
    q(x)) stays strictly below lambda q(x), computed via cumsum."""
    rng = np.random.default_rng(1)
    V, k = 32, 12
    nbr = _table(rng, V, k)
    for trial in range(200):
        q, _ = _dists(rng, V, conc=0.3)
        lam = float(rng.choice([1.0, 1.5, 2.0, 3.0, 20.0]))
        x = int(rng.integers(V))
        kk = int(rng.integers(0, k + 1))
        m, members = oracle.relaxed_mass(q, x, nbr, kk, lam, 0, V)
        run = q[x] + np.cumsum(q[nbr[x][:kk]])
        ok = run < lam * q[x]
        n_take = kk if ok.all() else int(np.argmin(ok))
        assert members == [int(a) for a in nbr[x][:n_take]]
        assert np.isclose(m, q[x] + q[nbr[x][:n_take]].sum(), rtol=1e-14)
        # bound of Sec. 4 and its consequence for the accept probability
        assert m >= q[x]
        assert m < lam * q[x] or (n_take == 0 and m == q[x])
        assert x not in members and len(set(members)) == len(members)


def test_bound_on_accept_probability_and_monotonicity():
    rng = np.random.default_rng(2)
    V, k = 24, 10
    nbr = _table(rng, V, k)
    for trial in range(100):
        q, p = _dists(rng, V)
        x = int(rng.integers(V))
        prev = None
        for lam in (1.0, 2.0, 3.0, 5.0, 10.0, 20.0):
            row = []
            for kk in (0, 1, 2, 5, 10):
                _, _, tested = oracle.sibling_loop(q, p, [1], [0, x], [0, 1.0], nbr, kk, lam, 0, V)
                m, thr = tested[1][:2]
                assert thr <= lam * min(1.0, q[x] / p[x]) * (1 + 1e-12)
                row.append((m, thr))
            ms = [r[0] for r in row]
            assert all(b >= a for a, b in zip(ms, ms[1:]))       # non-decreasing in k
            if prev is not None:
                assert all(b[0] >= a[0] and b[1] >= a[1] for a, b in zip(prev, row))  # and in lambda
            prev = row


def test_additive_bound_is_a_bound_on_the_total_variation_distance():
    """Sec. 2.2 (LANTERN's rule, delta > 0): A = longest prefix of the neighbour list whose own
    running sum stays strictly below delta, computed via cumsum; the distortion TVD(q, q~) is the
    moved mass and therefore < delta; delta -> 0 gives Eq. 1, delta > 1 takes all k neighbours;
    with delta = (lambda - 1) q(x) both rules draw the same set."""
    rng = np.random.default_rng(33)
    V, k = 32, 12
    nbr = _table(rng, V, k)
    for trial in range(300):
        q, p = _dists(rng, V, conc=0.3)
        x = int(rng.integers(V))
        kk = int(rng.integers(0, k + 1))
        delta = float(rng.choice([1e-9, 0.01, 0.05, 0.2, 0.5, 2.0]))
        m, members = oracle.relaxed_mass(q, x, nbr, kk, 1.0, 0, V, delta=delta)
        run = np.cumsum(q[nbr[x][:kk]])
        ok = run < delta
        n_take = kk if ok.all() else int(np.argmin(ok))
        assert members == [int(a) for a in nbr[x][:n_take]]
        assert np.isclose(m, q[x] + q[nbr[x][:n_take]].sum(), rtol=1e-14)
        qt = oracle.moved_mass(q, x, m, members)
        tvd = 0.5 * np.abs(qt - q).sum()
        assert abs(tvd - (m - q[x])) < 1e-13 and (tvd < delta or n_take == 0)
        if delta == 2.0:
            assert n_take == kk
        if delta == 1e-9:
            assert all(q[a] < 1e-9 for a in members)
        # the accept probability uses m exactly as in the multiplicative rule
        _, _, tested = oracle.sibling_loop(q, p, [1], [0, x], [0, 1.0], nbr, kk, 1.0, 0, V, delta=delta)
        assert tested[1][0] == m and tested[1][1] == (min(1.0, m / p[x]) if p[x] > 0 else float(m > 0))
        # same bound, written either way
        lam = float(rng.choice([1.5, 3.0, 8.0]))
        if q[x] > 0:
            m_l, mem_l = oracle.relaxed_mass(q, x, nbr, kk, lam, 0, V)
            m_d, mem_d = oracle.relaxed_mass(q, x, nbr, kk, 1.0, 0, V, delta=(lam - 1.0) * q[x])
            bound = lam * q[x]
            near = np.abs(q[x] + np.cumsum(q[nbr[x][:kk]]) - bound).min() < 1e-12 if kk else False
            assert near or (mem_l == mem_d and np.isclose(m_l, m_d, rtol=1e-14))


def test_moved_mass_is_a_distribution_with_tvd_equal_to_moved_mass():
    rng = np.random.default_rng(3)
    V, k = 20, 8
    nbr = _table(rng, V, k)
    for trial in range(100):
        q, _ = _dists(rng, V)
        x = int(rng.integers(V))
        m, members = oracle.relaxed_mass(q, x, nbr, k, 4.0, 0, V)
        qt = oracle.moved_mass(q, x, m, members)
        assert np.all(qt >= 0) and abs(qt.sum() - 1) < 1e-13
        assert abs(0.5 * np.abs(qt - q).sum() - (m - q[x])) < 1e-13


def test_codes_are_a_sub_range_of_the_vocabulary():
    """Tokens outside [code_offset, code_offset + L) have no neighbours; inside,
    neighbour r of token x is code_offset + table[x - code_offset][r]."""
    rng = np.random.default_rng(4)
    V, L, off, k = 40, 10, 7, 4
    nbr = _table(rng, L, k)
    q, _ = _dists(rng, V, conc=2.0)
    for x in range(V):
        m, members = oracle.relaxed_mass(q, x, nbr, k, 1e9, off, L)
        if off <= x < off + L:
            assert members == [off + int(a) for a in nbr[x - off]]
        else:
            assert members == [] and m == q[x]


def _emitted_exact(q, p, s, nbr, k, lam):
    """Exact law of the token emitted at one node with s children drawn without
    replacement from p: enumerate ordered draft tuples with their
    successive-sampling probabilities, read the accept thresholds and the
    final residual from a run with every child rejected."""
    V = len(q)
    out = np.zeros(V)
    for drafts in itertools.permutations(range(V), s):
        w, rest = 1.0, 1.0
        for x in drafts:
            w *= p[x] / rest
            rest -= p[x]
        if w == 0:
            continue
        tokens = [0] + list(drafts)
        _, q_fin, tested = oracle.sibling_loop(q, p, list(range(1, s + 1)), tokens,
                                               [0.0] + [1.0] * s, nbr, k, lam, 0, V)
        alive = 1.0
        for c in range(1, s + 1):
            thr = tested[c][1]
            out[drafts[c - 1]] += w * alive * thr
            alive *= 1 - thr
        out += w * alive * q_fin
    return out


def test_unrelaxed_tree_node_emits_exactly_the_target():
    """Speculative sampling is faithful to q (App. A.2, after Eq. 2); the same
    holds for s siblings drawn without replacement and tested in turn."""
    rng = np.random.default_rng(5)
    V = 6
    nbr = _table(rng, V, 3)
    for trial in range(3):
        q, p = _dists(rng, V, conc=1.0)
        for s in (1, 2, 3):
            assert np.allclose(_emitted_exact(q, p, s, nbr, 0, 3.0), q, atol=1e-12)
            assert np.allclose(_emitted_exact(q, p, s, nbr, 3, 1.0), q, atol=1e-12)
    # relaxed: still a distribution, and it differs from q
    q, p = _dists(rng, V, conc=1.0)
    e = _emitted_exact(q, p, 2, nbr, 3, 3.0)
    assert abs(e.sum() - 1) < 1e-12 and np.all(e >= 0) and np.abs(e - q).max() > 1e-4


def test_monte_carlo_emitted_distribution_chi_square():
    """V = 16: tokens emitted by sampler + verifier with random uniforms follow
    the exact relaxed law (and q itself without relaxation)."""
    rng = np.random.default_rng(6)
    V, trials = 16, 12000
    nbr = _table(rng, V, 4)
    q, p = _dists(rng, V, conc=1.0)
    for k, lam in ((0, 1.0), (4, 2.5)):
        expect = _emitted_exact(q, p, 2, nbr, k, lam) if k else q
        counts = np.zeros(V)
        for t in range(trials):
            toks, _ = oracle.sample_children(p, rng.uniform(1e-9, 1, V), 2)
            nxt, tok, _ = oracle.verify_node(q, p, [1, 2], [0] + toks, rng.uniform(0, 1, 3),
                                             rng.uniform(), nbr, k, lam, 0, V)
            counts[toks[nxt - 1] if nxt > 0 else tok] += 1
        chi2 = ((counts - trials * expect) ** 2 / (trials * expect)).sum()
        assert chi2 < 44.3      # 15 dof, p ~ 1e-4


def test_full_neighbourhood_unbounded_lambda_always_accepts():
    rng = np.random.default_rng(7)
    V = 12
    nbr = _table(rng, V, V - 1)
    q, p = _dists(rng, V)
    for x in range(V):
        _, _, tested = oracle.sibling_loop(q, p, [1], [0, x], [0, 0.999999], nbr, V - 1, 1e30, 0, V)
        m, thr = tested[1][:2]
        assert abs(m - 1) < 1e-12 and thr == 1.0 or p[x] > m


def test_inverse_cdf_token_order():
    d = np.array([0.0, 0.25, 0.0, 0.5, 0.25, 0.0])
    assert oracle.inverse_cdf(d, 0.0) == 1
    assert oracle.inverse_cdf(d, 0.2499) == 1
    assert oracle.inverse_cdf(d, 0.25) == 3       # cdf must exceed u strictly
    assert oracle.inverse_cdf(d, 0.7499) == 3
    assert oracle.inverse_cdf(d, 0.75) == 4
    assert oracle.inverse_cdf(d, 0.999999) == 4
    assert oracle.inverse_cdf(3 * d, 0.5) == 3    # unnormalised input


def test_walk_every_path_of_a_seven_node_tree():
    #        0
    #      1   2
    #     3 4  5
    #     6
    parent = [-1, 0, 0, 1, 1, 2, 3]
    tokens = [0, 11, 12, 13, 14, 15, 16]
    children = oracle.tree_children(parent)
    assert children == [[1, 2], [3, 4], [5], [6], [], [], []]
    node_token = [100, 101, 102, 103, 104, 105, 106]
    cases = {
        (): (0, [100], [0]),
        (1,): (1, [11, 101], [1, 1]),
        (2,): (1, [12, 102], [2, 2]),
        (1, 3): (2, [11, 13, 103], [1, 3, 3]),
        (1, 4): (2, [11, 14, 104], [1, 4, 4]),
        (2, 5): (2, [12, 15, 105], [2, 5, 5]),
        (1, 3, 6): (3, [11, 13, 16, 106], [1, 3, 6, 6]),
    }
    for path, want in cases.items():
        nxt = [-1] * 7
        cur = 0
        for c in path:
            nxt[cur] = c
            cur = c
        assert oracle.walk(nxt, node_token, tokens) == want


def test_identical_models_accept_the_first_child_chain():
    """p == q: the first child has accept probability 1 at every node."""
    rng = np.random.default_rng(8)
    parent = [-1, 0, 0, 1, 1, 2, 3]
    V = 32
    logits = rng.standard_normal((7, V)).astype(np.float32)
    gum = rng.uniform(0.01, 0.99, (7, V))
    tokens, prob = oracle.sample_draft_tree(parent, logits, None, gum)
    tokens[0] = 0
    nbr = _table(rng, V, 4)
    out = oracle.verify_sequence(parent, logits, None, logits, None, tokens,
                                 rng.uniform(0, 1, 7), rng.uniform(0, 1, 7), nbr, lam=2.0, k=4,
                                 n_codes=V)
    assert out["accept_len"] == 3 and out["out_nodes"] == [1, 3, 6, 6]
    assert out["out_tokens"][:3] == [int(tokens[1]), int(tokens[3]), int(tokens[6])]
    assert list(out["node_thresh"][[1, 3, 6]]) == [1.0, 1.0, 1.0]
    assert list(out["node_mass"][[0, 2, 4]]) == [-1, -1, -1]      # root and later siblings: never tested
    # emitted count = accepted + 1 (step-compression numerator, Sec. 5)
    assert len(out["out_tokens"]) == out["accept_len"] + 1


def test_bound_is_strict_at_an_exact_tie():
    """Sec. 4 displays the bound with "<": a neighbour whose mass brings the running sum exactly
    to lambda * q(x) stays out (binary fractions, so the tie is exact in floating point), and
    with lambda = 1 nothing can join."""
    q = np.array([0.25, 0.25, 0.125, 0.125, 0.25])
    nbr = np.array([[1, 2, 3, 4], [0, 2, 3, 4], [0, 1, 3, 4], [0, 1, 2, 4], [0, 1, 2, 3]])
    m, members = oracle.relaxed_mass(q, 0, nbr, 4, 2.0, 0, 5)          # 0.25 + 0.25 == 2 * 0.25: stop
    assert m == 0.25 and members == []
    m, members = oracle.relaxed_mass(q, 2, nbr, 4, 3.0, 0, 5)          # bound 0.375: 0.125 + 0.25 == bound
    assert m == 0.125 and members == []
    m, members = oracle.relaxed_mass(q, 0, nbr, 4, 2.5, 0, 5)          # bound 0.625: one joins, 0.5 + 0.125 == bound stops
    assert m == 0.5 and members == [1]
    m, members = oracle.relaxed_mass(q, 0, nbr, 4, 1.0, 0, 5)
    assert m == 0.25 and members == []
    # additive variant (Sec. 2.2): the neighbours' own sum must stay strictly below delta
    m, members = oracle.relaxed_mass(q, 0, nbr, 4, 1.0, 0, 5, delta=0.25)
    assert m == 0.25 and members == []
    m, members = oracle.relaxed_mass(q, 0, nbr, 4, 1.0, 0, 5, delta=0.375)
    assert m == 0.5 and members == [1]


def test_greedy_skip_subset():
    """The other reading of Sec. 4's subset: a neighbour that would break the bound is passed
    over.  Checked through the defining property (r joins iff the sum of x and of the earlier
    members plus q(r) stays below the bound), not through the loop that builds it."""
    rng = np.random.default_rng(11)
    V, k = 32, 12
    nbr = _table(rng, V, k)
    differs = 0
    for trial in range(300):
        q, _ = _dists(rng, V, conc=0.3)
        lam = float(rng.choice([1.0, 1.5, 2.0, 3.0]))
        x = int(rng.integers(V))
        m, members = oracle.relaxed_mass(q, x, nbr, k, lam, 0, V, skip=True)
        m0, prefix = oracle.relaxed_mass(q, x, nbr, k, lam, 0, V)
        assert members[: len(prefix)] == prefix and m >= m0           # the prefix comes first
        assert m < lam * q[x] or (members == [] and m == q[x])
        assert np.isclose(m, q[x] + sum(q[a] for a in members), rtol=1e-14)
        inside = set(members)
        run = q[x]
        for a in (int(t) for t in nbr[x][:k]):
            fits = run + q[a] < lam * q[x]
            assert fits == (a in inside)
            if fits:
                run += q[a]
        differs += members != prefix
    assert differs > 20          # the two readings really differ on these inputs


def test_deterministic_draft_mode():
    """Sec. 3: a deterministically chosen draft has p(x) = 1, so it is accepted with probability
    m (= q(x) without relaxation), and the emitted token still follows q exactly when k = 0,
    whatever the drafts are: enumerate the sibling loop for s = 1, 2, 3."""
    rng = np.random.default_rng(12)
    V = 9
    nbr = _table(rng, V, 4)
    for trial in range(20):
        q, _ = _dists(rng, V, conc=0.6)
        for s in (1, 2, 3):
            xs = [int(t) for t in rng.choice(V, size=s, replace=False)]
            tokens = [0] + xs
            kids = list(range(1, s + 1))
            # thresholds met along the all-reject path, and the distribution left at its end
            _, q_fin, tested = oracle.sibling_loop(q, None, kids, tokens, [0.0] + [1.0] * s, nbr, 0, 3.0, 0, V,
                                                   det_draft=True)
            law = np.zeros(V)
            reach = 1.0
            for c in kids:
                m, thr = tested[c][:2]
                assert thr == m
                law[tokens[c]] += reach * thr
                reach *= 1.0 - thr
            law += reach * q_fin
            assert np.allclose(law, q, atol=1e-14)
            m1 = tested[1][0]
            assert m1 == q[xs[0]]
        # with relaxation the accept probability is the relaxed mass, within the bound
        x = int(rng.integers(V))
        _, _, tested = oracle.sibling_loop(q, None, [1], [0, x], [0.0, 1.0], nbr, 4, 2.0, 0, V, det_draft=True)
        m, thr = tested[1][:2]
        assert thr == min(1.0, m) and q[x] <= m and (m < 2.0 * q[x] or m == q[x])
