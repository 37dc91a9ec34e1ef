"""Parity of lantern_verify_tree with the oracle (Sec. 4; App. A.2 Eq. 1-2; Sec. 2.1)."""
import numpy as np
import pytest
import torch

import oracle
import workloads as W
from gpu_cases import Case, small_config
from parity_util import check_walk, compare_verify

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    import paper_2502_06352_b200 as lib
    return lib


def _run(L, case, **kw):
    """Parity of one case; run with the streaming kernels forced and with them excluded, so that
    every kernel that can serve the parameters is compared with the oracle."""
    out = None
    for kernels in (2, 1):
        case.kernels = kernels
        res = case.gpu_verify(L, **kw)
        assert res["status"] == 0
        orc = case.oracle_verify()
        ua = case.u_accept.numpy()
        stats = compare_verify(res, orc, case.parent, ua, case.seqs, rerun=case.oracle_node)
        check_walk(res, case.tokens, res["max_depth"], orc, stats["dirty_sequences"], case.seqs, stats["patched"])
        assert stats["tie_accept"] + stats["tie_cut"] + stats["tie_resample"] <= max(1, stats["nodes"] // 500)
        out = (res, stats)
        if case.params["skip"] or case.params["det_draft"] or (case.params["top_k_target"] and case.params["top_k_draft"]):
            break               # one family of kernels serves these parameters
    return out


@pytest.mark.parametrize("cs", [0, 1, 2, 4, 8, 16])
def test_small_vocab_all_cluster_sizes(L, cs):
    # V = 1003 with a padded row stride: ragged tail in the last slice, several slices
    case = Case(small_config(vocab=1003, codebook_size=1003, k=8, lam=3.0), seed=1, pad=5)
    old = L.set_cluster_size(cs)
    try:
        _run(L, case)
    finally:
        L.set_cluster_size(old)


@pytest.mark.parametrize("kw", [
    dict(cfg_scale=None),                                   # no guidance rows
    dict(top_k=50),                                         # truncation on both sides
    dict(k=0),                                              # standard speculative sampling
    dict(lam=1.0),                                          # bound 1: A = {x}
    dict(lam=20.0, k=50),                                   # wide relaxation
    dict(dtype="bf16", cfg_scale=None),
    dict(dtype="bf16", top_k=30),
    dict(temperature=0.7, top_k=100),
    dict(codebook_size=300, code_offset=200, k=10),         # codes are a sub-range of the vocabulary
    dict(n_nodes=60, batch=3),
])
def test_parameter_variants(L, kw):
    case = Case(small_config(**kw), seed=2)
    _run(L, case)


@pytest.mark.parametrize("cs", [0, 1, 2])
@pytest.mark.parametrize("kw", [
    dict(vocab=3001, codebook_size=3001, top_k=200, k=12),
    dict(vocab=9000, codebook_size=2000, code_offset=500, top_k=1000, k=20, dtype="bf16", cfg_scale=None),
])
def test_topk_rows_on_every_path(L, cs, kw):
    # cs = 0: the list-based top-k kernel (rows of at most 16384 entries); cs = 1, 2: the dense
    # kernel in one CTA / a cluster of two
    case = Case(small_config(**kw), seed=13, pad=3 if kw.get("dtype", "f32") == "f32" else 8)   # rows stay 16-byte aligned
    old = L.set_cluster_size(cs)
    try:
        _run(L, case)
    finally:
        L.set_cluster_size(old)


def test_topk_target_only_and_leaf_only_tree(L):
    # top-k on the target side only: the drafter rows are dense, so the dense kernel runs
    case = Case(small_config(top_k=0), seed=14, top_k_target=60, top_k_draft=0)
    _run(L, case)
    # a tree without internal nodes never reads a drafter row
    leaf = Case(small_config(batch=3, top_k=40), parent=[-1], seed=15)
    _run(L, leaf)


def test_topk_with_massive_ties_is_repaired_by_the_dense_kernel(L):
    # logits on a grid of 2.0: a handful of distinct values per row, so the k-th largest value
    # is shared by far more entries than the list kernel's buffers hold (512 ties); those nodes
    # must come out right all the same
    case = Case(small_config(vocab=8000, codebook_size=1000, top_k=300, cfg_scale=None, batch=2), seed=16)
    for v in case.padded.values():
        if v is not None:
            v.copy_(torch.round(v / 2.0) * 2.0)
    _run(L, case)


def test_path_queries_and_graph_replay_match_eager_calls(L):
    """The library says which kernels a call runs; a captured and replayed call (the way the
    benchmark launches) gives the results of the eager call bit for bit."""
    case = Case(small_config(vocab=3001, codebook_size=3001, top_k=200, k=12), seed=17, pad=3)
    g, par, nbr, tok = case.gpu_inputs(L)
    tree = L.Tree(case.parent)
    B = case.B
    assert L.verify_tree_path(par, tree, B) == 1 and L.sample_draft_tree_path(par, tree, B) == 1
    par_dense = L.Params(**{**par.__dict__, "top_k_target": 0, "top_k_draft": 0})
    assert L.verify_tree_path(par_dense, tree, B) == 2 and L.sample_draft_tree_path(par_dense, tree, B) == 2      # streaming kernels (forced)
    par_auto = L.Params(**{**par_dense.__dict__, "kernels": 0})
    assert L.verify_tree_path(par_auto, tree, B) == 0 and L.sample_draft_tree_path(par_auto, tree, B) == 0    # a small call
    assert L.verify_tree_path(par_auto, tree, 64) == 2 and L.sample_draft_tree_path(par_auto, tree, 64) == 2
    par_walk = L.Params(**{**par.__dict__, "lazy_walk": 1})
    assert L.verify_tree_path(par_walk, tree, B) == 0         # top-k rows walk with the dense kernel
    old = L.set_cluster_size(1)
    try:
        assert L.verify_tree_path(par, tree, B) == 0
    finally:
        L.set_cluster_size(old)
    ua, ur = case.u_accept.cuda(), case.u_resample.cuda()
    eager = {k: v.clone() for k, v in L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"],
                                                    g["draft_cond"], g["draft_uncond"], tok, ua, ur, debug=True).items()}
    out = {}
    ws = torch.empty(L.lib.lantern_verify_tree_workspace(tree.handle, case.B), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):      # warm-up outside the capture (function attributes are set here)
        L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"],
                      tok, ua, ur, debug=True, out=out, workspace=ws)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(2):               # two dependent calls: the second overwrites the first's results
            L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"],
                          tok, ua, ur, debug=True, out=out, workspace=ws)
    for v in out.values():
        v.fill_(-3)
    graph.replay()
    torch.cuda.synchronize()
    for k, v in eager.items():
        assert torch.equal(out[k], v), k


def test_topk_rows_without_workspace_take_the_dense_kernel(L):
    # node_next / node_token are given and the workspace is too small for the repair flags: the
    # call is still valid (the dense kernel and the separate walk launch run) and gives the same results
    case = Case(small_config(top_k=50), seed=18)
    g, par, nbr, tok = case.gpu_inputs(L)
    tree = L.Tree(case.parent)
    ua, ur = case.u_accept.cuda(), case.u_resample.cuda()
    full = L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"],
                         tok, ua, ur, debug=True)
    tiny = L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"],
                         tok, ua, ur, debug=True, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    for k in ("accept_len", "out_tokens", "out_nodes", "node_next", "node_token"):
        assert torch.equal(full[k], tiny[k]), k
    for k in ("node_mass", "node_thresh"):
        assert torch.allclose(full[k], tiny[k], atol=1e-5), k
    res = {k: v.cpu().numpy() for k, v in tiny.items()}
    compare_verify(res, case.oracle_verify(), case.parent, case.u_accept.numpy(), case.seqs)


@pytest.mark.parametrize("delta", [0.02, 0.3, 2.0])
@pytest.mark.parametrize("kw", [dict(k=10), dict(k=16, top_k=100, vocab=3001, codebook_size=3001)])
def test_additive_bound_variant(L, delta, kw):
    # Sec. 2.2: neighbours are aggregated while their own mass stays below delta (lambda unused);
    # dense kernel (first case) and list kernel (second case)
    case = Case(small_config(lam=1.0, **kw), seed=19, delta=delta, pad=3 if "vocab" in kw else 0)
    res, stats = _run(L, case)
    if delta == 2.0:        # every neighbour joins: m = q(x) + sum over all k neighbours
        orc = case.oracle_verify()
        assert all(np.all(o["cut_margin"][np.isfinite(o["cut_margin"])] > 0.5) for o in orc)


@pytest.mark.parametrize("cs", [0, 1, 4])
@pytest.mark.parametrize("kw", [dict(batch=5, n_nodes=60), dict(top_k=80, dtype="bf16", cfg_scale=None, batch=3),
                                dict(draft_noise=0.05, batch=4)])
def test_path_walk_gives_the_results_of_verifying_every_node(L, cs, kw):
    """lazy_walk = 1 (Sec. 2.1 read as a walk from the root): same accepted path and emitted tokens
    as the launch over all nodes, and the per-node results on the path agree with the oracle."""
    case = Case(small_config(**kw), seed=20)
    g, par, nbr, tok = case.gpu_inputs(L)
    tree = L.Tree(case.parent)
    ua, ur = case.u_accept.cuda(), case.u_resample.cuda()
    old = L.set_cluster_size(cs)
    try:
        eager = L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"],
                              g["draft_uncond"], tok, ua, ur, debug=True)
        par.lazy_walk = 1
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = {k: torch.full_like(v, -5) for k, v in eager.items()}
        lazy = L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"],
                             g["draft_uncond"], tok, ua, ur, debug=True, out=out, device_status=status)
        torch.cuda.synchronize()
    finally:
        L.set_cluster_size(old)
    assert int(status.item()) == 0
    for k in ("accept_len", "out_tokens", "out_nodes"):
        assert torch.equal(lazy[k], eager[k]), k
    orc = case.oracle_verify()
    for b in range(case.B):
        path = [0] + [int(n) for n in lazy["out_nodes"][b, : int(lazy["accept_len"][b])].cpu()]
        for n in path:               # nodes on the path carry the same per-node results
            assert int(lazy["node_next"][b, n]) == int(eager["node_next"][b, n])
            assert int(lazy["node_token"][b, n]) == int(eager["node_token"][b, n])
        assert int(lazy["accept_len"][b]) == orc[b]["accept_len"] or b in _dirty(case, eager, orc)
    assert int(lazy["accept_len"].max()) >= 1 or kw.get("draft_noise") is None


def _dirty(case, eager, orc):
    res = {k: v.cpu().numpy() for k, v in eager.items()}
    return compare_verify(res, orc, case.parent, case.u_accept.numpy(), case.seqs)["dirty_sequences"]


def test_allowed_range_and_topk_counts_only_allowed(L):
    case = Case(small_config(vocab=2048, codebook_size=512, code_offset=256, k=6, top_k=40), seed=3,
                allowed=(256, 768))
    res, _ = _run(L, case)
    tok = res["node_token"]
    assert np.all((tok == -1) | ((tok >= 256) & (tok < 768)))


def test_unrelaxed_equals_textbook_thresholds(L):
    """k = 0: thr = min(1, q/p) on the rows as torch computes them."""
    case = Case(small_config(k=0, cfg_scale=None, batch=1), seed=4)
    res, _ = _run(L, case)
    q = torch.softmax(case.logits["target_cond"][0].double(), -1).numpy()
    p = torch.softmax(case.logits["draft_cond"][0].double(), -1).numpy()
    kids = oracle.tree_children(case.parent)
    for n in range(case.N):
        if kids[n]:
            c = kids[n][0]          # the first child sees the unmodified rows
            x = case.tokens[0, c]
            assert abs(res["node_thresh"][0, c] - min(1.0, q[n, x] / p[n, x])) < 1e-5
            assert abs(res["node_mass"][0, c] - q[n, x]) < 1e-6


def test_identical_models_accept_first_chain(L):
    cfg = small_config(draft_mix=1.0, draft_noise=0.0, batch=2)
    case = Case(cfg, seed=5)
    res, _ = _run(L, case)
    depth = 0
    n = 0
    kids = oracle.tree_children(case.parent)
    while kids[n]:
        n = kids[n][0]
        depth += 1
    assert list(res["accept_len"]) == [depth, depth]


def test_missing_drafts_and_single_node_tree(L):
    case = Case(small_config(batch=2), seed=6)
    case.tokens[0, 1] = -1           # first child of the root has no draft
    case.tokens[1, 2:5] = -1
    _run(L, case)
    leaf = Case(small_config(batch=3), parent=[-1], seed=7)
    res, _ = _run(L, leaf)
    assert list(res["accept_len"]) == [0, 0, 0] and res["out_tokens"].shape == (3, 1)


def test_philox_uniforms_match_oracle_stream(L):
    case = Case(small_config(batch=2), seed=8)
    seed, step = 0x1A27E2, (3 << 32) | 41
    for b in range(case.B):
        for n in range(case.N):
            case.u_accept[b, n] = float(oracle.stream_uniforms(seed, step, b * case.N + n, 1))
            case.u_resample[b, n] = float(oracle.stream_uniforms(seed, step, b * case.N + n, 2))
    _run(L, case, use_philox=(seed, step))


def test_bitwise_repeatable(L):
    case = Case(small_config(top_k=64), seed=9)
    a = case.gpu_verify(L)
    b = case.gpu_verify(L)
    for k in ("node_next", "node_token", "node_mass", "node_thresh", "accept_len", "out_tokens"):
        assert a[k].tobytes() == b[k].tobytes()


def test_bulk_copy_and_plain_table_paths_agree(L):
    # k_table = 8 rows are 16-byte aligned (bulk async copy); k_table = 7 uses plain loads
    a = Case(small_config(k=7), seed=10, k_table=8)
    b = Case(small_config(k=7), seed=10, k_table=7)
    ra, _ = _run(L, a)
    rb, _ = _run(L, b)
    assert np.array_equal(ra["node_next"], rb["node_next"]) and np.array_equal(ra["node_mass"], rb["node_mass"])


def test_bad_table_index_is_flagged_not_faulted(L):
    case = Case(small_config(batch=1, k=4), seed=11)
    case.nbr = case.nbr.copy()
    case.nbr[:, 1] = 10 ** 6          # outside the vocabulary
    res = case.gpu_verify(L)
    assert res["status"] & 1


def test_invalid_arguments_are_rejected(L):
    case = Case(small_config(batch=1), seed=12)
    g, par, nbr, tok = case.gpu_inputs(L)
    tree = L.Tree(case.parent)
    par.lam = 0.5
    with pytest.raises(L.LanternError) as e:
        L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"], tok)
    assert e.value.status == 1
    par.lam = 2.0
    par.k = 100                       # larger than the table
    with pytest.raises(L.LanternError):
        L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"], tok)
    par.k = 4
    bad = g["target_cond"][:, :, 1:]  # rows no longer 16-byte aligned
    with pytest.raises((L.LanternError, ValueError)):
        L.verify_tree(par, tree, nbr, bad, None, bad, None, tok)


@pytest.mark.parametrize("name", ["c1_tiny", "c2_llamagen512"])
def test_named_configs_full_size(L, name):
    case = Case(W.CONFIGS[name], seed=0)
    res, stats = _run(L, case)
    print(name, {k: v for k, v in stats.items() if k not in ("dirty_sequences", "patched")})


@pytest.mark.parametrize("name,seqs", [("c3_lumina", [0, 3]), ("c4_batch64", [0, 37, 63])])
def test_large_vocab_configs_sampled_sequences(L, name, seqs):
    case = Case(W.CONFIGS[name], seed=0, oracle_seqs=seqs)
    res, stats = _run(L, case)
    # properties that hold for every sequence
    tok = res["node_token"]
    nxt = res["node_next"]
    assert np.all((nxt >= 0) != (tok >= 0))
    thr = res["node_thresh"]
    assert np.all((thr == -1) | ((thr >= 0) & (thr <= 1)))
    print(name, {k: v for k, v in stats.items() if k not in ("dirty_sequences", "patched")})


def test_lumina_shape_with_the_table_the_library_built(L):
    """Config-3 shapes end to end: the verifier reads the neighbour table that
    lantern_build_neighbors made of the 8192 x 256 bf16 codebook; the oracle uses its own
    brute-force rows for the drafted codes."""
    import dataclasses
    cfg = dataclasses.replace(W.CONFIGS["c3_lumina"], batch=2)
    case = Case(cfg, seed=4, library_table=True, allowed=(cfg.code_offset, cfg.code_offset + cfg.codebook_size))
    res, stats = _run(L, case)
    assert stats["tested"] > 50


@pytest.mark.parametrize("cs", [0, 1, 4])
@pytest.mark.parametrize("kw", [dict(k=24, lam=1.8), dict(k=24, lam=1.8, dtype="bf16", cfg_scale=None),
                                dict(vocab=5003, codebook_size=5003, k=40, lam=1.6)])
def test_greedy_skip_subset_rule(L, cs, kw):
    """subset_rule = 1 (the other reading of Sec. 4's subset): parity with the oracle's greedy set."""
    pad = 5 if "vocab" in kw else 0
    old = L.set_cluster_size(cs)
    try:
        case = Case(small_config(**kw), seed=41, skip=True, pad=pad)
        _run(L, case)
    finally:
        L.set_cluster_size(old)
    # the rule matters on these inputs: the prefix rule gives other masses somewhere
    plain = Case(small_config(**kw), seed=41, pad=pad).oracle_verify()
    assert any(not np.allclose(a["node_mass"], b["node_mass"]) for a, b in zip(case.oracle_verify(), plain))


@pytest.mark.parametrize("cs", [0, 2])
@pytest.mark.parametrize("kw", [dict(), dict(dtype="bf16", cfg_scale=None, k=0), dict(n_nodes=60, lam=1.5)])
def test_deterministic_draft_mode(L, cs, kw):
    """draft_deterministic = 1 (Sec. 3): accept probability m, drafter rows never read (NULL)."""
    old = L.set_cluster_size(cs)
    try:
        case = Case(small_config(**kw), seed=43, det_draft=True)
        g, par, nbr, tok = case.gpu_inputs(L)
        tree = L.Tree(case.parent)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], None, None, tok,
                            case.u_accept.cuda(), case.u_resample.cuda(), debug=True, device_status=status)
        torch.cuda.synchronize()
        res = {k: v.cpu().numpy() for k, v in out.items()}
        assert int(status.item()) == 0
        orc = case.oracle_verify()
        stats = compare_verify(res, orc, case.parent, case.u_accept.numpy(), case.seqs, rerun=case.oracle_node)
        check_walk(res, case.tokens, tree.max_depth, orc, stats["dirty_sequences"], case.seqs, stats["patched"])
        thr, mass = res["node_thresh"], res["node_mass"]
        tested = mass >= 0
        assert np.allclose(thr[tested], np.minimum(1.0, mass[tested]), atol=1e-6)
    finally:
        L.set_cluster_size(old)


def test_path_walk_with_a_rule_variant_runs_on_the_streaming_kernel(L):
    case = Case(small_config(k=24, lam=1.8, batch=4, n_nodes=60), seed=45, skip=True)
    g, par, nbr, tok = case.gpu_inputs(L)
    tree = L.Tree(case.parent)
    ua, ur = case.u_accept.cuda(), case.u_resample.cuda()
    eager = L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"],
                          tok, ua, ur, debug=True)
    par.lazy_walk = 1
    assert L.verify_tree_path(par, tree, case.B) == 2
    lazy = L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"],
                         tok, ua, ur, debug=True)
    torch.cuda.synchronize()
    for k in ("accept_len", "out_tokens", "out_nodes"):
        assert torch.equal(lazy[k], eager[k]), k


def test_variants_are_refused_on_topk_rows(L):
    case = Case(small_config(top_k=50), seed=44)
    g, par, nbr, tok = case.gpu_inputs(L)
    tree = L.Tree(case.parent)
    for kw in (dict(subset_rule=1), dict(draft_deterministic=1)):
        bad = L.Params(**{**par.__dict__, **kw})
        with pytest.raises(L.LanternError) as e:
            L.verify_tree(bad, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"], tok)
        assert e.value.status == 2


@pytest.mark.parametrize("kernels", [1, 2])
def test_emitted_token_follows_the_relaxed_law_chi_square(L, kernels):
    """V = 16, a root with two children, the library's own Philox for the drafts, the accept tests
    and the residual draw: over 2^18 independent sequences the first emitted token follows the law
    that the sibling loop defines, enumerated exactly with the oracle over all ordered draft pairs
    (weights p_a p_b / (1 - p_a): sampling without replacement)."""
    V, B, k, lam = 16, 1 << 18, 3, 2.0
    g = torch.Generator().manual_seed(11)
    zq = (torch.randn(V, generator=g) * 1.3).float()
    zp = (zq * 0.8 + torch.randn(V, generator=g) * 0.6).float()
    cb = W.make_codebook(V, 3, "f32", seed=5)
    nbr, _ = oracle.neighbor_table(cb.to(torch.float64).numpy(), k)
    q, _ = oracle.postprocess_row(zq.numpy(), None, 1.0, 1.0, 0)
    p, _ = oracle.postprocess_row(zp.numpy(), None, 1.0, 1.0, 0)
    law = np.zeros(V)
    for a in range(V):
        for b in range(V):
            if a == b:
                continue
            w = p[a] * p[b] / (1.0 - p[a])
            _, q_fin, tested = oracle.sibling_loop(q, p, [1, 2], [0, a, b], [0.0, 1.0, 1.0], nbr, k, lam, 0, V)
            t1, t2 = tested[1][1], tested[2][1]
            law[a] += w * t1
            law[b] += w * (1 - t1) * t2
            law += w * (1 - t1) * (1 - t2) * q_fin
    assert abs(law.sum() - 1.0) < 1e-12
    parent = [-1, 0, 0]
    tree = L.Tree(parent)
    tq = zq.cuda().repeat(3, 1).view(1, 3, V).expand(B, 3, V)          # stride 0 over the sequences
    tp = zp.cuda().repeat(3, 1).view(1, 3, V).expand(B, 3, V)
    par = L.Params(vocab=V, lam=lam, k=k, n_codes=V, seed=2024, step=3, kernels=kernels)
    tok = L.sample_draft_tree(par, tree, tp, None)
    out = L.verify_tree(par, tree, torch.from_numpy(nbr.astype(np.int32)).cuda(), tq, None, tp, None, tok)
    torch.cuda.synchronize()
    first = out["out_tokens"][:, 0].cpu().numpy()
    counts = np.bincount(first, minlength=V).astype(np.float64)
    chi2 = ((counts - B * law) ** 2 / (B * law)).sum()
    assert chi2 < 50.0, (chi2, counts / B, law)            # 15 degrees of freedom: P(chi2 > 50) ~ 1e-5
    # and it is not the unrelaxed law: the relaxation is visible at this sample size
    plain = np.zeros(V)
    for a in range(V):
        for b in range(V):
            if a == b:
                continue
            w = p[a] * p[b] / (1.0 - p[a])
            _, q_fin, tested = oracle.sibling_loop(q, p, [1, 2], [0, a, b], [0.0, 1.0, 1.0], nbr, 0, 1.0, 0, V)
            t1, t2 = tested[1][1], tested[2][1]
            plain[a] += w * t1
            plain[b] += w * (1 - t1) * t2
            plain += w * (1 - t1) * (1 - t2) * q_fin
    assert np.allclose(plain, q, atol=1e-12)               # standard speculative sampling emits q
    assert ((counts - B * plain) ** 2 / (B * plain)).sum() > 200.0
