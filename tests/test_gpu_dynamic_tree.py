"""Parity of lantern_expand_frontier / lantern_trim_tree with oracle/dynamic_tree.py (Sec. 2.1, dynamic tree
drafting; Sec. 3), and verification of the drafted (ragged, per-sequence) trees with deterministic drafts."""
import numpy as np
import pytest
import torch

import oracle
from oracle import dynamic_tree as DT
from gpu_cases import Case, small_config, f64
from parity_util import compare_verify, check_walk

pytestmark = pytest.mark.gpu

TIE = 1e-6          # a choice may differ from the oracle's only where the oracle's log V gap is below this


@pytest.fixture(scope="module")
def L():
    import paper_2502_06352_b200 as lib
    return lib


def _draft(L, data, unc, K, E, m, dtype, **pk):
    """Runs the device loop over depths on rows data[d][b][slot][:] and the oracle on the same rows."""
    D, B, _, V = data.shape
    to = lambda t: None if t is None else t.to(dtype).cuda()
    par = L.Params(vocab=V, **pk)
    pool = L.DraftPool(B, D, K, E)
    for d in range(D):
        F = pool.frontier.shape[1]
        L.expand_frontier(par, pool, to(data[d][:, :F].contiguous()), to(None if unc is None else unc[d][:, :F].contiguous()))
    n, parent, token, index, logv = L.trim_tree(pool, m)
    torch.cuda.synchronize()
    gpu = dict(n=n.cpu().numpy(), parent=parent.cpu().numpy(), token=token.cpu().numpy(), index=index.cpu().numpy(),
               logv=logv.cpu().numpy(), pool_parent=pool.parent.cpu().numpy(), pool_token=pool.token.cpu().numpy(),
               pool_logv=pool.logv.cpu().numpy(), pool_depth=pool.depth.cpu().numpy())
    as32 = lambda t: t.to(dtype).to(torch.float32).numpy()
    orc = []
    for b in range(B):
        margins = []
        row_of = lambda d, s, b=b: (as32(data[d][b][s]), None if unc is None else as32(unc[d][b][s]))
        t = DT.draft_dynamic_tree(row_of, D, K, E, m, cfg_scale=pk.get("cfg_scale"), temperature=pk.get("temperature", 1.0),
                                  allowed_begin=pk.get("allowed_begin", 0), allowed_end=pk.get("allowed_end") or None,
                                  margins=margins)
        t["margins"] = margins
        orc.append(t)
    return gpu, orc


def _compare(gpu, orc, m):
    ties = 0
    for b, t in enumerate(orc):
        Pn = len(t["pool_parent"])
        same_pool = (np.array_equal(gpu["pool_parent"][b][:Pn], t["pool_parent"])
                     and np.array_equal(gpu["pool_token"][b][:Pn], t["pool_token"]))
        n = int(gpu["n"][b])
        same_tree = (same_pool and n == len(t["parent"]) and np.array_equal(gpu["parent"][b][:n], t["parent"])
                     and np.array_equal(gpu["token"][b][:n], t["token"]) and np.array_equal(gpu["index"][b][:n], t["pool_index"]))
        if not same_tree:
            # only a near-tie of two log V at a cut may make the choices differ
            assert t["margins"] and min(t["margins"]) < TIE, (b, min(t["margins"]) if t["margins"] else None)
            ties += 1
            continue
        assert np.array_equal(gpu["pool_depth"][b][:Pn], t["pool_depth"])
        fin = np.isfinite(t["pool_logv"])
        assert np.array_equal(np.isfinite(gpu["pool_logv"][b][:Pn]), fin)
        assert np.allclose(gpu["pool_logv"][b][:Pn][fin], t["pool_logv"][fin], rtol=0, atol=1e-5)
        assert np.allclose(gpu["logv"][b][:n], t["logv"], rtol=0, atol=1e-5)
        assert np.all(gpu["parent"][b][n:] == -1) and np.all(gpu["index"][b][n:] == -1)
    return ties


@pytest.mark.parametrize("V,K,E,D,m,scale,dtype,pk", [
    (1003, 3, 4, 4, 20, 1.0, torch.float32, {}),
    (16384, 4, 8, 5, 48, 2.0, torch.float32, {}),
    (16384, 8, 8, 6, 59, 0.5, torch.float32, dict(temperature=0.8)),                 # diffuse rows: shallow trees
    (65536, 8, 10, 6, 59, 3.0, torch.bfloat16, dict(allowed_begin=4096, allowed_end=12288)),
    (4096, 2, 2, 7, 1000, 4.0, torch.bfloat16, {}),                                  # m above the pool: nothing trimmed
    (257, 8, 16, 3, 30, 1.0, torch.float32, {}),
])
def test_drafted_trees_match_the_oracle(L, V, K, E, D, m, scale, dtype, pk):
    g = torch.Generator().manual_seed(V + K + E)
    B = 3
    data = torch.randn((D, B, E, V), generator=g) * scale
    gpu, orc = _draft(L, data, None, K, E, m, dtype, **pk)
    ties = _compare(gpu, orc, m)
    assert ties <= 1


def test_guidance_rows_and_ties_inside_a_row(L):
    g = torch.Generator().manual_seed(5)
    D, B, E, V, K = 3, 2, 4, 2000, 4
    cond = torch.randn((D, B, E, V), generator=g)
    unc = torch.randn((D, B, E, V), generator=g)
    cond[:, :, :, 100:140] = 6.0          # forty equal best tokens per row: children are the lowest ids
    unc[:, :, :, 100:140] = 1.0
    gpu, orc = _draft(L, cond, unc, K, E, 25, torch.float32, cfg_scale=2.5, temperature=1.3)
    assert _compare(gpu, orc, 25) == 0
    assert list(gpu["token"][0][1:5]) == [100, 101, 102, 103]


def test_low_confidence_gives_shallow_trees_on_the_device_too(L):
    """Sec. 3: the product of low confidences decays fast, so diffuse rows give wide, shallow trees."""
    g = torch.Generator().manual_seed(8)
    D, B, E, V, K, m = 6, 8, 8, 8192, 8, 40
    base = torch.randn((D, B, E, V), generator=g)
    depth = {}
    for scale in (0.25, 6.0):
        gpu, orc = _draft(L, base * scale, None, K, E, m, torch.float32)
        assert _compare(gpu, orc, m) <= 1
        means = []
        for b in range(B):
            n = int(gpu["n"][b])
            dep = gpu["pool_depth"][b][gpu["index"][b][:n]]
            means.append(dep.mean())
        depth[scale] = float(np.mean(means))
    assert depth[6.0] > depth[0.25] + 0.5


def test_drafted_trees_are_verified_with_deterministic_drafts(L):
    """The workload end to end: every sequence drafts its own tree (different shapes), and each tree is
    verified with draft_deterministic = 1 (Sec. 3: p(x) = 1, accept probability = the relaxed mass)."""
    g = torch.Generator().manual_seed(21)
    D, B, E, V, K, m = 5, 3, 6, 1000, 4, 26
    data = torch.randn((D, B, E, V), generator=g) * 2.0
    gpu, orc = _draft(L, data, None, K, E, m, torch.float32)
    assert _compare(gpu, orc, m) == 0
    shapes = set()
    for b in range(B):
        n = int(gpu["n"][b])
        parent = [int(x) for x in gpu["parent"][b][:n]]
        shapes.add(tuple(parent))
        case = Case(small_config(batch=1, n_nodes=n, vocab=V, codebook_size=V, k=8, lam=3.0, cfg_scale=None), parent=parent,
                    seed=60 + b, det_draft=True, tokens="random")
        case.tokens[0, 1:] = gpu["token"][b][1:n]
        gi, par, nbr, tok = case.gpu_inputs(L)
        tree = L.Tree(parent)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = L.verify_tree(par, tree, nbr, gi["target_cond"], gi["target_uncond"], None, None, tok,
                            case.u_accept.cuda(), case.u_resample.cuda(), debug=True, device_status=status)
        torch.cuda.synchronize()
        res = {k: v.cpu().numpy() for k, v in out.items()}
        assert int(status.item()) == 0
        o = case.oracle_verify()
        stats = compare_verify(res, o, case.parent, case.u_accept.numpy(), case.seqs, rerun=case.oracle_node)
        check_walk(res, case.tokens, tree.max_depth, o, stats["dirty_sequences"], case.seqs, stats["patched"])
    assert len(shapes) > 1            # the trees really differ from sequence to sequence


@pytest.mark.parametrize("dtype,guided", [("f32", False), ("bf16", True)])
def test_a_forest_of_drafted_trees_is_verified_in_one_call(L, dtype, guided):
    """lantern_forest_create: every sequence keeps its own tree (padded to the largest); one verify call
    covers the batch; each sequence is compared with the oracle run on its own tree."""
    g = torch.Generator().manual_seed(33)
    D, B, E, V, K, m = 5, 4, 6, 1200, 4, 30
    data = torch.randn((D, B, E, V), generator=g) * torch.tensor([0.5, 1.5, 3.0, 6.0]).view(1, B, 1, 1)
    gpu, orc = _draft(L, data, None, K, E, m, torch.float32)
    assert _compare(gpu, orc, m) == 0
    n_nodes = [int(x) for x in gpu["n"]]
    parents = [[int(x) for x in gpu["parent"][b][:n_nodes[b]]] for b in range(B)]
    assert len({tuple(p) for p in parents}) > 1
    Nmax = max(n_nodes)
    cfg = small_config(batch=B, n_nodes=Nmax, vocab=V, codebook_size=V, k=8, lam=3.0, dtype=dtype,
                       cfg_scale=3.0 if guided else None)
    # the inputs of one [B][Nmax] call; a dummy chain tree only sizes the generators
    base = Case(cfg, parent=[-1] + list(range(Nmax - 1)), seed=70, det_draft=True, tokens="random")
    for b in range(B):
        base.tokens[b, 1:n_nodes[b]] = gpu["token"][b][1:n_nodes[b]]
    gi, par, nbr, tok = base.gpu_inputs(L)
    forest = L.Forest(parents, n_nodes, Nmax)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = L.verify_tree(par, forest, nbr, gi["target_cond"], gi["target_uncond"], None, None, tok,
                        base.u_accept.cuda(), base.u_resample.cuda(), debug=True, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    res = {k: v.cpu().numpy() for k, v in out.items()}
    lg = base.logits
    for b in range(B):
        n = n_nodes[b]
        o = oracle.verify_sequence(
            parents[b], f64(lg["target_cond"][b][:n]), None if lg["target_uncond"] is None else f64(lg["target_uncond"][b][:n]),
            None, None, base.tokens[b][:n], base.u_accept[b].numpy()[:n], base.u_resample[b].numpy()[:n], base.nbr,
            **base.params)
        stats = compare_verify(res, [o], parents[b], base.u_accept.numpy(), [b])
        assert stats["tie_accept"] + stats["tie_cut"] + stats["tie_resample"] == 0
        # the walk: accepted path and its length as the oracle walks them
        assert int(res["accept_len"][b]) == o["accept_len"]
        L1 = o["accept_len"] + 1
        assert list(res["out_tokens"][b][:L1]) == list(o["out_tokens"][:L1])
        # padding nodes: -1 on output
        assert np.all(res["node_next"][b][n:] == -1) and np.all(res["node_token"][b][n:] == -1)


def test_argument_errors_are_reported_before_anything_runs(L):
    """Error behaviour of the dynamic-tree entry points and of the forest handle (host-side checks)."""
    V = 512
    rows = torch.randn((1, 1, V)).cuda()
    pool = L.DraftPool(1, 2, 4, 4)
    with pytest.raises(L.LanternError):                       # truncated rows: confidences of a top-k row are not built
        L.expand_frontier(L.Params(vocab=V, top_k_draft=10), pool, rows)
    assert pool.used == 1 and pool.n_depths == 0              # nothing advanced
    with pytest.raises(L.LanternError):                       # more children than a tree node may have
        L.expand_frontier(L.Params(vocab=V), L.DraftPool(1, 2, 9, 4), rows)
    with pytest.raises(L.LanternError):                       # parents must be numbered breadth first
        L.Forest([[-1, 0, 0], [-1, 0, 1, 0]], [3, 4], 4)
    forest = L.Forest([[-1, 0, 0], [-1, 0, 1, 1]], [3, 4], 4)
    par = L.Params(vocab=V, k=0, draft_deterministic=1)
    tc = torch.randn((2, 4, V)).cuda()
    tok = torch.zeros((2, 4), dtype=torch.int32).cuda()
    u = torch.rand((2, 4)).cuda()
    with pytest.raises(L.LanternError):                       # a forest serves exactly its own number of sequences
        L.verify_tree(par, forest, None, tc[:1], None, None, None, tok[:1], u[:1], u[:1])
    with pytest.raises(L.LanternError):                       # ... on the streaming kernels only
        L.verify_tree(L.Params(vocab=V, k=0, draft_deterministic=1, top_k_target=50), forest, None, tc, None, None, None,
                      tok, u, u)
    with pytest.raises(L.LanternError):                       # ... and is never sampled
        L.sample_draft_tree(L.Params(vocab=V), forest, tc)
    out = L.verify_tree(par, forest, None, tc, None, None, None, tok, u, u)
    torch.cuda.synchronize()
    assert out["accept_len"].shape == (2,)
