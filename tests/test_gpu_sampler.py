"""Parity of lantern_sample_draft_tree with the oracle (Sec. 2.1: s tokens per node drawn from
p, read as Gumbel-top-s without replacement)."""
import numpy as np
import pytest
import torch

import oracle
import workloads as W
from gpu_cases import Case, f64, small_config
from parity_util import KEY_TIE

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    import paper_2502_06352_b200 as lib
    return lib


def _gpu_sample(L, case, gumbel=None, seed_step=None, parent_range=(0, None), tokens=None):
    g, par, _, _ = case.gpu_inputs(L)
    tree = L.Tree(case.parent)
    if seed_step:
        par.seed, par.step = seed_step
    prob = torch.zeros((case.B, case.N), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tok = L.sample_draft_tree(par, tree, g["draft_cond"], g["draft_uncond"], tokens=tokens,
                              parent_begin=parent_range[0], parent_end=parent_range[1],
                              gumbel_uniforms=None if gumbel is None else gumbel.cuda(), draft_prob=prob,
                              device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return tok.cpu().numpy(), prob.cpu().numpy(), tok


def _compare(case, gum, gtok, gprob):
    kids = oracle.tree_children(case.parent)
    ties = 0
    for b in range(case.B):
        du = case.logits["draft_uncond"]
        for n in range(case.N):
            if not kids[n]:
                continue
            p, _ = oracle.postprocess_row(f64(case.logits["draft_cond"][b, n]), None if du is None else f64(du[b, n]),
                                          case.params["cfg_scale"], case.params["temperature"],
                                          case.params["top_k_draft"], case.params["allowed_begin"],
                                          case.params["allowed_end"])
            want, wp, gaps = oracle.sample_children(p, gum[b, n], len(kids[n]), return_gaps=True)
            got = [int(gtok[b, c]) for c in kids[n]]
            if got != want:
                r = next(i for i in range(len(want)) if got[i] != want[i])
                assert min(gaps[max(0, r - 1): r + 1]) < KEY_TIE, ("sampler mismatch", b, n, got, want, gaps)
                ties += 1
                continue
            assert np.allclose(gprob[b, kids[n]], wp, atol=1e-5)
            real = [t for t in got if t >= 0]
            assert len(set(real)) == len(real)
    return ties


@pytest.mark.parametrize("kw", [dict(), dict(cfg_scale=None), dict(top_k=20), dict(dtype="bf16", cfg_scale=None),
                                dict(vocab=1003, codebook_size=1003), dict(n_nodes=60, temperature=0.8)])
@pytest.mark.parametrize("kernels", [1, 2])          # streaming kernel forced / excluded
def test_explicit_uniforms(L, kw, kernels):
    pad = 5 if kw.get("vocab") == 1003 else 0
    case = Case(small_config(**kw), seed=21, tokens="random", pad=pad, kernels=kernels)
    gum = W.make_gumbel_uniforms(case.B, case.N, case.V, 1234)
    gtok, gprob, _ = _gpu_sample(L, case, gumbel=gum)
    assert _compare(case, gum.numpy(), gtok, gprob) <= 1
    assert np.all(gtok[:, 0] == -1)


@pytest.mark.parametrize("cs", [1, 2, 8])
def test_cluster_sizes_and_allowed_range(L, cs):
    case = Case(small_config(vocab=2048, codebook_size=512, code_offset=256, top_k=30), seed=22,
                tokens="random", allowed=(256, 768))
    gum = W.make_gumbel_uniforms(case.B, case.N, case.V, 99)
    old = L.set_cluster_size(cs)
    try:
        gtok, gprob, _ = _gpu_sample(L, case, gumbel=gum)
    finally:
        L.set_cluster_size(old)
    assert _compare(case, gum.numpy(), gtok, gprob) <= 1
    assert np.all((gtok[:, 1:] >= 256) & (gtok[:, 1:] < 768))


@pytest.mark.parametrize("cs", [0, 1])
@pytest.mark.parametrize("kw", [dict(vocab=3001, codebook_size=3001, top_k=200),
                                dict(vocab=9000, codebook_size=2000, top_k=1000, dtype="bf16", cfg_scale=None)])
def test_topk_rows_list_and_dense_kernels(L, cs, kw):
    # cs = 0: the list-based kernel; cs = 1: the dense kernel.  Philox uniforms, so the list kernel
    # has to pick the right word of each token's counter block.
    case = Case(small_config(**kw), seed=25, tokens="random", pad=3 if kw.get("dtype", "f32") == "f32" else 8)
    seed, step = 0x5EED, 11
    gum = np.empty((case.B, case.N, case.V), dtype=np.float32)
    for b in range(case.B):
        for n in range(case.N):
            gum[b, n] = oracle.stream_uniforms(seed, step, b * case.N + n, 0, count=case.V)
    old = L.set_cluster_size(cs)
    try:
        gtok, gprob, _ = _gpu_sample(L, case, seed_step=(seed, step))
    finally:
        L.set_cluster_size(old)
    assert _compare(case, gum, gtok, gprob) <= 1


def test_topk_with_massive_ties_is_redrawn_by_the_dense_kernel(L):
    # logits on a grid of 2.0: the k-th largest value is shared by more entries than the list
    # kernel holds, so it marks every parent and the dense kernel draws them
    case = Case(small_config(vocab=8000, codebook_size=1000, top_k=300, cfg_scale=None, batch=2), seed=26,
                tokens="random")
    for v in case.padded.values():
        if v is not None:
            v.copy_(torch.round(v / 2.0) * 2.0)
    gum = W.make_gumbel_uniforms(case.B, case.N, case.V, 77)
    gtok, gprob, _ = _gpu_sample(L, case, gumbel=gum)
    assert _compare(case, gum.numpy(), gtok, gprob) <= 1
    assert np.all(gtok[:, 1:] >= 0)


def test_philox_uniforms_and_level_by_level(L):
    case = Case(small_config(batch=2), seed=23, tokens="random")
    seed, step = 0xABCDEF12345, 7
    gum = np.empty((case.B, case.N, case.V), dtype=np.float32)
    for b in range(case.B):
        for n in range(case.N):
            gum[b, n] = oracle.stream_uniforms(seed, step, b * case.N + n, 0, count=case.V)
    gtok, gprob, _ = _gpu_sample(L, case, seed_step=(seed, step))
    assert _compare(case, gum, gtok, gprob) <= 1
    # expanding one level at a time fills the same tokens
    depth = [0] * case.N
    for i in range(1, case.N):
        depth[i] = depth[case.parent[i]] + 1
    tok = None
    for d in range(max(depth) + 1):
        ids = [i for i in range(case.N) if depth[i] == d]
        _, _, tok = _gpu_sample(L, case, seed_step=(seed, step), parent_range=(ids[0], ids[-1] + 1), tokens=tok)
    assert np.array_equal(tok.cpu().numpy(), gtok)


def test_small_support_gives_minus_one(L):
    # only 2 allowed tokens but 4 children at the root
    case = Case(small_config(batch=1), seed=24, tokens="random", allowed=(10, 12))
    gum = W.make_gumbel_uniforms(case.B, case.N, case.V, 5)
    gtok, gprob, _ = _gpu_sample(L, case, gumbel=gum)
    kids = oracle.tree_children(case.parent)
    root = [int(gtok[0, c]) for c in kids[0]]
    assert sorted(root[:2]) == [10, 11] and root[2:] == [-1] * (len(root) - 2)
    assert _compare(case, gum.numpy(), gtok, gprob) == 0


def test_first_child_follows_p_chi_square(L):
    """V = 16: over many independent rows the first child is distributed as p (Philox path)."""
    V, B = 16, 4096
    cfg = small_config(vocab=V, codebook_size=V, batch=B, cfg_scale=None, k=0)
    parent = [-1, 0, 0]
    row = torch.randn(V, generator=torch.Generator().manual_seed(3)) * 1.2
    logits = row.repeat(B, 3, 1).contiguous().cuda()
    tree = L.Tree(parent)
    par = L.Params(vocab=V, seed=77, step=1)
    counts = np.zeros(V)
    pair = {}
    for step in range(8):
        par.step = step
        tok = L.sample_draft_tree(par, tree, logits, None).cpu().numpy()
        counts += np.bincount(tok[:, 1], minlength=V)
        assert np.all(tok[:, 1] != tok[:, 2])
    p = torch.softmax(row.double(), 0).numpy()
    n = counts.sum()
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < 44.3       # 15 dof, p ~ 1e-4


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
@pytest.mark.parametrize("kw", [dict(vocab=65536, codebook_size=1024, dtype="bf16", cfg_scale=None),
                                dict(vocab=16384, codebook_size=1024, temperature=0.7),
                                dict(vocab=5000, codebook_size=1024, n_nodes=26, cfg_scale=None)])
def test_streaming_kernel_over_seeds_and_row_shapes(L, seed, kw):
    """The streaming sampler (forced) on rows of the benchmark's width and smaller, several seeds: first
    threshold from the warps' best keys, the scheduled cut, the exact ranking."""
    case = Case(small_config(batch=2, **kw), seed=100 + seed, tokens="random", kernels=1)
    gum = W.make_gumbel_uniforms(case.B, case.N, case.V, 4321 + seed)
    gtok, gprob, _ = _gpu_sample(L, case, gumbel=gum)
    assert _compare(case, gum.numpy(), gtok, gprob) <= 1


@pytest.mark.parametrize("shape", ["rising", "falling", "flat"])
def test_streaming_kernel_on_monotone_and_constant_rows(L, shape):
    """Rows whose logits rise along the row keep producing keys above every earlier threshold (the candidate
    list overflows and the row is redone with a cut after every chunk); falling rows never do; constant rows
    leave everything to the uniforms.  All must agree with the oracle."""
    case = Case(small_config(batch=2, vocab=65536, codebook_size=1024, dtype="f32", cfg_scale=None), seed=77,
                tokens="random", kernels=1)
    V = case.V
    ramp = torch.linspace(-30.0, 30.0, V)
    row = {"rising": ramp, "falling": ramp.flip(0), "flat": torch.zeros(V)}[shape]
    case.padded["draft_cond"][:, :, :V] = row
    gum = W.make_gumbel_uniforms(case.B, case.N, V, 99)
    gtok, gprob, _ = _gpu_sample(L, case, gumbel=gum)
    assert _compare(case, gum.numpy(), gtok, gprob) <= 1
