"""lantern_verify_tree_static: the verify entry point for callers that cannot allocate device
memory (its scratch is a fixed array inside the library).  Its results must equal those of
lantern_verify_tree on the same inputs, call after call, because both run the same kernels and
only the home of the per-node scratch differs.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from gpu_cases import Case, small_config

pytestmark = pytest.mark.gpu


def _both(L, case, lazy_walk=0):
    g, par, nbr, tok = case.gpu_inputs(L)
    par.lazy_walk = lazy_walk
    tree = L.Tree(case.parent)
    ua, ur = case.u_accept.cuda(), case.u_resample.cuda()
    ref = L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"],
                        tok, ua, ur, debug=True)
    D1 = tree.max_depth + 1
    out = dict(accept_len=torch.full((case.B,), -7, dtype=torch.int32, device="cuda"),
               out_tokens=torch.full((case.B, D1), -7, dtype=torch.int32, device="cuda"),
               out_nodes=torch.full((case.B, D1), -7, dtype=torch.int32, device="cuda"),
               node_mass=torch.zeros((case.B, case.N), dtype=torch.float32, device="cuda"),
               node_thresh=torch.zeros((case.B, case.N), dtype=torch.float32, device="cuda"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    L.verify_tree_static(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"], g["draft_uncond"],
                         tok, ua, ur, out=out, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for k in ("accept_len", "out_tokens", "out_nodes"):
        assert torch.equal(out[k], ref[k]), k
    # probabilities: same kernels, same inputs -> within the tolerance of the parity tests
    # (the path walk writes them for the nodes on the accepted path only)
    for k in ("node_mass", "node_thresh"):
        got, want = out[k].cpu().numpy(), ref[k].cpu().numpy()
        if lazy_walk:
            on = ref["out_nodes"].cpu().numpy()
            ln = ref["accept_len"].cpu().numpy()
            for b in range(case.B):
                path = [int(x) for x in on[b, : ln[b]]]
                assert np.allclose(got[b, path], want[b, path], atol=1e-5), k
        else:
            assert np.allclose(got, want, atol=1e-5), k
    return out


def test_static_scratch_matches_workspace_entry_point_twice():
    import paper_2502_06352_b200 as L
    assert L.lib.lantern_verify_tree_static_max_nodes() == 65536
    # two different calls in a row: the second finds the first call's contents in the scratch
    a = _both(L, Case(small_config(batch=3, top_k=40), seed=31))
    b = _both(L, Case(small_config(batch=2, n_nodes=60, cfg_scale=None, k=0), seed=32))
    assert a["accept_len"].shape == (3,) and b["accept_len"].shape == (2,)
    # and the first case again, after a larger one has overwritten the scratch
    _both(L, Case(small_config(batch=3, top_k=40), seed=31))


def test_path_walk_through_the_static_scratch_after_a_larger_call():
    """lazy_walk = 1 writes only the entries of the nodes on the accepted paths: whatever an
    earlier, larger call left in the shared array must not leak into its results."""
    import paper_2502_06352_b200 as L
    _both(L, Case(small_config(batch=6, n_nodes=60), seed=35))            # fills 360 entries
    _both(L, Case(small_config(batch=2), seed=36), lazy_walk=1)
    _both(L, Case(small_config(batch=3, top_k=40), seed=37), lazy_walk=1)


def test_static_scratch_allocates_nothing_and_holds_exactly_its_capacity():
    """The property the entry point exists for: a (warmed-up) call leaves the allocator's counters
    and the device's free memory where they were.  Run at exactly the capacity of the array."""
    import paper_2502_06352_b200 as L
    case = Case(small_config(vocab=64, codebook_size=64, batch=1, k=0, cfg_scale=None), parent=[-1], seed=34)
    g, par, nbr, tok = case.gpu_inputs(L)
    tree = L.Tree(case.parent)
    full = L.lib.lantern_verify_tree_static_max_nodes()      # batch * 1 node == capacity
    rows = g["target_cond"].expand(full, 1, 64)              # a view: stride 0 over the batch
    out = dict(accept_len=torch.full((full,), -7, dtype=torch.int32, device="cuda"),
               out_tokens=torch.full((full, 1), -7, dtype=torch.int32, device="cuda"),
               out_nodes=torch.full((full, 1), -7, dtype=torch.int32, device="cuda"))
    tokens = torch.zeros((full, 1), dtype=torch.int32, device="cuda")
    ur = case.u_resample.cuda().expand(full, 1).contiguous()
    ua = torch.zeros((full, 1), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def call():
        L.verify_tree_static(par, tree, None, rows, None, rows, None, tokens, ua, ur, out=out, device_status=status)
        torch.cuda.synchronize()

    call()                                                   # first call on the device: one-time set-up
    before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    call()
    after = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    assert after[0] == before[0] and after[1] == before[1]
    assert after[2] >= before[2]                             # free device memory did not shrink
    assert int(status.item()) == 0
    # every sequence saw the same row and the same uniform: one drawn token, the oracle's
    want = int(case.oracle_verify()[0]["node_token"][0])
    assert torch.all(out["accept_len"] == 0) and torch.all(out["out_tokens"] == want) and torch.all(out["out_nodes"] == 0)


def test_static_scratch_rejects_sizes_beyond_its_capacity():
    import paper_2502_06352_b200 as L
    case = Case(small_config(vocab=64, codebook_size=64, batch=1, k=0), parent=[-1], seed=33)
    g, par, nbr, tok = case.gpu_inputs(L)
    tree = L.Tree(case.parent)
    big = 65537                                      # batch * 1 node > capacity
    rows = g["target_cond"].expand(big, 1, 64)       # a view: stride 0 over the batch, no allocation
    out = dict(accept_len=torch.empty((big,), dtype=torch.int32, device="cuda"),
               out_tokens=torch.empty((big, 1), dtype=torch.int32, device="cuda"),
               out_nodes=torch.empty((big, 1), dtype=torch.int32, device="cuda"))
    tokens = torch.zeros((big, 1), dtype=torch.int32, device="cuda")
    with pytest.raises(L.LanternError) as e:
        L.verify_tree_static(par, tree, None, rows, None, rows, None, tokens, None, None, out=out)
    assert e.value.status == 2
