"""Parity of lantern_build_neighbors with the oracle's brute force (Sec. 2.2 / Sec. 4: B_k)."""
import numpy as np
import pytest
import torch

import workloads as W
from parity_util import compare_neighbors

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    import paper_2502_06352_b200 as lib
    return lib


def _check(L, cb, k, rows=None):
    idx, dist = L.build_neighbors(cb.cuda(), k, return_dist=True)
    torch.cuda.synchronize()
    idx, dist = idx.cpu().numpy(), dist.cpu().numpy()
    cb64 = cb.to(torch.float64).numpy()
    n = cb.shape[0]
    rows = list(range(n)) if rows is None else rows
    ties = compare_neighbors(idx, dist, cb64, rows, k)
    assert ties == 0 or ties <= len(rows) // 1000
    return idx, dist


@pytest.mark.parametrize("n,d,k,dt", [(2, 1, 1, "f32"), (17, 3, 16, "f32"), (300, 8, 10, "f32"),
                                      (1000, 8, 50, "bf16"), (777, 64, 33, "bf16"), (600, 256, 200, "bf16"),
                                      (1500, 40, 700, "f32"), (64, 32, 63, "bf16"), (2000, 128, 320, "bf16"),
                                      (1000, 48, 321, "bf16"), (333, 256, 7, "bf16")])
def test_small_codebooks_all_rows(L, n, d, k, dt):
    cb = W.make_codebook(n, d, dt, seed=n + d, dup_frac=0.05 if n > 50 else 0.0)
    _check(L, cb, k)


def test_duplicates_tie_by_index_and_zero_distance(L):
    cb = W.make_codebook(64, 8, "bf16", seed=1)
    cb[10] = cb[3]
    cb[40] = cb[3]
    idx, dist = _check(L, cb, 5)
    assert list(idx[3][:2]) == [10, 40] and list(dist[3][:2]) == [0, 0]
    assert list(idx[10][:2]) == [3, 40] and list(idx[40][:2]) == [3, 10]


def test_tensor_path_margin_keeps_near_ties_exact(L):
    """bf16 rows that differ in one low-order entry: approximate distances nearly tie, the exact
    re-rank must still order them by true distance and then by index."""
    g = torch.Generator().manual_seed(3)
    base = (torch.randn((1, 64), generator=g) * 4).to(torch.bfloat16)
    cb = base.repeat(512, 1).contiguous()
    # row i differs from the base in entry (i % 64) by one bf16 step of that entry, sign by parity
    for i in range(1, 512):
        e = i % 64
        v = cb[i, e].float()
        step = 2.0 ** (torch.floor(torch.log2(v.abs())) - 7)
        cb[i, e] = (v + step * (1 if i % 2 else -1) * (1 + i // 128)).to(torch.bfloat16)
    _check(L, cb, 40)


def test_massive_ties_take_the_exact_fallback(L):
    # every row equal: all distances are 0, neighbours are the lowest indices
    cb = torch.ones((700, 4), dtype=torch.float32)
    idx, dist = _check(L, cb, 20)
    assert list(idx[0]) == list(range(1, 21)) and list(idx[5][:6]) == [0, 1, 2, 3, 4, 6]
    # integer line: closed-form neighbours
    cb = torch.arange(900, dtype=torch.float32)[:, None].contiguous()
    idx, _ = _check(L, cb, 4, rows=[0, 450, 899])
    assert list(idx[450]) == [449, 451, 448, 452]


@pytest.mark.parametrize("n,d,k,dt", [(16384, 8, 100, "f32"), (8192, 256, 200, "bf16")])
def test_config_codebooks_sampled_rows(L, n, d, k, dt):
    cb = W.make_codebook(n, d, dt, seed=5, dup_frac=0.05)
    rows = [0, 1, 2, n // 2, n - 1] + list(np.random.default_rng(0).integers(0, n, 20))
    idx, _ = _check(L, cb, k, rows=rows)
    # properties on every row: no self, distinct, in range
    assert not np.any(idx == np.arange(n)[:, None])
    s = np.sort(idx, axis=1)
    assert np.all(s[:, 1:] != s[:, :-1]) and idx.min() >= 0 and idx.max() < n


@pytest.mark.parametrize("n,d,k", [(65536, 64, 50), (65536, 256, 200), (65536, 8, 200)])
def test_sweep_largest_shapes_sampled_rows(L, n, d, k):
    """The largest codebooks of the table sweep (bf16, 5 % duplicate rows): sampled rows against
    the oracle, duplicates among them."""
    cb = W.make_codebook(n, d, "bf16", seed=6, dup_frac=0.05)
    rows = [0, n - 1] + list(np.random.default_rng(1).integers(0, n, 10))
    # rows that have an exact copy elsewhere (zero distance, tie by index)
    _, inv, cnt = np.unique(cb.view(torch.int16).numpy(), axis=0, return_inverse=True, return_counts=True)
    dup_rows = np.nonzero(cnt[inv.ravel()] > 1)[0]
    rows += [int(x) for x in dup_rows[:3]]
    _check(L, cb, k, rows=rows)


@pytest.mark.parametrize("n,d,k", [(8192, 8, 10), (8200, 24, 100), (8325, 48, 320), (9000, 80, 64), (8500, 128, 200),
                                   (16384, 8, 100)])
def test_tcgen05_kernel_ragged_tiles_sampled_rows(L, n, d, k):
    """Shapes served by the tcgen05 kernel (bf16, at least 8192 rows): a ragged last query and
    candidate tile (n not a multiple of 128), d below and between multiples of 16 (rows are
    zero-padded on chip), the smallest and the largest k of that kernel; rows of the first, an
    inner and the ragged last tile, and the -1 abort marker never appears."""
    cb = W.make_codebook(n, d, "bf16", seed=n + k, dup_frac=0.05)
    rng = np.random.default_rng(2)
    rows = [0, 127, 128, n - 1, n - 2, ((n - 1) // 128) * 128] + [int(x) for x in rng.integers(0, n, 12)]
    idx, _ = _check(L, cb, k, rows=rows)
    assert idx.min() >= 0 and idx.max() < n and not np.any(idx == np.arange(n)[:, None])
    s = np.sort(idx, axis=1)
    assert np.all(s[:, 1:] != s[:, :-1])


def test_tcgen05_kernel_overflowing_lists_take_the_exact_fallback(L):
    """A block of 1200 equal rows inside a large codebook: their lists hold more rows within the
    error margin than the exact ranking takes, so those queries go through the arg-min fallback;
    ties by index."""
    n, d, k = 8300, 32, 20
    cb = W.make_codebook(n, d, "bf16", seed=9)
    cb[1000:2200] = cb[1000]
    idx, dist = _check(L, cb, k, rows=[0, 999, 1000, 1001, 1500, 2199, 2200, n - 1])
    assert list(idx[1000]) == list(range(1001, 1021)) and list(idx[1500]) == list(range(1000, 1020))
    assert np.all(dist[1000:2200] == 0)


@pytest.mark.parametrize("n,d,k", [(8192, 16, 50), (9000, 40, 200)])
def test_tcgen05_and_brute_force_kernels_build_the_same_table(L, n, d, k):
    """Every row, not a sample: the same codebook as bfloat16 (tcgen05 kernel) and widened to float32 (exact
    brute-force kernel; the widening is exact) must give the same indices and the same distances, twice."""
    cb = W.make_codebook(n, d, "bf16", seed=n + d, dup_frac=0.05).cuda()
    i1, d1 = L.build_neighbors(cb, k, return_dist=True)
    i2, d2 = L.build_neighbors(cb.to(torch.float32), k, return_dist=True)
    i3, d3 = L.build_neighbors(cb, k, return_dist=True)
    torch.cuda.synchronize()
    assert torch.equal(i1, i3) and torch.equal(d1, d3)          # run to run
    assert torch.equal(i1, i2) and torch.equal(d1, d2)          # kernel to kernel


def test_outputs_stay_inside_their_extent(L):
    """Guard words before and after the table and the distance array (one allocation each) survive a build
    by the tcgen05 kernel (ragged last tile) and by the brute-force kernel."""
    import ctypes
    from paper_2502_06352_b200.binding import lib, _check
    for n, d, k, dt in ((8200, 24, 33, torch.bfloat16), (700, 5, 9, torch.float32)):
        cb = W.make_codebook(n, d, "bf16" if dt == torch.bfloat16 else "f32", seed=3).cuda()
        pad = 64
        gi = torch.full((n * k + 2 * pad,), 0x5a5a5a5a, dtype=torch.int32, device="cuda")
        gd = torch.full((n * k + 2 * pad,), -7.0, dtype=torch.float32, device="cuda")
        code = 1 if dt == torch.bfloat16 else 0
        wb = lib.lantern_build_neighbors_workspace(code, n, d, k)
        ws = torch.empty(max(wb, 256), dtype=torch.uint8, device="cuda")
        _check(lib.lantern_build_neighbors(ctypes.c_void_p(cb.data_ptr()), code, n, d, k,
                                           ctypes.c_void_p(gi.data_ptr() + 4 * pad), ctypes.c_void_p(gd.data_ptr() + 4 * pad),
                                           ctypes.c_void_p(ws.data_ptr()), ws.numel(),
                                           ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)), "lantern_build_neighbors")
        torch.cuda.synchronize()
        assert torch.all(gi[:pad] == 0x5a5a5a5a) and torch.all(gi[-pad:] == 0x5a5a5a5a)
        assert torch.all(gd[:pad] == -7.0) and torch.all(gd[-pad:] == -7.0)
        body = gi[pad:-pad].view(n, k)
        assert int(body.min()) >= 0 and int(body.max()) < n


def test_tcgen05_kernel_on_clustered_rows_with_many_near_ties(L):
    """64 tight clusters of about 130 rows (noise of a few bf16 steps, so many rows coincide after rounding):
    inside a cluster the approximate distances are nearly equal, the cut-backs work on keys that differ in their
    last bits only, and k reaches past the query's own cluster."""
    g = torch.Generator().manual_seed(12)
    n, d, k = 8320, 32, 150
    centres = torch.randn((64, d), generator=g) * 4
    cb = (centres[torch.arange(n) % 64] + torch.randn((n, d), generator=g) * 0.02).to(torch.bfloat16)
    rows = [0, 1, 63, 64, 4000, n - 1] + [int(x) for x in np.random.default_rng(3).integers(0, n, 10)]
    idx, _ = _check(L, cb, k, rows=rows)
    assert idx.min() >= 0 and idx.max() < n
    # the first 129 neighbours of a row lie in its own cluster (same index modulo 64)
    assert np.all(idx[:, :100] % 64 == (np.arange(n) % 64)[:, None])
