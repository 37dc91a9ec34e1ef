"""The shared library loads and exports every function that include/lantern.h declares; calls
that are rejected on the host before any CUDA work return their status codes."""
import ctypes
import os
import re

import paper_2502_06352_b200 as L

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "lantern.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lantern_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert {"lantern_build_neighbors", "lantern_sample_draft_tree", "lantern_verify_tree",
            "lantern_tree_create", "lantern_tree_destroy"} <= set(names)
    raw = ctypes.CDLL(L.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n


def test_host_side_rejections_need_no_gpu():
    assert L.lib.lantern_status_string(0) == b"ok"
    assert L.lib.lantern_build_neighbors(None, 0, 16, 4, 3, None, None, None, 0, None) == 1
    assert L.lib.lantern_build_neighbors(ctypes.c_void_p(256), 7, 16, 4, 3, ctypes.c_void_p(256), None, None, 0, None) == 1
    assert L.lib.lantern_build_neighbors(ctypes.c_void_p(256), 0, 16, 4, 16, ctypes.c_void_p(256), None, None, 0, None) == 1
    assert L.lib.lantern_build_neighbors(ctypes.c_void_p(256), 0, 4096, 5000, 3, ctypes.c_void_p(256), None, None, 0, None) == 2
    h = ctypes.c_void_p()
    bad = (ctypes.c_int32 * 3)(-1, 0, 2)
    assert L.lib.lantern_tree_create(bad, 3, ctypes.byref(h)) == 1          # parent[i] >= i
    bad = (ctypes.c_int32 * 4)(-1, 0, 1, 0)
    assert L.lib.lantern_tree_create(bad, 4, ctypes.byref(h)) == 1          # not breadth first
    wide = (ctypes.c_int32 * 10)(-1, *([0] * 9))
    assert L.lib.lantern_tree_create(wide, 10, ctypes.byref(h)) == 2        # fan-out 9
    assert L.lib.lantern_verify_tree(None, None, None, 0, None, None, None, None, 0, 0, 0, 0, None, None, None,
                                     None, None, None, None, None, None, None, None, None, 0, None) == 1
    assert L.lib.lantern_sample_draft_tree(None, None, None, None, 0, 0, 0, 0, 0, 0, None, None, None, None, None) == 1
    assert L.lib.lantern_verify_tree_workspace(None, 4) == 0
    assert L.set_cluster_size(3) == 0 and L.set_cluster_size(0) == 0        # 3 is refused


def test_neighbour_table_file_round_trip_and_checksums(tmp_path):
    """save_neighbors / load_neighbors (host utilities): bytes come back, a flipped entry or another codebook is refused."""
    import numpy as np
    import pytest
    import torch
    import paper_2502_06352_b200 as L
    g = torch.Generator().manual_seed(0)
    idx = torch.randint(0, 100, (100, 7), generator=g, dtype=torch.int32)
    cb = torch.randn((100, 4), generator=g)
    path = str(tmp_path / "table.npz")
    L.save_neighbors(path, idx, cb)
    back = L.load_neighbors(path, cb, device="cpu")
    assert torch.equal(back, idx)
    with pytest.raises(ValueError):
        L.load_neighbors(path, cb + 1.0, device="cpu")
    with np.load(path) as z:
        d = {k: z[k] for k in z.files}
    d["nbr_idx"] = d["nbr_idx"].copy()
    d["nbr_idx"][3, 2] ^= 1
    np.savez(path, **d)
    with pytest.raises(ValueError):
        L.load_neighbors(path, device="cpu")
