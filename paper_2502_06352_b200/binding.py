"""ctypes binding of include/lantern.h.  Same names, argument marshalling only.

Tensors are torch CUDA tensors (PyTorch supplies device memory and streams);
pointers, strides and the current stream are handed to the C ABI.
"""
import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblantern.so")

STATUS = {0: "ok", 1: "invalid argument", 2: "unsupported size", 3: "workspace", 4: "CUDA runtime error"}
DEV_BAD_INDEX, DEV_TIMEOUT, DEV_EMPTY_ROW = 1, 2, 4


class LanternError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, STATUS.get(status, "?"), status))


class _CParams(ctypes.Structure):
    _fields_ = [
        ("cfg_scale", ctypes.c_float), ("temperature", ctypes.c_float),
        ("top_k_target", ctypes.c_int32), ("top_k_draft", ctypes.c_int32),
        ("lam", ctypes.c_float), ("k", ctypes.c_int32), ("vocab", ctypes.c_int32),
        ("code_offset", ctypes.c_int32), ("n_codes", ctypes.c_int32),
        ("allowed_begin", ctypes.c_int32), ("allowed_end", ctypes.c_int32),
        ("seed", ctypes.c_uint64), ("step", ctypes.c_uint64),
        ("delta", ctypes.c_float), ("lazy_walk", ctypes.c_int32),
        ("subset_rule", ctypes.c_int32), ("draft_deterministic", ctypes.c_int32), ("kernels", ctypes.c_int32),
    ]


@dataclass
class Params:
    """Mirror of lantern_params (see include/lantern.h)."""
    vocab: int
    cfg_scale: float = 1.0
    temperature: float = 1.0
    top_k_target: int = 0
    top_k_draft: int = 0
    lam: float = 1.0
    k: int = 0
    code_offset: int = 0
    n_codes: int = 0
    allowed_begin: int = 0
    allowed_end: int = 0
    seed: int = 0
    step: int = 0
    delta: float = 0.0
    lazy_walk: int = 0
    subset_rule: int = 0
    draft_deterministic: int = 0
    kernels: int = 0

    def c(self):
        return _CParams(self.cfg_scale, self.temperature, self.top_k_target, self.top_k_draft,
                        self.lam, self.k, self.vocab, self.code_offset, self.n_codes,
                        self.allowed_begin, self.allowed_end, self.seed, self.step, self.delta, self.lazy_walk,
                        self.subset_rule, self.draft_deterministic, self.kernels)


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "liblantern.so is missing: build it with `python paper_2502_06352_b200/build.py` "
            "(needs nvcc; there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    L.lantern_status_string.restype = ctypes.c_char_p
    L.lantern_status_string.argtypes = [ctypes.c_int]
    L.lantern_tree_create.restype = ctypes.c_int
    L.lantern_tree_create.argtypes = [vp, i32, ctypes.POINTER(vp)]
    L.lantern_forest_create.restype = ctypes.c_int
    L.lantern_forest_create.argtypes = [vp, vp, i32, i32, ctypes.POINTER(vp)]
    L.lantern_tree_destroy.restype = ctypes.c_int
    L.lantern_tree_destroy.argtypes = [vp]
    L.lantern_tree_max_depth.restype = i32
    L.lantern_tree_max_depth.argtypes = [vp]
    L.lantern_build_neighbors_workspace.restype = sz
    L.lantern_build_neighbors_workspace.argtypes = [ctypes.c_int, i32, i32, i32]
    L.lantern_build_neighbors.restype = ctypes.c_int
    L.lantern_build_neighbors.argtypes = [vp, ctypes.c_int, i32, i32, i32, vp, vp, vp, sz, vp]
    L.lantern_sample_draft_tree.restype = ctypes.c_int
    L.lantern_sample_draft_tree.argtypes = [ctypes.POINTER(_CParams), vp, vp, vp, ctypes.c_int, i64, i64,
                                            i32, i32, i32, vp, vp, vp, vp, vp]
    L.lantern_verify_tree_workspace.restype = sz
    L.lantern_verify_tree_workspace.argtypes = [vp, i32]
    L.lantern_verify_tree.restype = ctypes.c_int
    L.lantern_verify_tree.argtypes = [ctypes.POINTER(_CParams), vp, vp, i32, vp, vp, vp, vp, ctypes.c_int,
                                      i64, i64, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.lantern_verify_tree_static.restype = ctypes.c_int
    L.lantern_verify_tree_static.argtypes = [ctypes.POINTER(_CParams), vp, vp, i32, vp, vp, vp, vp, ctypes.c_int,
                                             i64, i64, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.lantern_verify_tree_static_max_nodes.restype = i32
    L.lantern_verify_tree_static_max_nodes.argtypes = []
    L.lantern_philox_raw.restype = ctypes.c_int
    L.lantern_philox_raw.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                                     ctypes.c_uint32, i32, vp, vp]
    L.lantern_set_cluster_size.restype = i32
    L.lantern_set_cluster_size.argtypes = [i32]
    L.lantern_get_cluster_size.restype = i32
    L.lantern_get_cluster_size.argtypes = []
    L.lantern_verify_tree_path.restype = i32
    L.lantern_verify_tree_path.argtypes = [ctypes.POINTER(_CParams), vp, i32]
    L.lantern_sample_draft_tree_path.restype = i32
    L.lantern_sample_draft_tree_path.argtypes = [ctypes.POINTER(_CParams), vp, i32]
    L.lantern_expand_frontier.restype = ctypes.c_int
    L.lantern_expand_frontier.argtypes = [ctypes.POINTER(_CParams), vp, vp, ctypes.c_int, i64, i64, i32, i32, i32, i32,
                                          vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    L.lantern_trim_tree.restype = ctypes.c_int
    L.lantern_trim_tree.argtypes = [i32, i32, i32, i32, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]
    return L


lib = _load()


def _check(status, where):
    if status != 0:
        raise LanternError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t):
    if t.dtype == torch.float32:
        return 0
    if t.dtype == torch.bfloat16:
        return 1
    raise TypeError("logits / codebook must be float32 or bfloat16")


class Tree:
    """Static draft tree handle (lantern_tree_create / lantern_tree_destroy)."""

    def __init__(self, parent):
        self.parent = [int(x) for x in parent]
        self.n_nodes = len(self.parent)
        arr = (ctypes.c_int32 * self.n_nodes)(*self.parent)
        h = ctypes.c_void_p()
        _check(lib.lantern_tree_create(arr, self.n_nodes, ctypes.byref(h)), "lantern_tree_create")
        self.handle = h
        self.max_depth = lib.lantern_tree_max_depth(h)

    def __del__(self):
        h = getattr(self, "handle", None)
        if h is not None and lib is not None:
            lib.lantern_tree_destroy(h)
            self.handle = None


class Forest(Tree):
    """One tree per sequence, padded to max_nodes (lantern_forest_create); used like a Tree."""

    def __init__(self, parents, n_nodes, max_nodes=None):
        B = len(n_nodes)
        self.n_nodes = int(max_nodes if max_nodes is not None else max(int(n) for n in n_nodes))
        flat = []
        for b in range(B):
            row = [int(x) for x in parents[b][:int(n_nodes[b])]]
            flat += row + [-1] * (self.n_nodes - len(row))
        self.parent = flat
        arr = (ctypes.c_int32 * len(flat))(*flat)
        cnt = (ctypes.c_int32 * B)(*[int(n) for n in n_nodes])
        h = ctypes.c_void_p()
        _check(lib.lantern_forest_create(arr, cnt, B, self.n_nodes, ctypes.byref(h)), "lantern_forest_create")
        self.handle = h
        self.max_depth = lib.lantern_tree_max_depth(h)


def _rows(t: torch.Tensor, B, N, V):
    """(row_stride, seq_stride) in elements of a [B][N][V] tensor with unit inner stride."""
    if t.dim() != 3 or t.shape[0] != B or t.shape[1] != N or t.shape[2] != V or t.stride(2) != 1:
        raise ValueError("expected a [B][N][V] tensor with contiguous rows")
    return t.stride(1), t.stride(0)


def build_neighbors(codebook: torch.Tensor, k: int, return_dist=False):
    """lantern_build_neighbors: [L][k] int32 nearest-neighbour table of an [L][d] codebook."""
    if not codebook.is_cuda or not codebook.is_contiguous() or codebook.dim() != 2:
        raise ValueError("codebook must be a contiguous [L][d] CUDA tensor")
    L, d = codebook.shape
    idx = torch.empty((L, k), dtype=torch.int32, device=codebook.device)
    dist = torch.empty((L, k), dtype=torch.float32, device=codebook.device) if return_dist else None
    dt = _dtype_code(codebook)
    wbytes = lib.lantern_build_neighbors_workspace(dt, L, d, k)
    ws = torch.empty(max(wbytes, 256), dtype=torch.uint8, device=codebook.device)
    with torch.cuda.device(codebook.device):
        _check(lib.lantern_build_neighbors(_ptr(codebook), dt, L, d, k, _ptr(idx), _ptr(dist), _ptr(ws),
                                           ws.numel(), _stream()), "lantern_build_neighbors")
    return (idx, dist) if return_dist else idx


def save_neighbors(path: str, nbr_idx: torch.Tensor, codebook: torch.Tensor = None):
    """Writes a neighbour table ([L][k] int32) to `path` (numpy .npz) with a SHA-256 of its bytes and,
    if the codebook is given, of the codebook's bytes, so that a table is never paired with another codebook."""
    import hashlib
    import numpy as np
    t = nbr_idx.detach().cpu().contiguous().numpy().astype(np.int32)
    meta = {"table_sha256": hashlib.sha256(t.tobytes()).hexdigest()}
    if codebook is not None:
        cb = codebook.detach().cpu().contiguous()
        meta["codebook_sha256"] = hashlib.sha256(cb.view(torch.uint8).numpy().tobytes()).hexdigest()
    np.savez(path, nbr_idx=t, **{k: np.array(v) for k, v in meta.items()})


def load_neighbors(path: str, codebook: torch.Tensor = None, device="cuda"):
    """Reads a table written by save_neighbors; raises ValueError if the bytes do not match their checksum or
    (when a codebook is given and one was recorded) the table belongs to another codebook."""
    import hashlib
    import numpy as np
    with np.load(path) as z:
        t = np.ascontiguousarray(z["nbr_idx"], dtype=np.int32)
        if hashlib.sha256(t.tobytes()).hexdigest() != str(z["table_sha256"]):
            raise ValueError("neighbour table does not match its checksum: " + path)
        if codebook is not None and "codebook_sha256" in z.files:
            cb = codebook.detach().cpu().contiguous()
            if hashlib.sha256(cb.view(torch.uint8).numpy().tobytes()).hexdigest() != str(z["codebook_sha256"]):
                raise ValueError("neighbour table was built from another codebook: " + path)
    return torch.from_numpy(t).to(device)


def sample_draft_tree(params: Params, tree: Tree, draft_cond, draft_uncond=None, *, tokens=None,
                      parent_begin=0, parent_end=None, gumbel_uniforms=None, draft_prob=None,
                      device_status=None):
    """lantern_sample_draft_tree.  Returns tokens [B][N] int32 (allocated when not given)."""
    B, N, V = draft_cond.shape[0], tree.n_nodes, params.vocab
    rs, ss = _rows(draft_cond, B, N, V)
    if draft_uncond is not None and _rows(draft_uncond, B, N, V) != (rs, ss):
        raise ValueError("cond and uncond rows must share strides")
    if tokens is None:
        tokens = torch.full((B, N), -1, dtype=torch.int32, device=draft_cond.device)
    if gumbel_uniforms is not None and (not gumbel_uniforms.is_contiguous() or gumbel_uniforms.dtype != torch.float32
                                        or tuple(gumbel_uniforms.shape) != (B, N, V)):
        raise ValueError("gumbel_uniforms must be contiguous float32 [B][N][V]")
    cp = params.c()
    with torch.cuda.device(draft_cond.device):
        _check(lib.lantern_sample_draft_tree(
            ctypes.byref(cp), tree.handle, _ptr(draft_cond), _ptr(draft_uncond), _dtype_code(draft_cond), rs, ss,
            B, parent_begin, N if parent_end is None else parent_end, _ptr(gumbel_uniforms), _ptr(tokens),
            _ptr(draft_prob), _ptr(device_status), _stream()), "lantern_sample_draft_tree")
    return tokens


def verify_tree(params: Params, tree: Tree, nbr_idx, target_cond, target_uncond, draft_cond, draft_uncond,
                tokens, u_accept=None, u_resample=None, *, out=None, debug=False, device_status=None,
                workspace=None):
    """lantern_verify_tree.  Returns a dict of tensors: accept_len [B], out_tokens and
    out_nodes [B][max_depth+1]; with debug=True also node_next, node_token, node_mass,
    node_thresh [B][N].  `out` may carry preallocated tensors under the same names."""
    B, N, V = target_cond.shape[0], tree.n_nodes, params.vocab
    rs, ss = _rows(target_cond, B, N, V)
    for t in (target_uncond, draft_cond, draft_uncond):
        if t is not None and _rows(t, B, N, V) != (rs, ss):
            raise ValueError("all logit tensors must share strides")
    dev = target_cond.device
    out = {} if out is None else out
    D1 = tree.max_depth + 1

    def get(name, shape, dtype):
        if name not in out:
            out[name] = torch.empty(shape, dtype=dtype, device=dev)
        return out[name]

    accept_len = get("accept_len", (B,), torch.int32)
    out_tokens = get("out_tokens", (B, D1), torch.int32)
    out_nodes = get("out_nodes", (B, D1), torch.int32)
    node_next = node_token = node_mass = node_thresh = None
    if debug:
        node_next = get("node_next", (B, N), torch.int32)
        node_token = get("node_token", (B, N), torch.int32)
        node_mass = get("node_mass", (B, N), torch.float32)
        node_thresh = get("node_thresh", (B, N), torch.float32)
    if workspace is None:
        need = lib.lantern_verify_tree_workspace(tree.handle, B)
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    k_table = 0 if nbr_idx is None else nbr_idx.shape[1]
    cp = params.c()
    with torch.cuda.device(dev):
        _check(lib.lantern_verify_tree(
            ctypes.byref(cp), tree.handle, _ptr(nbr_idx), k_table, _ptr(target_cond), _ptr(target_uncond),
            _ptr(draft_cond), _ptr(draft_uncond), _dtype_code(target_cond), rs, ss, B, _ptr(tokens),
            _ptr(u_accept), _ptr(u_resample), _ptr(accept_len), _ptr(out_tokens), _ptr(out_nodes),
            _ptr(node_next), _ptr(node_token), _ptr(node_mass), _ptr(node_thresh), _ptr(device_status),
            _ptr(workspace), workspace.numel(), _stream()), "lantern_verify_tree")
    return out


def verify_tree_static(params: Params, tree: Tree, nbr_idx, target_cond, target_uncond, draft_cond, draft_uncond,
                       tokens, u_accept=None, u_resample=None, *, out, device_status=None):
    """lantern_verify_tree_static: verification for callers that cannot allocate.

    The library call allocates nothing; to keep this wrapper allocation-free as well, `out`
    must already hold accept_len [B], out_tokens and out_nodes [B][max_depth+1] (int32, on the
    logits' device).  batch * n_nodes may not exceed lantern_verify_tree_static_max_nodes().
    Calls share one built-in scratch array per GPU: do not let two of them overlap."""
    B, N, V = target_cond.shape[0], tree.n_nodes, params.vocab
    rs, ss = _rows(target_cond, B, N, V)
    for t in (target_uncond, draft_cond, draft_uncond):
        if t is not None and _rows(t, B, N, V) != (rs, ss):
            raise ValueError("all logit tensors must share strides")
    k_table = 0 if nbr_idx is None else nbr_idx.shape[1]
    cp = params.c()
    with torch.cuda.device(target_cond.device):
        _check(lib.lantern_verify_tree_static(
            ctypes.byref(cp), tree.handle, _ptr(nbr_idx), k_table, _ptr(target_cond), _ptr(target_uncond),
            _ptr(draft_cond), _ptr(draft_uncond), _dtype_code(target_cond), rs, ss, B, _ptr(tokens),
            _ptr(u_accept), _ptr(u_resample), _ptr(out["accept_len"]), _ptr(out["out_tokens"]),
            _ptr(out["out_nodes"]), _ptr(out.get("node_mass")), _ptr(out.get("node_thresh")),
            _ptr(device_status), _stream()), "lantern_verify_tree_static")
    return out


class DraftPool:
    """Candidate pool of dynamic-tree drafting: [B][P] parent / token / depth (int32) and log V
    (float64) with entry 0 the root, plus the current frontier [B][F] of pool indices."""

    def __init__(self, batch, n_depths, n_children, n_expand, device="cuda"):
        self.B, self.K, self.E = batch, n_children, n_expand
        # depth 1 expands the root alone, every later depth the n_expand chosen candidates
        self.P = 1 + n_children + max(0, n_depths - 1) * n_expand * n_children
        self.parent = torch.full((batch, self.P), -1, dtype=torch.int32, device=device)
        self.token = torch.full((batch, self.P), -1, dtype=torch.int32, device=device)
        self.depth = torch.zeros((batch, self.P), dtype=torch.int32, device=device)
        self.logv = torch.full((batch, self.P), float("-inf"), dtype=torch.float64, device=device)
        self.logv[:, 0] = 0.0
        self.frontier = torch.zeros((batch, 1), dtype=torch.int32, device=device)
        self.used, self.n_depths = 1, 0


def expand_frontier(params: Params, pool: DraftPool, draft_cond, draft_uncond=None):
    """lantern_expand_frontier: one depth of dynamic-tree drafting.  draft_cond [B][F][V] holds the
    drafter rows of the nodes in pool.frontier (F = its width).  The pool and its frontier advance."""
    B, F, V = pool.B, pool.frontier.shape[1], params.vocab
    rs, ss = _rows(draft_cond, B, F, V)
    if draft_uncond is not None and _rows(draft_uncond, B, F, V) != (rs, ss):
        raise ValueError("cond and uncond rows must share strides")
    nxt = torch.empty((B, pool.E), dtype=torch.int32, device=draft_cond.device)
    cp = params.c()
    with torch.cuda.device(draft_cond.device):
        _check(lib.lantern_expand_frontier(
            ctypes.byref(cp), _ptr(draft_cond), _ptr(draft_uncond), _dtype_code(draft_cond), rs, ss, B, F, pool.K, pool.E,
            _ptr(pool.frontier), pool.P, pool.used, pool.n_depths + 1, _ptr(pool.parent), _ptr(pool.token),
            _ptr(pool.logv), _ptr(pool.depth), _ptr(nxt), _stream()), "lantern_expand_frontier")
    pool.used += F * pool.K
    pool.n_depths += 1
    pool.frontier = nxt
    return nxt


def trim_tree(pool: DraftPool, max_nodes: int):
    """lantern_trim_tree: (n_nodes [B], parent, token, pool_index [B][max_nodes] int32, logv float64)."""
    dev = pool.parent.device
    n = torch.empty((pool.B,), dtype=torch.int32, device=dev)
    parent = torch.empty((pool.B, max_nodes), dtype=torch.int32, device=dev)
    token = torch.empty_like(parent)
    index = torch.empty_like(parent)
    logv = torch.empty((pool.B, max_nodes), dtype=torch.float64, device=dev)
    with torch.cuda.device(dev):
        _check(lib.lantern_trim_tree(pool.B, pool.P, pool.used, pool.n_depths, _ptr(pool.parent), _ptr(pool.token),
                                     _ptr(pool.logv), _ptr(pool.depth), max_nodes, _ptr(n), _ptr(parent), _ptr(token),
                                     _ptr(index), _ptr(logv), _stream()), "lantern_trim_tree")
    return n, parent, token, index, logv


def philox_raw(seed, first, c1, c2, c3, n, device="cuda"):
    """lantern_philox_raw: [n][4] raw Philox-4x32-10 words as int64 (values < 2^32)."""
    out = torch.empty((n, 4), dtype=torch.int32, device=device)
    with torch.cuda.device(out.device):
        _check(lib.lantern_philox_raw(seed, first, c1, c2, c3, n, _ptr(out), _stream()), "lantern_philox_raw")
    return out.to(torch.int64) & 0xFFFFFFFF


def verify_tree_path(params: "Params", tree: "Tree", batch: int) -> int:
    """lantern_verify_tree_path: 0 = dense kernels, 1 = list-based kernels + repair launch,
    2 = streaming kernel (rows without top-k)."""
    cp = params.c()
    return lib.lantern_verify_tree_path(ctypes.byref(cp), tree.handle, batch)


def sample_draft_tree_path(params: "Params", tree: "Tree", batch: int) -> int:
    """lantern_sample_draft_tree_path: 0 = dense kernel, 1 = list-based kernel + repair launch,
    2 = streaming kernel (rows without top-k)."""
    cp = params.c()
    return lib.lantern_sample_draft_tree_path(ctypes.byref(cp), tree.handle, batch)


def set_cluster_size(ctas_per_row: int) -> int:
    """lantern_set_cluster_size: 0 = automatic; returns the previous value."""
    return lib.lantern_set_cluster_size(ctas_per_row)
