"""Seeded random inputs (torch generators; CPU or CUDA device).

Nothing here depends on the method: only Gaussian draws, uniform draws on the
24-bit grid and row copies.
"""

import torch

_DT = {"f32": torch.float32, "bf16": torch.bfloat16}


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_logits(cfg, step=0, device="cpu", batch=None):
    """Logit rows of one verify call.

    Returns a dict with target_cond, target_uncond, draft_cond, draft_uncond
    (the uncond entries are None without guidance), each [B][N][V] in
    cfg.dtype.  Drafter rows are draft_mix * (matching target row) plus
    Gaussian noise of std draft_noise, rounded to the storage type.
    """
    B = cfg.batch if batch is None else batch
    g = _gen(1000 * cfg.index + step, device)
    shape = (B, cfg.n_nodes, cfg.vocab)
    dt = _DT[cfg.dtype]
    out = {}
    names = ("cond", "uncond") if cfg.cfg_scale is not None else ("cond",)
    for nm in names:
        t = torch.randn(shape, generator=g, device=device, dtype=torch.float32) * cfg.logit_std
        d = t * cfg.draft_mix + torch.randn(shape, generator=g, device=device,
                                            dtype=torch.float32) * cfg.draft_noise
        out["target_" + nm] = t.to(dt)
        out["draft_" + nm] = d.to(dt)
    if cfg.cfg_scale is None:
        out["target_uncond"] = None
        out["draft_uncond"] = None
    return out


def make_codebook(L, d, dtype="f32", seed=0, dup_frac=0.0, device="cpu"):
    """L x d codebook ~ N(0,1); a fraction dup_frac of the rows is overwritten
    by exact copies of other (non-overwritten) rows."""
    g = _gen(seed, device)
    cb = torch.randn((L, d), generator=g, device=device, dtype=torch.float32).to(_DT[dtype])
    n_dup = int(round(L * dup_frac))
    if n_dup > 0:
        perm = torch.randperm(L, generator=g, device=device)
        dst = perm[:n_dup]
        src = perm[n_dup:][torch.randint(0, L - n_dup, (n_dup,), generator=g, device=device)]
        cb[dst] = cb[src]
    return cb.contiguous()


def make_uniforms(B, N, seed, device="cpu"):
    """(u_accept, u_resample), each [B][N] float32 on the grid i * 2^-24, i in [0, 2^24)."""
    g = _gen(seed, device)
    ua = torch.randint(0, 1 << 24, (B, N), generator=g, device=device).to(torch.float32) * (2.0 ** -24)
    ur = torch.randint(0, 1 << 24, (B, N), generator=g, device=device).to(torch.float32) * (2.0 ** -24)
    return ua, ur


def make_gumbel_uniforms(B, N, V, seed, device="cpu"):
    """[B][N][V] float32 uniforms in (0,1) on the grid (i + 0.5) * 2^-23 (exact in float32)."""
    g = _gen(seed, device)
    i = torch.randint(0, 1 << 23, (B, N, V), generator=g, device=device).to(torch.float32)
    return (i + 0.5) * (2.0 ** -23)


def random_sibling_tokens(parent, B, lo, hi, seed, device="cpu"):
    """[B][N] int32 tokens drawn uniformly from [lo, hi); siblings are made
    distinct by redrawing.  tokens[:, 0] (the root) is 0.  Used where a
    distribution-aware draft is not needed (large-size property tests)."""
    g = _gen(seed, device)
    N = len(parent)
    tok = torch.randint(lo, hi, (B, N), generator=g, device=device, dtype=torch.int32)
    tok[:, 0] = 0
    kids = {}
    for i in range(1, N):
        kids.setdefault(parent[i], []).append(i)
    for ch in kids.values():
        for a in range(1, len(ch)):
            for _ in range(8):
                clash = torch.zeros(B, dtype=torch.bool, device=device)
                for b_ in range(a):
                    clash |= tok[:, ch[a]] == tok[:, ch[b_]]
                if not bool(clash.any()):
                    break
                new = torch.randint(lo, hi, (B,), generator=g, device=device, dtype=torch.int32)
                tok[:, ch[a]] = torch.where(clash, new, tok[:, ch[a]])
    return tok


def random_neighbor_table(L, k, seed, device="cpu"):
    """[L][k] int32 table of k distinct indices != row per row, uniformly random.  A stand-in
    for a real neighbour table where only its shape matters (the synthetic logits carry no
    relation to codebook geometry)."""
    g = _gen(seed, device)
    # k distinct values of [0, L-1) per row via random keys, then skip over the row's own index
    keys = torch.rand((L, L - 1) if L <= 2048 else (L, min(L - 1, 8 * k)), generator=g, device=device)
    if keys.shape[1] == L - 1:
        idx = keys.argsort(dim=1)[:, :k]
    else:
        # large L: draw with replacement from a wide range and keep the first k distinct values
        cand = torch.randint(0, L - 1, (L, 8 * k), generator=g, device=device)
        idx = torch.empty((L, k), dtype=torch.int64, device=device)
        srt, order = cand.sort(dim=1, stable=True)
        first = torch.ones_like(srt, dtype=torch.bool)
        first[:, 1:] = srt[:, 1:] != srt[:, :-1]
        keep = torch.zeros_like(first)
        keep.scatter_(1, order, first)          # keep[r, c] = cand[r, c] is a first occurrence
        rank = keep.cumsum(dim=1) - 1
        sel = keep & (rank < k)
        assert bool((sel.sum(dim=1) == k).all())
        idx = cand[sel].view(L, k)
    rows = torch.arange(L, device=device).unsqueeze(1)
    idx = idx + (idx >= rows).to(idx.dtype)
    return idx.to(torch.int32).contiguous()
