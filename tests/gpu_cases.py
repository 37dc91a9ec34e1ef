"""Builds one verify/sampler test case on the CPU (inputs + oracle results)."""
import dataclasses

import numpy as np
import torch

import oracle
import workloads as W


def small_config(**kw):
    base = dict(name="case", index=9, batch=2, n_nodes=26, vocab=1000, dtype="f32", cfg_scale=3.0,
                temperature=1.0, top_k=0, logit_std=1.5, draft_mix=1.0, draft_noise=0.5,
                codebook_size=1000, codebook_dim=4, codebook_dtype="f32", code_offset=0, k=8, lam=3.0, steps=1)
    base.update(kw)
    return W.WorkloadConfig(**base)


def f64(t):
    return None if t is None else t.to(torch.float32).numpy()


class Case:
    """Inputs of one call (CPU tensors) and everything the oracle says about them."""

    def __init__(self, cfg, parent=None, seed=0, allowed=(0, 0), k_table=None, temperature=None,
                 top_k_target=None, top_k_draft=None, pad=0, oracle_seqs=None, tokens="oracle", delta=0.0,
                 library_table=False, skip=False, det_draft=False, kernels=1):
        self.cfg = cfg
        self.kernels = kernels      # lantern_params.kernels: 1 = streaming kernels wherever they apply (tests are small)
        self.parent = W.static_tree(cfg.n_nodes) if parent is None else parent
        N, B, V = len(self.parent), cfg.batch, cfg.vocab
        self.N, self.B, self.V = N, B, V
        self.padded = W.make_logits(dataclasses.replace(cfg, n_nodes=N, vocab=V + pad), step=seed)
        self.logits = {k: (None if v is None else v[:, :, :V]) for k, v in self.padded.items()}
        cb = W.make_codebook(cfg.codebook_size, cfg.codebook_dim, cfg.codebook_dtype, seed=77 + seed)
        self.codebook = cb
        self.k_table = cfg.k if k_table is None else k_table
        self.nbr = None
        if self.k_table > 0 and cfg.codebook_size <= 2048:
            self.nbr, _ = oracle.neighbor_table(cb.to(torch.float64).numpy(), self.k_table)
        elif self.k_table > 0:      # large tables: only the shape matters to the verifier
            self.nbr = W.random_neighbor_table(cfg.codebook_size, self.k_table, 55 + seed).numpy()
        self.u_accept, self.u_resample = W.make_uniforms(B, N, 500 + seed)
        self.params = dict(
            cfg_scale=cfg.cfg_scale if cfg.cfg_scale is not None else 1.0,
            temperature=cfg.temperature if temperature is None else temperature,
            top_k_target=cfg.top_k if top_k_target is None else top_k_target,
            top_k_draft=cfg.top_k if top_k_draft is None else top_k_draft,
            lam=cfg.lam, k=cfg.k, code_offset=cfg.code_offset, n_codes=cfg.codebook_size,
            allowed_begin=allowed[0], allowed_end=allowed[1] if allowed[1] else V, delta=delta,
            skip=skip, det_draft=det_draft)
        self.seqs = list(range(B)) if oracle_seqs is None else list(oracle_seqs)
        # draft tokens: oracle sampler on the checked sequences, uniform random elsewhere
        lo, hi = self.params["allowed_begin"], self.params["allowed_end"]
        tok = W.random_sibling_tokens(self.parent, B, lo, hi, 900 + seed).numpy().astype(np.int64)
        self.gumbel = None
        if tokens == "oracle":
            self.gumbel = W.make_gumbel_uniforms(len(self.seqs), N, V, 300 + seed)
            for i, b in enumerate(self.seqs):
                t, _ = oracle.sample_draft_tree(
                    self.parent, f64(self.logits["draft_cond"][b]), f64(self.logits["draft_uncond"][b])
                    if self.logits["draft_uncond"] is not None else None, self.gumbel[i].numpy(),
                    **self._sampler_kw())
                tok[b, 1:] = t[1:]
        self.tokens = tok
        self._orc = None
        # library_table: the device side verifies with the table lantern_build_neighbors makes of
        # the codebook; the oracle gets its own brute-force rows for the codes the checked
        # sequences draft (the other rows are never read)
        self.library_table = library_table
        if library_table:
            codes = sorted({int(t) - cfg.code_offset for b in self.seqs for t in tok[b, 1:]
                            if 0 <= int(t) - cfg.code_offset < cfg.codebook_size})
            rows, _ = oracle.neighbor_table(cb.to(torch.float64).numpy(), self.k_table, rows=codes)
            self.nbr = np.zeros((cfg.codebook_size, self.k_table), dtype=np.int32)
            self.nbr[codes] = rows

    def _sampler_kw(self):
        p = self.params
        return dict(cfg_scale=p["cfg_scale"], temperature=p["temperature"], top_k_draft=p["top_k_draft"],
                    allowed_begin=p["allowed_begin"], allowed_end=p["allowed_end"])

    def oracle_verify(self):
        if self._orc is None:
            lg = self.logits
            self._orc = []
            for b in self.seqs:
                self._orc.append(oracle.verify_sequence(
                    self.parent, f64(lg["target_cond"][b]),
                    None if lg["target_uncond"] is None else f64(lg["target_uncond"][b]),
                    f64(lg["draft_cond"][b]),
                    None if lg["draft_uncond"] is None else f64(lg["draft_uncond"][b]),
                    self.tokens[b], self.u_accept[b].numpy(), self.u_resample[b].numpy(), self.nbr,
                    **self.params))
        return self._orc

    def oracle_node(self, b, n, forced):
        """oracle.verify_node of node n of sequence b with decisions imposed (near-tie rule)."""
        lg, p = self.logits, self.params
        children = oracle.tree_children(self.parent)
        row = lambda t: None if t is None else f64(t[b][n])
        q, _ = oracle.postprocess_row(row(lg["target_cond"]), row(lg["target_uncond"]), p["cfg_scale"], p["temperature"],
                                      p["top_k_target"], p["allowed_begin"], p["allowed_end"])
        pd = None
        if children[n]:
            pd, _ = oracle.postprocess_row(row(lg["draft_cond"]), row(lg["draft_uncond"]), p["cfg_scale"],
                                           p["temperature"], p["top_k_draft"], p["allowed_begin"], p["allowed_end"])
        return oracle.verify_node(q, pd, children[n], self.tokens[b], self.u_accept[b].numpy(),
                                  self.u_resample[b].numpy()[n], self.nbr, p["k"], p["lam"], p["code_offset"],
                                  p["n_codes"], p["delta"], forced=forced, skip=p["skip"], det_draft=p["det_draft"])

    # ---- device side
    def gpu_inputs(self, L):
        dev = "cuda"
        g = {k: (None if v is None else v.to(dev)[:, :, :self.V]) for k, v in self.padded.items()}   # padded stride kept
        p = self.params
        par = L.Params(vocab=self.V, cfg_scale=p["cfg_scale"], temperature=p["temperature"],
                       top_k_target=p["top_k_target"], top_k_draft=p["top_k_draft"], lam=p["lam"], k=p["k"],
                       code_offset=p["code_offset"], n_codes=p["n_codes"], allowed_begin=p["allowed_begin"],
                       allowed_end=p["allowed_end"], delta=p["delta"], subset_rule=int(p["skip"]),
                       draft_deterministic=int(p["det_draft"]), kernels=self.kernels)
        nbr = None if self.nbr is None else torch.from_numpy(self.nbr).to(dev)
        if self.library_table:
            nbr = L.build_neighbors(self.codebook.to(dev), self.k_table)
        tok = torch.from_numpy(self.tokens.astype(np.int32)).to(dev)
        return g, par, nbr, tok

    def gpu_verify(self, L, use_philox=None):
        g, par, nbr, tok = self.gpu_inputs(L)
        tree = L.Tree(self.parent)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        ua = ur = None
        if use_philox is None:
            ua, ur = self.u_accept.cuda(), self.u_resample.cuda()
        else:
            par.seed, par.step = use_philox
        out = L.verify_tree(par, tree, nbr, g["target_cond"], g["target_uncond"], g["draft_cond"],
                            g["draft_uncond"], tok, ua, ur, debug=True, device_status=status)
        torch.cuda.synchronize()
        res = {k: v.cpu().numpy() for k, v in out.items()}
        res["status"] = int(status.item())
        res["max_depth"] = tree.max_depth
        return res
