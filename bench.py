"""Benchmark of the relaxed tree-verification hot path.

One step = one pass of the path over one batch of synthetic input: the draft sampler over
every internal node, then the relaxed verification of every node and the walk.  The
neighbour table is built once per codebook and is timed separately.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints one JSON line (rank 0).  The headline numbers (value, roofline, e2e, cpu_baseline) are
those of --workload (default: the largest single-GPU configuration, c4_batch64); the `configs`
object of the same line carries the verify / sampler timings and roofline fractions of every
other configuration (c1..c3, c3 restricted to its image tokens, and the neighbour-table sweep).
Under torchrun every rank verifies its own batch of sequences (no data-path collective); the
value is all ranks' nodes over the slowest rank's device time.
"""
import argparse
import dataclasses
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verified tree nodes/sec"
UNIT = "nodes/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
MIN_TIMED_MS = 50.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c4_batch64")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (sequences per call); 0 = as configured")
    ap.add_argument("--ring", type=int, default=0, help="input buffer sets cycled through (0 = enough to exceed L2)")
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--configs", default="all", choices=["all", "none"],
                    help="all: also time the other configurations and report them under `configs`")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of CUDA-graph replays")
    ap.add_argument("--walk", default="eager", choices=["eager", "lazy"],
                    help="eager: verify every tree node, then walk (the configuration the metric is quoted on); "
                         "lazy: verify only the nodes on each sequence's accepted path (params.lazy_walk)")
    return ap.parse_args()


def algorithmic_bytes(cfg, parent, batch, allowed=None):
    """(verify bytes, sampler bytes) one call must move: every target row and every internal
    node's drafter row once (only the allowed slice of a row when the tokens are restricted),
    the neighbour rows of the draft tokens, and the per-node inputs / outputs."""
    N = len(parent)
    I = len(set(parent[1:]))
    c = 2 if cfg.cfg_scale is not None else 1
    e = 4 if cfg.dtype == "f32" else 2
    width = cfg.vocab if allowed is None else allowed[1] - allowed[0]
    rows = batch * (N + I) * c * width * e
    table = batch * (N - 1) * cfg.k * 4
    outs = batch * N * (4 + 4 + 4 + 4 + 4)      # tokens, two uniforms in; next, token out
    return rows + table + outs, batch * I * c * width * e


# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu
# capture summarised under profiles/ (taken on a smaller batch and scaled by the number of rows,
# as stated there); valid only for the kernel source it was taken from
TRAFFIC = {"c4_batch64": {"kernel_sha256": "74a92df7271d5105", "bytes": 1321464832},
           "c2_llamagen512": {"kernel_sha256": "74a92df7271d5105", "bytes": 104124160}}


def kernel_sha256():
    import hashlib
    h = hashlib.sha256()
    for f in ("verify_stream.cuh", "verify_sparse.cuh", "verify_kernel.cuh", "verify_launch.cuh", "verify.cu",
              "rowops.cuh", "common.cuh"):
        with open(os.path.join(ROOT, "paper_2502_06352_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def measured_traffic(workload):
    t = TRAFFIC.get(workload)
    if not t or t["bytes"] is None or t["kernel_sha256"] != kernel_sha256():
        return None
    return t["bytes"]


def peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle samples of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        sm.sort()
        # the busy half of the samples (the tool also samples before and after the region)
        busy = sm[len(sm) // 2:] if sm else []
        return {"sm_mhz": busy[len(busy) // 2] if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle baseline (the reference arm and the cpu_baseline leg)

def oracle_step_inputs(cfg, parent, n_seqs, seed):
    import workloads as W
    N, V = len(parent), cfg.vocab
    gum = W.make_gumbel_uniforms(n_seqs, N, V, seed).numpy()
    ua, ur = W.make_uniforms(n_seqs, N, seed + 1)
    nbr = W.random_neighbor_table(cfg.codebook_size, cfg.k, seed + 2).numpy()
    return gum, ua.numpy(), ur.numpy(), nbr


def oracle_run_nodes(cfg, parent, lg, b, gum, ua, ur, nbr, n_nodes):
    """Oracle sampler + verifier on the first n_nodes nodes of sequence b (bounded sample)."""
    import oracle
    f = lambda t: None if t is None else t[b].float().numpy()
    kw = dict(cfg_scale=cfg.cfg_scale if cfg.cfg_scale is not None else 1.0, temperature=cfg.temperature)
    tc, tu, dc, du = f(lg["target_cond"]), f(lg["target_uncond"]), f(lg["draft_cond"]), f(lg["draft_uncond"])
    children = oracle.tree_children(parent)
    tokens, _ = oracle.sample_draft_tree(parent, dc, du, gum, top_k_draft=cfg.top_k, **kw)
    tokens[0] = 0
    done = 0
    for n in range(min(n_nodes, len(parent))):
        q, _ = oracle.postprocess_row(tc[n], None if tu is None else tu[n], kw["cfg_scale"], cfg.temperature, cfg.top_k)
        p = None
        if children[n]:
            p, _ = oracle.postprocess_row(dc[n], None if du is None else du[n], kw["cfg_scale"], cfg.temperature, cfg.top_k)
        oracle.verify_node(q, p, children[n], tokens, ua, ur[n], nbr, cfg.k, cfg.lam, cfg.code_offset, cfg.codebook_size)
        done += 1
    return done


def _oracle_worker(job):
    """One process of the all-cores baseline: whole sequences of the workload (its own seeded
    inputs) until the time budget is spent.  Returns (nodes, seconds)."""
    name, worker, budget_s = job
    import torch
    torch.set_num_threads(1)
    import workloads as W
    cfg = W.CONFIGS[name]
    parent = W.static_tree(cfg.n_nodes)
    lg = W.make_logits(cfg, step=7000 + worker, device="cpu", batch=1)
    gum, ua, ur, nbr = oracle_step_inputs(cfg, parent, 1, 4242 + worker)
    t0 = time.perf_counter()
    nodes = 0
    while True:
        nodes += oracle_run_nodes(cfg, parent, lg, 0, gum[0], ua[0], ur[0], nbr, len(parent))
        if time.perf_counter() - t0 > budget_s:
            break
    return nodes, time.perf_counter() - t0


def cpu_baseline(cfg, parent, budget_s=10.0):
    """The oracle, as it stands, on whole sequences of the workload: one process for about
    budget_s, then one process per host core for about budget_s (each on its own sequence)."""
    import multiprocessing as mp
    n1, t1 = _oracle_worker((cfg.name, 0, budget_s))
    cores = os.cpu_count() or 1
    value_all, used = None, 1
    if cores > 1:
        try:
            ctx = mp.get_context("spawn")
            with ctx.Pool(cores) as pool:
                res = pool.map(_oracle_worker, [(cfg.name, w, budget_s) for w in range(cores)])
            value_all = sum(n / t for n, t in res)
            used = cores
        except Exception as exc:          # no process pool on this host: the one-core figure stands
            sys.stderr.write("all-cores oracle baseline not run: %r\n" % (exc,))
    value = value_all if value_all is not None else n1 / t1
    return {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "value_one_core": n1 / t1,
            "sample": "whole sequences of %s (draft sampling + relaxed verification of every node), about %.0f s "
                      "per process; one process: %d nodes in %.1f s; %d processes, one sequence each, run "
                      "together" % (cfg.name, budget_s, n1, t1, used)}


def parity_sample(L, W, cfg, parent, lg, nbr, seq_ids):
    """Near-tie accounting on the benchmarked workload (part of the CPU-baseline leg: it runs the
    oracle): a few sequences of one input set go through the same kernels with explicit uniforms
    and are compared with the oracle under the near-tie rule.  Returns the counts per class."""
    import numpy as np
    import torch
    import oracle
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from parity_util import KEY_TIE, check_walk, compare_verify
    N, V, n = len(parent), cfg.vocab, len(seq_ids)
    dev = lg["target_cond"].device
    idx = torch.tensor(seq_ids, device=dev)
    sub = {k: (None if v is None else v.index_select(0, idx).contiguous()) for k, v in lg.items()}
    cpu = {k: (None if v is None else v.float().cpu().numpy()) for k, v in sub.items()}
    gum = W.make_gumbel_uniforms(n, N, V, 777)
    ua, ur = W.make_uniforms(n, N, 778)
    tree = L.Tree(parent)
    par = L.Params(vocab=V, cfg_scale=cfg.cfg_scale if cfg.cfg_scale is not None else 1.0, temperature=cfg.temperature,
                   top_k_target=cfg.top_k, top_k_draft=cfg.top_k, lam=cfg.lam, k=cfg.k, code_offset=cfg.code_offset,
                   n_codes=cfg.codebook_size, kernels=1)
    tok = L.sample_draft_tree(par, tree, sub["draft_cond"], sub["draft_uncond"], gumbel_uniforms=gum.to(dev))
    res = L.verify_tree(par, tree, nbr, sub["target_cond"], sub["target_uncond"], sub["draft_cond"], sub["draft_uncond"],
                        tok, ua.to(dev), ur.to(dev), debug=True)
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in res.items()}
    gtok = tok.cpu().numpy()
    nbr_np = nbr.cpu().numpy()
    kw = dict(cfg_scale=par.cfg_scale, temperature=cfg.temperature)
    vkw = dict(top_k_target=cfg.top_k, top_k_draft=cfg.top_k, lam=cfg.lam, k=cfg.k, code_offset=cfg.code_offset,
               n_codes=cfg.codebook_size, **kw)
    children = oracle.tree_children(parent)
    sampler_ties, orc = 0, []
    for i in range(n):
        g = lambda name: None if cpu[name] is None else cpu[name][i]
        otok, _ = oracle.sample_draft_tree(parent, g("draft_cond"), g("draft_uncond"), gum[i].numpy(),
                                           top_k_draft=cfg.top_k, **kw)
        for node in range(N):
            kids = children[node]
            if kids and [int(gtok[i, c]) for c in kids] != [int(otok[c]) for c in kids]:
                p_row, _ = oracle.postprocess_row(g("draft_cond")[node], None if g("draft_uncond") is None else g("draft_uncond")[node],
                                                  kw["cfg_scale"], cfg.temperature, cfg.top_k)
                _, _, gaps = oracle.sample_children(p_row, gum[i][node].numpy(), len(kids), return_gaps=True)
                if min(gaps) >= KEY_TIE:
                    raise AssertionError(("draft sampler differs from the oracle", seq_ids[i], node))
                sampler_ties += 1
        # the verifier is compared on the device's drafts (they are the oracle's unless a key near-tie was counted)
        orc.append(oracle.verify_sequence(parent, g("target_cond"), g("target_uncond"), g("draft_cond"), g("draft_uncond"),
                                          gtok[i].astype(np.int64), ua[i].numpy(), ur[i].numpy(), nbr_np, **vkw))

    def rerun(b, node, forced):
        g = lambda name: None if cpu[name] is None else cpu[name][b][node]
        q, _ = oracle.postprocess_row(g("target_cond"), g("target_uncond"), kw["cfg_scale"], cfg.temperature, cfg.top_k)
        pd = None
        if children[node]:
            pd, _ = oracle.postprocess_row(g("draft_cond"), g("draft_uncond"), kw["cfg_scale"], cfg.temperature, cfg.top_k)
        return oracle.verify_node(q, pd, children[node], gtok[b].astype(np.int64), ua[b].numpy(), ur[b].numpy()[node], nbr_np,
                                  cfg.k, cfg.lam, cfg.code_offset, cfg.codebook_size, forced=forced)

    stats = compare_verify(res, orc, parent, ua.numpy(), rerun=rerun)
    check_walk(res, gtok, tree.max_depth, orc, stats["dirty_sequences"], None, stats["patched"])
    return {"sequences": n, "nodes": stats["nodes"], "tested_children": stats["tested"], "tie_accept": stats["tie_accept"],
            "tie_cut": stats["tie_cut"], "tie_resample": stats["tie_resample"], "tie_sampler_key": sampler_ties,
            "rule": "integers exact; a difference counts as a tie only where the oracle's margin is below 1e-6"}


def run_reference(args, cfg, parent):
    """--impl reference: the CPU oracle on bounded samples of the same workload."""
    import workloads as W
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    N = len(parent)
    lg = W.make_logits(cfg, step=0, device="cpu", batch=1)
    gum, ua, ur, nbr = oracle_step_inputs(cfg, parent, 1, 4242)
    t0 = time.perf_counter()
    oracle_run_nodes(cfg, parent, lg, 0, gum[0], ua[0], ur[0], nbr, 4)
    t_node = (time.perf_counter() - t0) / 4
    per_step = int(max(1, min(N, 120.0 / (max(1, args.steps + args.warmup) * t_node))))
    for _ in range(args.warmup):
        oracle_run_nodes(cfg, parent, lg, 0, gum[0], ua[0], ur[0], nbr, per_step)
    t0 = time.perf_counter()
    nodes = 0
    for _ in range(args.steps):
        nodes += oracle_run_nodes(cfg, parent, lg, 0, gum[0], ua[0], ur[0], nbr, per_step)
    dt = time.perf_counter() - t0
    val = nodes / dt
    sample = "each step: draft sampling of one sequence + relaxed verification of its first %d of %d nodes" % (per_step, N)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": 1, "tree_nodes": N, "vocab": cfg.vocab, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ------------------------------------------------------------------------------------------------
# neighbour-table sweep (config 5)

def table_sweep(with_oracle):
    """Every (L, d, k) neighbour-table build of the sweep, timed with CUDA events (best of 3 after
    a warm-up); with_oracle also times the oracle on a few rows of each shape."""
    import torch
    import workloads as W
    from workloads.configs import SWEEP_L, SWEEP_D, SWEEP_K, SWEEP_DUP_FRAC
    import paper_2502_06352_b200 as L
    rows = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for n in SWEEP_L:
        for d in SWEEP_D:
            cb = W.make_codebook(n, d, "bf16", seed=5, dup_frac=SWEEP_DUP_FRAC, device="cuda")
            t_or = None
            if with_oracle:
                import oracle
                cb64 = cb.cpu().to(torch.float64).numpy()
                t0 = time.perf_counter()
                oracle.neighbor_table(cb64, max(SWEEP_K), rows=list(range(0, n, max(1, n // 8)))[:8])
                t_or = (time.perf_counter() - t0) / 8          # seconds per query row
            for k in SWEEP_K:
                L.build_neighbors(cb, k)
                best = None
                for _ in range(3):
                    ev0.record()
                    L.build_neighbors(cb, k)
                    ev1.record()
                    torch.cuda.synchronize()
                    ms = ev0.elapsed_time(ev1)
                    best = ms if best is None else min(best, ms)
                alg = n * d * 2 + n * k * 4
                rows.append({"L": n, "d": d, "k": k, "ms": round(best, 3), "rows_per_s": n / (best * 1e-3),
                             "gbs": alg / (best * 1e-3) / 1e9, "contraction_tflops": 2.0 * n * n * d / (best * 1e-3) / 1e12,
                             "candidates_per_s": float(n) * n / (best * 1e-3),
                             "path": ("tcgen05" if (n >= 8192 and d % 8 == 0 and d <= 256 and k <= 320)
                                      else "mma.sync" if (d % 16 == 0 and 32 <= d <= 256 and k <= 320) else "brute"),
                             "oracle_rows_per_s": None if t_or is None else 1.0 / t_or})
    return rows, SWEEP_DUP_FRAC


def run_table_sweep(args):
    """--workload c5_table_sweep: the sweep as the headline of its own JSON line."""
    import torch
    torch.cuda.set_device(0)
    rows, dup = table_sweep(not args.no_cpu_baseline)
    total_rows = sum(r["L"] for r in rows)
    total_ms = sum(r["ms"] for r in rows)
    print(json.dumps({"metric": "neighbour-table rows/sec", "value": total_rows / (total_ms * 1e-3), "unit": "rows/s",
                      "n_gpus": 1, "steps": 3, "warmup": 1, "ms_per_step": total_ms, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "bf16 mma + f64 re-rank", "data": "synthetic",
                      "config": {"workload": "c5_table_sweep", "dup_frac": dup}, "builds": rows,
                      "gpu_launches": 4 * 2 * len(rows)}))


def run_dynamic_tree(args):
    """--workload f3_dynamic_tree: dynamic-tree drafting as the headline of its own JSON line."""
    import torch
    import paper_2502_06352_b200 as L
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    peak, peak_kind = peak_hbm()
    ent = dynamic_tree_entry(torch, L, dev, peak)
    rows = 64 * (1 + 5 * 8)
    print(json.dumps({"metric": "drafter rows expanded/sec", "value": rows / (ent["us_median"] * 1e-6), "unit": "rows/s",
                      "n_gpus": 1, "steps": 20, "warmup": 3, "ms_per_step": ent["us_median"] * 1e-3, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "f32 (log V in f64)", "data": "synthetic",
                      "config": {"workload": ent["workload"]}, "roofline": {"bound": "hbm", "achieved": ent["gbs"], "peak": peak,
                      "unit": "GB/s", "frac": ent["frac_measured"], "peak_kind": peak_kind, "traffic": None,
                      "kernel": ent["kernels"]}, "gpu_launches": ent["launches"] * 20, "detail": ent}))


# ------------------------------------------------------------------------------------------------
# one configuration on the device

class Workload:
    """Inputs of one configuration resident on the device: a ring of step buffers larger than
    L2, the neighbour table, parameters and output buffers; step / verify / sampler calls."""

    def __init__(self, L, W, cfg, dev, rank=0, ring=0, allowed=None, walk="eager", build_table=True, max_ring_bytes=40e9):
        import torch
        self.L, self.cfg, self.dev, self.allowed = L, cfg, dev, allowed
        self.parent = W.static_tree(cfg.n_nodes)
        self.N, self.B, self.V = len(self.parent), cfg.batch, cfg.vocab
        self.tree = L.Tree(self.parent)
        n_ops = 4 if cfg.cfg_scale is not None else 2
        self.set_bytes = n_ops * self.B * self.N * self.V * (4 if cfg.dtype == "f32" else 2)
        r = ring if ring > 0 else max(2, -(-3 * 126 * 2 ** 20 // self.set_bytes))
        self.ring = min(r, max(2, int(max_ring_bytes // self.set_bytes)))
        self.table_ms = None
        if build_table:
            codebook = W.make_codebook(cfg.codebook_size, cfg.codebook_dim, cfg.codebook_dtype, seed=cfg.index, device=dev)
            self.nbr = L.build_neighbors(codebook, cfg.k)
            torch.cuda.synchronize()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            tb = []
            for _ in range(3):
                ev0.record()
                self.nbr = L.build_neighbors(codebook, cfg.k)
                ev1.record()
                torch.cuda.synchronize()
                tb.append(ev0.elapsed_time(ev1))
            self.table_ms = min(tb)
        else:
            self.nbr = W.random_neighbor_table(cfg.codebook_size, cfg.k, 7, device=dev)
        self.bufs = [W.make_logits(cfg, step=1000 * rank + s, device=dev) for s in range(self.ring)]
        self.params = L.Params(vocab=self.V, cfg_scale=cfg.cfg_scale if cfg.cfg_scale is not None else 1.0,
                               temperature=cfg.temperature, top_k_target=cfg.top_k, top_k_draft=cfg.top_k, lam=cfg.lam,
                               k=cfg.k, code_offset=cfg.code_offset, n_codes=cfg.codebook_size, seed=0x1A27E2 + rank,
                               allowed_begin=0 if allowed is None else allowed[0],
                               allowed_end=0 if allowed is None else allowed[1], lazy_walk=1 if walk == "lazy" else 0)
        self.tokens = [torch.zeros((self.B, self.N), dtype=torch.int32, device=dev) for _ in range(self.ring)]
        self.out = {}
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        need = L.lib.lantern_verify_tree_workspace(self.tree.handle, self.B)
        self.workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
        self.alg_bytes, self.sampler_bytes = algorithmic_bytes(cfg, self.parent, self.B, allowed)
        for i in range(self.ring):                       # draft tokens for the verify-only timing
            self.sample(i, i)
        torch.cuda.synchronize()

    def sample(self, i, step, lg=None):
        lg = self.bufs[i % self.ring] if lg is None else lg
        self.params.step = step
        self.L.sample_draft_tree(self.params, self.tree, lg["draft_cond"], lg["draft_uncond"],
                                 tokens=self.tokens[i % self.ring], device_status=self.status)

    def verify(self, i, step, lg=None):
        lg = self.bufs[i % self.ring] if lg is None else lg
        self.params.step = step
        self.L.verify_tree(self.params, self.tree, self.nbr, lg["target_cond"], lg["target_uncond"], lg["draft_cond"],
                           lg["draft_uncond"], self.tokens[i % self.ring], None, None, out=self.out,
                           device_status=self.status, workspace=self.workspace)

    def step(self, i, step, lg=None):
        self.sample(i, step, lg)
        self.verify(i, step, lg)

    def kernels(self):
        """Which kernels the library runs for these parameters (it decides; this only reports)."""
        pv = self.L.verify_tree_path(self.params, self.tree, self.B)
        ps = self.L.sample_draft_tree_path(self.params, self.tree, self.B)
        v = {0: ("verify_nodes_kernel + walk_kernel", 2),
             1: ("verify_sparse_kernel + verify_nodes_kernel (repair launch, walks the trees)", 2),
             2: ("verify_stream_kernel + walk_kernel", 2)}[pv]
        if self.params.lazy_walk:
            v = ("verify_nodes_kernel (path walk: one cluster per sequence)", 1)
        s = {0: ("sample_children_kernel", 1), 1: ("sample_sparse_kernel + sample_children_kernel (repair launch)", 2),
             2: ("sample_stream_kernel", 1)}[ps]
        return v, s


def time_calls(torch, call, ring, use_graph=True, min_ms=MIN_TIMED_MS, min_reps=20, max_reps=2000):
    """Device time per call: `ring` consecutive calls (one per input set) are captured in a CUDA
    graph and replayed; every replay is timed on its own with CUDA events on the launching
    stream, until min_reps replays and min_ms of device time.  Returns the per-call times in ms
    (sorted) of the replays."""
    for i in range(min(ring, 3)):
        call(i)
    torch.cuda.synchronize()
    g = None
    if use_graph:
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(ring):
                    call(i)
            g.replay()
            torch.cuda.synchronize()
        except Exception as exc:
            sys.stderr.write("graph capture failed, timing eager launches: %r\n" % (exc,))
            g = None
            torch.cuda.synchronize()
    times, total, reps = [], 0.0, 0
    while reps < max_reps and (reps < min_reps or total < min_ms):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if g is not None:
            g.replay()
        else:
            for i in range(ring):
                call(i)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        times.append(ms / ring)
        total += ms
        reps += 1
    times.sort()
    return times


def summarize(times, nbytes, peak):
    med = times[len(times) // 2]
    gbs = nbytes / (med * 1e-3) / 1e9
    return {"us_median": round(1e3 * med, 2), "us_min": round(1e3 * times[0], 2), "replays": len(times),
            "gbs": round(gbs, 1), "frac_measured": round(gbs / peak, 4), "frac_nominal_8tbs": round(gbs / NOMINAL_HBM_GBS, 4)}


def config_entry(torch, L, W, cfg, dev, peak, allowed=None, use_graph=True, ring=0, note=None):
    """Verify / sampler / step timings of one configuration for the `configs` object."""
    w = Workload(L, W, cfg, dev, allowed=allowed, build_table=False, ring=ring)
    tv = time_calls(torch, lambda i: w.verify(i, 100000 + i), w.ring, use_graph)
    ts = time_calls(torch, lambda i: w.sample(i, 100000 + i), w.ring, use_graph)
    tt = time_calls(torch, lambda i: w.step(i, 100000 + i), w.ring, use_graph)
    (vk, _), (sk, _) = w.kernels()
    med = tt[len(tt) // 2]
    ent = {"batch": w.B, "tree_nodes": w.N, "vocab": w.V, "logits": cfg.dtype, "allowed": allowed,
           "ring": "%d input sets, %.0f MB (> 126 MB L2)" % (w.ring, w.ring * w.set_bytes / 1e6),
           "verify_bytes": w.alg_bytes, "sampler_bytes": w.sampler_bytes,
           "verify": dict(summarize(tv, w.alg_bytes, peak), kernel=vk),
           "sampler": dict(summarize(ts, w.sampler_bytes, peak), kernel=sk),
           "step_us_median": round(1e3 * med, 2), "nodes_per_s": round(w.B * w.N / (med * 1e-3)),
           "mean_accept_len": float(w.out["accept_len"].float().mean().item()), "device_status": int(w.status.item())}
    if note:
        ent["note"] = note
    del w
    torch.cuda.empty_cache()
    return ent


def dynamic_tree_entry(torch, L, dev, peak):
    """Dynamic-tree drafting (Sec. 2.1) on rows of the headline shape: B = 64 sequences, V = 65536 bf16 drafter rows,
    6 depths, 8 children per node, frontier of 8, trimmed to 59 nodes (the node count the paper quotes for dynamic
    trees); the frontier rows of a depth are synthetic stand-ins for the drafter's forward pass.  Timed: the six
    expand calls and the trim as one CUDA graph, CUDA events around a replay, median of 20 after 3 warm-ups;
    bytes = every frontier row once."""
    B, V, D, K, E, m = 64, 65536, 6, 8, 8, 59
    g = torch.Generator(device=dev).manual_seed(17)
    rows = [(torch.randn((B, 1 if d == 0 else E, V), generator=g, device=dev) * 2.0).to(torch.bfloat16) for d in range(D)]
    par = L.Params(vocab=V)
    pool = L.DraftPool(B, D, K, E, device=dev)
    root = pool.frontier

    def run():
        pool.used, pool.n_depths, pool.frontier = 1, 0, root
        for d in range(D):
            L.expand_frontier(par, pool, rows[d])
        return L.trim_tree(pool, m)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(3):
            run()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        n, parent, token, index, logv = run()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    for it in range(23):
        ev0.record()
        graph.replay()
        ev1.record()
        torch.cuda.synchronize()
        if it >= 3:
            times.append(ev0.elapsed_time(ev1))
    dep = torch.gather(pool.depth, 1, index.clamp(min=0).long()).float()
    depth_mean = float((dep * (index >= 0)).sum() / (index >= 0).sum())
    times.sort()
    med = times[len(times) // 2]
    alg = sum(int(r.numel()) * 2 for r in rows)
    return {"workload": "f3_dynamic_tree: B=64, V=65536 bf16, 6 depths, top-8 children, frontier 8, trim to 59 nodes",
            "kernels": "expand_rows_kernel + select_frontier_kernel (x6), trim_tree_kernel", "launches": 2 * D + 1,
            "us_median": round(1e3 * med, 1), "us_min": round(1e3 * times[0], 1), "algorithmic_bytes": alg,
            "gbs": round(alg / (med * 1e-3) / 1e9, 1), "frac_measured": round(alg / (med * 1e-3) / 1e9 / peak, 4),
            "mean_nodes": float(n.float().mean()), "mean_node_depth": round(depth_mean, 3),
            "note": "two passes per row (HBM, then L2); about 10 instructions per logit and pass, latency-bound chain per row"}


def c1_three_numbers(torch, L, W, dev, peak, use_graph=True):
    """Config 1 is smaller than a launch: (i) latency of a single eager verify call on an idle
    stream, (ii) 256 decode steps over 256 distinct input sets replayed back to back in one CUDA
    graph, (iii) the 256 steps' 256 x 26 rows verified by one launch through the batch dimension."""
    cfg = W.CONFIGS["c1_tiny"]
    w = Workload(L, W, cfg, dev, build_table=False, ring=256)
    lat = []
    for i in range(60):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        w.verify(i, 300000 + i)
        e1.record()
        torch.cuda.synchronize()
        lat.append(e0.elapsed_time(e1))
    lat = sorted(lat[10:])
    tv = time_calls(torch, lambda i: w.verify(i, 100000 + i), w.ring, use_graph)
    tt = time_calls(torch, lambda i: w.step(i, 100000 + i), w.ring, use_graph)
    out = {"single_call_verify_us_median": round(1e3 * lat[len(lat) // 2], 2),
           "graph_256_steps_verify": summarize(tv, w.alg_bytes, peak),
           "graph_256_steps_step_us_median": round(1e3 * tt[len(tt) // 2], 2)}
    del w
    torch.cuda.empty_cache()
    big = dataclasses.replace(cfg, batch=256)
    wb = Workload(L, W, big, dev, build_table=False, ring=2)
    tb = time_calls(torch, lambda i: wb.verify(i, 100000 + i), wb.ring, use_graph)
    sb = time_calls(torch, lambda i: wb.sample(i, 100000 + i), wb.ring, use_graph)
    out["steps_batched_256x26_rows_verify"] = summarize(tb, wb.alg_bytes, peak)
    out["steps_batched_256x26_rows_sampler"] = summarize(sb, wb.sampler_bytes, peak)
    del wb
    torch.cuda.empty_cache()
    return out


def main():
    args = parse_args()
    import workloads as W
    if args.workload == "c5_table_sweep":
        run_table_sweep(args)
        return
    if args.workload == "f3_dynamic_tree":
        run_dynamic_tree(args)
        return
    cfg = W.CONFIGS[args.workload]
    if args.batch > 0:
        cfg = dataclasses.replace(cfg, batch=args.batch)
    parent = W.static_tree(cfg.n_nodes)
    if args.impl == "reference":
        run_reference(args, cfg, parent)
        return

    import torch
    import torch.distributed as dist
    import paper_2502_06352_b200 as L

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    use_graph = not args.no_graph
    peak, peak_kind = peak_hbm()

    w = Workload(L, W, cfg, dev, rank=rank, ring=args.ring, walk=args.walk)
    N, B, V, ring = w.N, w.B, w.V, w.ring

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    warm = max(3, args.warmup)
    for i in range(warm):
        w.step(i, i)
    sync_all()

    # ---- timed region: exactly K steps on device-resident inputs.  The launches of `ring`
    # consecutive steps are captured once in a CUDA graph and replayed (a step is a few short
    # launches: without a graph the host, not the GPU, sets the pace of the small workloads).
    # The K-step region is repeated until MIN_TIMED_MS of device time has been timed; the
    # median repetition is reported.
    K = args.steps
    per_graph = min(ring, max(1, K))
    g_step = None
    if use_graph:
        try:
            g_step = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_step):
                for i in range(per_graph):
                    w.step(i, 100000 + i)
            g_step.replay()
            torch.cuda.synchronize()
        except Exception as exc:                    # capture not possible: time eager launches
            sys.stderr.write("graph capture failed, timing eager launches: %r\n" % (exc,))
            g_step = None
            torch.cuda.synchronize()
    clocks = ClockSampler(local)
    time.sleep(0.3)
    regions, total_ms = [], 0.0
    while len(regions) < 3 or (total_ms < MIN_TIMED_MS and len(regions) < 200):
        sync_all()
        t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_start.record()
        done = 0
        if g_step is not None:
            while done + per_graph <= K:
                g_step.replay()
                done += per_graph
        while done < K:
            w.step(done, 100000 + done)
            done += 1
        t_end.record()
        sync_all()
        ms = t_start.elapsed_time(t_end)
        if world > 1:
            t = torch.tensor([ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        regions.append(ms)
        total_ms += ms
    regions.sort()
    elapsed_ms = regions[len(regions) // 2]
    # the dominant kernel on its own, and the sampler (same stream, same buffers, measured live)
    tv = time_calls(torch, lambda i: w.verify(i, 100000 + i), ring, use_graph)
    ts = time_calls(torch, lambda i: w.sample(i, 100000 + i), ring, use_graph)
    clk = clocks.stop()
    verify_med_ms = tv[len(tv) // 2]
    accept_mean = float(w.out["accept_len"].float().mean().item())
    # accepted path lengths of the last step: how many sequences accepted exactly d draft tokens, and the
    # share of sequences that got past each depth (the per-depth accept rate of the walk, Sec. 2.1)
    al = w.out["accept_len"].cpu().tolist()
    hist = [al.count(d) for d in range(max(al) + 1)]
    reach = [sum(1 for x in al if x >= d) / len(al) for d in range(1, max(al) + 1)]
    dev_status = int(w.status.item())
    total_nodes = world * B * N * K
    value = total_nodes / (elapsed_ms * 1e-3)

    # ---- end to end: per step, inputs come from pinned host memory and results go back
    KE = max(1, min(args.e2e_steps, K))
    host = {k: (None if v is None else torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v))
            for k, v in w.bufs[0].items()}
    stage = {k: (None if v is None else torch.empty_like(v)) for k, v in w.bufs[0].items()}
    h_len = torch.empty((B,), dtype=torch.int32, pin_memory=True)
    h_tok = torch.empty((B, w.tree.max_depth + 1), dtype=torch.int32, pin_memory=True)
    h2d = sum(v.numel() * v.element_size() for v in host.values() if v is not None)
    d2h = h_len.numel() * 4 + h_tok.numel() * 4

    def e2e_step(i):
        for k_, v in host.items():
            if v is not None:
                stage[k_].copy_(v, non_blocking=True)
        w.step(0, 200000 + i, stage)
        h_len.copy_(w.out["accept_len"], non_blocking=True)
        h_tok.copy_(w.out["out_tokens"], non_blocking=True)
        torch.cuda.synchronize()

    for i in range(3):
        e2e_step(i)
    sync_all()
    w0 = time.perf_counter()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(KE):
        e2e_step(i)
    t_end.record()
    sync_all()
    e2e_ms = max(t_start.elapsed_time(t_end), 1e3 * (time.perf_counter() - w0))
    if world > 1:
        t = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    e2e_value = world * B * N * KE / (e2e_ms * 1e-3)
    del host, stage

    alg_bytes = w.alg_bytes
    if args.walk == "lazy":
        # the path walk reads only the rows of the nodes it visits: count them for the same calls
        # the verify-only timing made (each input set of the ring once)
        kids = {}
        for i, pa in enumerate(parent):
            if i:
                kids.setdefault(pa, []).append(i)
        c_ops = 2 if cfg.cfg_scale is not None else 1
        e_sz = 4 if cfg.dtype == "f32" else 2
        total = 0
        for i in range(ring):
            w.verify(i, 100000 + i)
            torch.cuda.synchronize()
            al = w.out["accept_len"].cpu().numpy()
            on = w.out["out_nodes"].cpu().numpy()
            for b in range(B):
                for n in [0] + [int(x) for x in on[b, : int(al[b])]]:
                    total += (2 if n in kids else 1) * c_ops * V * e_sz
        alg_bytes = total // ring
    (vk, vl), (sk, sl) = w.kernels()
    launches_per_step = vl + sl
    table = {"ms": w.table_ms, "L": cfg.codebook_size, "d": cfg.codebook_dim, "k": cfg.k, "dtype": cfg.codebook_dtype}
    set_bytes = w.set_bytes
    parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.walk == "eager":
        parity = parity_sample(L, W, cfg, parent, w.bufs[0], w.nbr, sorted({0, B // 2}))
    del w
    torch.cuda.empty_cache()

    if rank == 0:
        achieved = alg_bytes / (verify_med_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": warm,
            "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": cfg.name + ("" if args.batch <= 0 else " (batch overridden)"), "batch_per_gpu": B, "tree_nodes": N, "vocab": V, "logits": cfg.dtype,
                       "arithmetic": "f32 (exact re-ranking steps in f64)",
                       "cfg_scale": cfg.cfg_scale, "top_k": cfg.top_k, "neighbours_k": cfg.k, "lambda": cfg.lam,
                       "codebook": [cfg.codebook_size, cfg.codebook_dim], "parallelism": "dp%d" % world,
                       "l2_policy": "ring of %d input sets, %.0f MB in total (> 126 MB L2)" % (ring, ring * set_bytes / 1e6),
                       "step": "sample_draft_tree + verify_tree (incl. walk), %d kernel launches" % launches_per_step,
                       "walk": args.walk + (" (only the rows on the accepted paths are read; algorithmic_bytes counts those)"
                                            if args.walk == "lazy" else ""),
                       "launch": "cuda graph of %d steps, replayed" % per_graph if g_step is not None else "eager",
                       "timed": "region of exactly %d steps, repeated %d times (%.0f ms of device time); median region"
                                % (K, len(regions), total_ms)},
            "roofline": {"bound": "hbm", "kernel": vk, "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind,
                         "frac_nominal_8tbs": achieved / NOMINAL_HBM_GBS,
                         "traffic": measured_traffic(cfg.name) if args.walk == "eager" else None,
                         "algorithmic_bytes": alg_bytes, "launch_ms_median": verify_med_ms, "launch_ms_min": tv[0],
                         "replays": len(tv),
                         "sampler": dict(summarize(ts, algorithmic_bytes(cfg, parent, B)[1], peak), kernel=sk),
                         "step_bytes_incl_sampler": alg_bytes + algorithmic_bytes(cfg, parent, B)[1],
                         "step_gbs": (alg_bytes + algorithmic_bytes(cfg, parent, B)[1]) / (elapsed_ms / K * 1e-3) / 1e9},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": KE},
            "gpu_launches": launches_per_step * K,
            "clocks": clk,
            "table_build": table,
            "stats": {"mean_accept_len": accept_mean, "tokens_per_step": accept_mean + 1.0, "device_status": dev_status,
                      "accept_len_hist": hist, "reached_depth_share": [round(x, 4) for x in reach]},
        }
        if world == 1 and args.configs == "all" and args.walk == "eager":
            cfgs = {}
            for name in ("c1_tiny", "c2_llamagen512", "c3_lumina", "c4_batch64"):
                if name == cfg.name:
                    cfgs[name] = {"see": "headline of this line", "verify": dict(summarize(tv, alg_bytes, peak), kernel=vk),
                                  "sampler": line["roofline"]["sampler"], "step_us_median": round(1e3 * elapsed_ms / K, 2),
                                  "nodes_per_s": round(value)}
                    continue
                cfgs[name] = config_entry(torch, L, W, W.CONFIGS[name], dev, peak, use_graph=use_graph)
            c3 = W.CONFIGS["c3_lumina"]
            cfgs["c3_lumina_image_tokens_only"] = config_entry(
                torch, L, W, c3, dev, peak, allowed=(c3.code_offset, c3.code_offset + c3.codebook_size), use_graph=use_graph,
                ring=16, note="tokens restricted to the 8192 image codes; bytes counted for that slice of every row")
            cfgs["c1_tiny"]["three_numbers"] = c1_three_numbers(torch, L, W, dev, peak, use_graph)
            cfgs["f3_dynamic_tree"] = dynamic_tree_entry(torch, L, dev, peak)
            rows, dup = table_sweep(False)
            cfgs["c5_table_sweep"] = {
                "dup_frac": dup, "total_ms": round(sum(r["ms"] for r in rows), 2),
                "builds": [[r["L"], r["d"], r["k"], r["ms"], round(r["contraction_tflops"], 2), r["path"]] for r in rows],
                "columns": ["L", "d", "k", "ms", "contraction TFLOP/s (2 L^2 d / time)", "path"]}
            line["configs"] = cfgs
        if parity is not None:
            line["stats"]["parity_sample"] = parity
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(cfg, parent)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
