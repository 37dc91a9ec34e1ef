"""Benchmark of the relaxed tree-verification hot path.

One step = one pass of the path over one batch of synthetic input: the draft sampler over
every internal node, the relaxed verification of every node and the walk (three kernel
launches).  The neighbour table is built once per codebook and is timed separately.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints one JSON line (rank 0).  Under torchrun every rank verifies its own batch of
sequences (no data-path collective); the value is all ranks' nodes over the slowest rank's
device time.
"""
import argparse
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


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="c2_llamagen512")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--ring", type=int, default=0, help="input buffer sets cycled through (0 = enough to exceed L2)")
    ap.add_argument("--e2e-steps", type=int, default=100)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of CUDA-graph replays")
    ap.add_argument("--walk", default="eager", choices=["eager", "lazy"],
                    help="eager: verify every tree node, then walk (the configuration the metric is quoted on); "
                         "lazy: verify only the nodes on each sequence's accepted path (params.lazy_walk)")
    return ap.parse_args()


def algorithmic_bytes(cfg, parent, batch):
    """Bytes one verify launch must move: every target row and every internal node's drafter
    row once, the neighbour rows of the draft tokens, and the per-node outputs."""
    N = len(parent)
    I = len(set(parent[1:]))
    c = 2 if cfg.cfg_scale is not None else 1
    e = 4 if cfg.dtype == "f32" else 2
    rows = batch * (N + I) * c * cfg.vocab * e
    table = batch * (N - 1) * cfg.k * 4
    outs = batch * N * (4 + 4 + 4 + 4 + 4)      # tokens, two uniforms in; next, token out
    return rows + table + outs, batch * I * c * cfg.vocab * e


# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel (mean of the two
# captured launches), from the ncu capture summarised under profiles/; valid only for the kernel
# source it was taken from
TRAFFIC = {"c2_llamagen512": {"kernel_sha256": "d16142fbf6a4b272", "bytes": 105080000}}


def kernel_sha256():
    import hashlib
    h = hashlib.sha256()
    for f in ("verify_sparse.cuh", "verify_kernel.cuh", "verify_launch.cuh", "verify.cu", "rowops.cuh", "common.cuh"):
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


def oracle_step_inputs(cfg, parent, logits_cpu, seqs, seed):
    import workloads as W
    N, V = len(parent), cfg.vocab
    gum = W.make_gumbel_uniforms(len(seqs), N, V, seed).numpy()
    ua, ur = W.make_uniforms(len(seqs), N, seed + 1)
    nbr = W.random_neighbor_table(cfg.codebook_size, cfg.k, seed + 2).numpy()
    return gum, ua.numpy(), ur.numpy(), nbr


def oracle_run_nodes(cfg, parent, lg, b, gum, ua, ur, nbr, n_nodes):
    """Oracle sampler + verifier on the first n_nodes nodes of sequence b (bounded sample)."""
    import numpy as np
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


def cpu_baseline(cfg, parent, lg_cpu, budget_s=12.0):
    """The oracle, as it stands, on whole sequences of the workload until about budget_s."""
    N = len(parent)
    B = lg_cpu["target_cond"].shape[0]
    gum, ua, ur, nbr = oracle_step_inputs(cfg, parent, lg_cpu, list(range(B)), 4242)
    t0 = time.perf_counter()
    nodes = 0
    seqs = 0
    while True:
        b = seqs % B
        nodes += oracle_run_nodes(cfg, parent, lg_cpu, b, gum[b], ua[b], ur[b], nbr, N)
        seqs += 1
        if time.perf_counter() - t0 > budget_s or seqs >= 256 * B:
            break
    dt = time.perf_counter() - t0
    return {"value": nodes / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "%d whole sequences (%d nodes: draft sampling + relaxed verification of every node) of %s, %.1f s"
                      % (seqs, nodes, cfg.name, dt)}


def run_reference(args, cfg, parent):
    """--impl reference: the CPU oracle on bounded samples of the same workload."""
    import workloads as W
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    N = len(parent)
    lg = W.make_logits(cfg, step=0, device="cpu", batch=1)
    gum, ua, ur, nbr = oracle_step_inputs(cfg, parent, lg, [0], 4242)
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


def run_table_sweep(args):
    """--workload c5_table_sweep: every (L, d, k) neighbour-table build of the sweep, timed with
    CUDA events (best of 3 after a warm-up), plus the oracle timed on a few rows of each shape."""
    import numpy as np
    import torch
    import workloads as W
    from workloads.configs import SWEEP_L, SWEEP_D, SWEEP_K, SWEEP_DUP_FRAC
    import paper_2502_06352_b200 as L
    import oracle
    torch.cuda.set_device(0)
    rows = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for n in SWEEP_L:
        for d in SWEEP_D:
            cb = W.make_codebook(n, d, "bf16", seed=5, dup_frac=SWEEP_DUP_FRAC, device="cuda")
            t_or = None
            if not args.no_cpu_baseline:
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
                             "path": "tensor" if (d % 16 == 0 and 32 <= d <= 256 and k <= 320) else "brute",
                             "oracle_rows_per_s": None if t_or is None else 1.0 / t_or})
    total_rows = sum(r["L"] for r in rows)
    total_ms = sum(r["ms"] for r in rows)
    print(json.dumps({"metric": "neighbour-table rows/sec", "value": total_rows / (total_ms * 1e-3), "unit": "rows/s",
                      "n_gpus": 1, "steps": 3, "warmup": 1, "ms_per_step": total_ms, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "bf16 mma + f64 re-rank", "data": "synthetic",
                      "config": {"workload": "c5_table_sweep", "dup_frac": SWEEP_DUP_FRAC}, "builds": rows,
                      "gpu_launches": 4 * 2 * len(rows)}))


def main():
    args = parse_args()
    import workloads as W
    if args.workload == "c5_table_sweep":
        run_table_sweep(args)
        return
    cfg = W.CONFIGS[args.workload]
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

    N, B, V = len(parent), cfg.batch, cfg.vocab
    tree = L.Tree(parent)
    alg_bytes, sampler_bytes = algorithmic_bytes(cfg, parent, B)
    set_bytes = sum(B * N * V * (4 if cfg.dtype == "f32" else 2) for _ in range(4 if cfg.cfg_scale is not None else 2))
    ring = args.ring if args.ring > 0 else max(2, -(-3 * 126 * 2 ** 20 // set_bytes))
    ring = min(ring, max(2, int(60e9 // set_bytes)))

    # ---- neighbour table: built once per codebook by the library (timed on its own)
    codebook = W.make_codebook(cfg.codebook_size, cfg.codebook_dim, cfg.codebook_dtype, seed=cfg.index, device=dev)
    nbr = L.build_neighbors(codebook, cfg.k)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tb = []
    for _ in range(3):
        ev0.record()
        nbr = L.build_neighbors(codebook, cfg.k)
        ev1.record()
        torch.cuda.synchronize()
        tb.append(ev0.elapsed_time(ev1))
    table_ms = min(tb)

    # ---- inputs: a ring of independent step buffers, together larger than L2
    bufs = [W.make_logits(cfg, step=1000 * rank + s, device=dev) for s in range(ring)]
    params = L.Params(vocab=V, cfg_scale=cfg.cfg_scale if cfg.cfg_scale is not None else 1.0,
                      temperature=cfg.temperature, top_k_target=cfg.top_k, top_k_draft=cfg.top_k, lam=cfg.lam,
                      k=cfg.k, code_offset=cfg.code_offset, n_codes=cfg.codebook_size, seed=0x1A27E2 + rank,
                      lazy_walk=1 if args.walk == "lazy" else 0)
    tokens = torch.zeros((B, N), dtype=torch.int32, device=dev)
    out = {}
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    need = L.lib.lantern_verify_tree_workspace(tree.handle, B)
    workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)

    def step(i, lg):
        params.step = i
        L.sample_draft_tree(params, tree, lg["draft_cond"], lg["draft_uncond"], tokens=tokens, device_status=status)
        L.verify_tree(params, tree, nbr, lg["target_cond"], lg["target_uncond"], lg["draft_cond"], lg["draft_uncond"],
                      tokens, None, None, out=out, device_status=status, workspace=workspace)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(i, bufs[i % ring])
    sync_all()

    # ---- timed region: exactly K steps, device-resident inputs.  The launches of `ring`
    # consecutive steps are captured once in a CUDA graph and replayed (the step is three small
    # launches: without a graph the host, not the GPU, sets the pace of the small workloads).
    K = args.steps

    def verify_only(i, lg):
        params.step = 100000 + i
        L.verify_tree(params, tree, nbr, lg["target_cond"], lg["target_uncond"], lg["draft_cond"], lg["draft_uncond"],
                      tokens, None, None, out=out, device_status=status, workspace=workspace)

    def full_step(i, lg):
        params.step = 100000 + i
        L.sample_draft_tree(params, tree, lg["draft_cond"], lg["draft_uncond"], tokens=tokens, device_status=status)
        verify_only(i, lg)

    per_graph = min(ring, max(1, K))
    g_step = g_verify = None
    if not args.no_graph:
        try:
            g_step = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_step):
                for i in range(per_graph):
                    full_step(i, bufs[i % ring])
            g_verify = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_verify):
                for i in range(per_graph):
                    verify_only(i, bufs[i % ring])
            g_step.replay()
            g_verify.replay()
            torch.cuda.synchronize()
        except Exception as exc:                    # capture not possible: time eager launches
            sys.stderr.write("graph capture failed, timing eager launches: %r\n" % (exc,))
            g_step = g_verify = None
            torch.cuda.synchronize()
    clocks = ClockSampler(local)
    time.sleep(0.3)
    sync_all()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    done = 0
    if g_step is not None:
        while done + per_graph <= K:
            g_step.replay()
            done += per_graph
    while done < K:
        full_step(done, bufs[done % ring])
        done += 1
    t_end.record()
    sync_all()
    elapsed_ms = t_start.elapsed_time(t_end)
    # the dominant kernel on its own (same stream, same buffers, measured live)
    v0, v1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_verify = 0
    v0.record()
    if g_verify is not None:
        while n_verify < min(K, 512):
            g_verify.replay()
            n_verify += per_graph
    else:
        while n_verify < min(K, 256):
            verify_only(n_verify, bufs[n_verify % ring])
            n_verify += 1
    v1.record()
    sync_all()
    clk = clocks.stop()
    verify_avg_ms = v0.elapsed_time(v1) / n_verify
    verify_ms = [verify_avg_ms]
    accept_mean = float(out["accept_len"].float().mean().item())
    dev_status = int(status.item())

    if world > 1:
        t = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())
    total_nodes = world * B * N * K
    value = total_nodes / (elapsed_ms * 1e-3)

    # ---- end to end: per step, inputs come from pinned host memory and results go back
    KE = max(1, min(args.e2e_steps, K))
    host = {k: (None if v is None else torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v))
            for k, v in bufs[0].items()}
    stage = {k: (None if v is None else torch.empty_like(v)) for k, v in bufs[0].items()}
    h_len = torch.empty((B,), dtype=torch.int32, pin_memory=True)
    h_tok = torch.empty((B, tree.max_depth + 1), dtype=torch.int32, pin_memory=True)
    h2d = sum(v.numel() * v.element_size() for v in host.values() if v is not None)
    d2h = h_len.numel() * 4 + h_tok.numel() * 4

    def e2e_step(i):
        for k_, v in host.items():
            if v is not None:
                stage[k_].copy_(v, non_blocking=True)
        step(200000 + i, stage)
        h_len.copy_(out["accept_len"], non_blocking=True)
        h_tok.copy_(out["out_tokens"], non_blocking=True)
        torch.cuda.synchronize()

    for i in range(3):
        e2e_step(i)
    sync_all()
    w0 = time.perf_counter()
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
            verify_only(i, bufs[i % ring])
            torch.cuda.synchronize()
            al = out["accept_len"].cpu().numpy()
            on = out["out_nodes"].cpu().numpy()
            for b in range(B):
                for n in [0] + [int(x) for x in on[b, : int(al[b])]]:
                    total += (2 if n in kids else 1) * c_ops * V * e_sz
        alg_bytes = total // ring
    # which kernels ran (the library decides from the parameters; this only reports it)
    lists_v = L.verify_tree_path(params, tree) == 1
    lists_s = L.sample_draft_tree_path(params) == 1
    verify_kernels = ("verify_sparse_kernel + verify_nodes_kernel (repair launch, walks the trees)" if lists_v
                      else "verify_nodes_kernel + walk_kernel")
    launches_per_step = (2 if lists_s else 1) + 2
    if args.walk == "lazy":
        verify_kernels = "verify_nodes_kernel (path walk: one cluster per sequence)"
        launches_per_step = (2 if lists_s else 1) + 1
    if rank == 0:
        peak, peak_kind = peak_hbm()
        achieved = alg_bytes / (verify_avg_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(3, args.warmup),
            "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": cfg.name, "batch_per_gpu": B, "tree_nodes": N, "vocab": V, "logits": cfg.dtype,
                       "cfg_scale": cfg.cfg_scale, "top_k": cfg.top_k, "neighbours_k": cfg.k, "lambda": cfg.lam,
                       "codebook": [cfg.codebook_size, cfg.codebook_dim], "parallelism": "dp%d" % world,
                       "l2_policy": "ring of %d input sets, %.0f MB in total (> 126 MB L2)" % (ring, ring * set_bytes / 1e6),
                       "step": "sample_draft_tree + verify_tree (incl. walk), %d kernel launches" % launches_per_step,
                       "walk": args.walk + (" (only the rows on the accepted paths are read; algorithmic_bytes counts those)"
                                            if args.walk == "lazy" else ""),
                       "launch": "cuda graph of %d steps, replayed" % per_graph if g_step is not None else "eager"},
            "roofline": {"bound": "hbm", "kernel": verify_kernels, "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind, "traffic": measured_traffic(cfg.name) if args.walk == "eager" else None,
                         "algorithmic_bytes": alg_bytes, "launch_ms_avg": verify_avg_ms,
                         "launch_ms_median": verify_ms[len(verify_ms) // 2],
                         "step_bytes_incl_sampler": alg_bytes + sampler_bytes,
                         "step_gbs": (alg_bytes + sampler_bytes) / (elapsed_ms / K * 1e-3) / 1e9},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": KE},
            "gpu_launches": launches_per_step * K,
            "clocks": clk,
            "table_build": {"ms": table_ms, "L": cfg.codebook_size, "d": cfg.codebook_dim, "k": cfg.k,
                            "dtype": cfg.codebook_dtype},
            "stats": {"mean_accept_len": accept_mean, "tokens_per_step": accept_mean + 1.0, "device_status": dev_status},
        }
        if world == 1 and not args.no_cpu_baseline:
            lg_cpu = {k: (None if v is None else v.cpu()) for k, v in bufs[0].items()}
            line["cpu_baseline"] = cpu_baseline(cfg, parent, lg_cpu)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
