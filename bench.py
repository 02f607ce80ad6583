#!/usr/bin/env python
"""Benchmark of the CaDDTree hot path: tree build + tree verify rounds per second on B200.

A *step* is one decoding round of the whole hot path over one batch of synthetic input:
    cadd_build_tree   (softmax + top-K over every live draft position, expansion, emission)
    cadd_verify_tree  (argmax over every target row, accepted-path walk)
The default workload is the largest benchmark configuration that fits one GPU: configuration 5 (batch 256, L 16 with
4..16 live positions per request, V 151936, bf16, K 8, B_max 384) with verification over the dense
[batch, B_max+1, V] target tensor, 30.7 GB of logits per round.  Configurations 2 and 4 (budget stress) are measured
the same way afterwards and reported as extra keys of the same line (`other_workloads`).  Inputs are seeded synthetic
logits (paper_2606_01813_b200.synth); they are far larger than L2, so no flush is needed between steps.

`python bench.py --gpus N --steps K --warmup W` prints ONE JSON line (rank 0).  With N > 1 every rank runs an
independent replica of the workload (requests are independent; there is no exchange step), and the value is the
rounds all ranks completed per second of the slowest rank; the N ranks come from torchrun, or, when the command is
started by hand, from this script starting N copies of itself.
`--impl reference` times the CPU oracle instead (the only baseline there is: the paper ships no code).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2606_01813_b200 import replicas, synth

METRIC = "tree build+verify rounds/sec"
UNIT = "rounds/s"
# Kernels per step: softmax_topk_partial, expand_emit, row_argmax, accept_walk; small problems (config 1) take one
# kernel per call, two per step.  The library says which (cadd_build_launches / cadd_verify_launches).

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one row_argmax launch as a multiple of its
# algorithmic bytes, from an ncu capture of the config-2 launch (summary kept under profiles/)
# (2.5037 GB for 2.4990 GB).  Traffic grows in proportion to the rows read, so other workloads scale it.
ARGMAX_TRAFFIC_RATIO = 1.0019
# The same for one softmax_topk_partial launch (171.5 MB read + written for 155.6 MB of logits: the records it writes and
# the part of its second look at ~16 two-kilobyte pieces per segment that misses L2),
# profiles/softmax_topk_partial_config2_config3.md.
TOPK_TRAFFIC_RATIO = 1.102
NOMINAL_HBM_GBS = 8000.0      # the nominal HBM3e figure the bandwidth target is stated against


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.proc = None
        self.path = None
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
            self.out.close()
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
            sm, mx, reasons = [], [], set()
            for r in rows:
                if len(r) < 8:
                    continue
                try:
                    sm.append(float(r[1])); mx.append(float(r[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                    if val.strip().lower() == "active":
                        reasons.add(name)
            if sm:
                res = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}
        except Exception:
            pass
        return res


def cost_kwargs(G, c):
    if c.kind == synth.COST_TABLE:
        return dict(cost_kind=G.COST_TABLE, cost_table=c.table, table_idx=c.table_idx, t_draft=c.t_draft)
    return dict(cost_kind=G.COST_QUADRATIC, cost_coef=c.coef)


def workload_string(cfg, rows_mode):
    return (f"config {cfg.index} ({cfg.name}): batch={cfg.batch} L={cfg.L} V={cfg.V} {cfg.dtype} "
            f"K={cfg.K} B_max={cfg.B_max} R={cfg.R}, verify rows_mode={rows_mode}")


def config_block(cfg, rows_mode, world):
    """The `config` object of the JSON line; the same for the CUDA arm and the reference arm."""
    dense_bytes = (cfg.batch * cfg.L + cfg.batch * cfg.R) * cfg.V * cfg.elem_bytes
    big = rows_mode == "dense" and dense_bytes > (126 << 20)
    return {"workload": workload_string(cfg, rows_mode),
            "l2": ("inputs larger than L2 (no flush needed)" if big else
                   "inputs may fit in L2 and are not flushed between steps (a launch-bound or live-rows case)"),
            "parallelism": f"replicas x{world}"}


def hbm_roofline(kernel, nbytes, ms, traffic_ratio, profile):
    """Roofline block of one streaming kernel: algorithmic bytes of one launch over its CUDA-event duration."""
    peak, peak_kind = measured_peak_gbs()
    ach = nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
    return {"kernel": kernel, "bound": "hbm", "achieved": round(ach, 1), "peak": peak, "peak_kind": f"of {peak_kind}",
            "unit": "GB/s", "frac": round(ach / peak, 4), "frac_of_nominal_8tbs": round(ach / NOMINAL_HBM_GBS, 4),
            "traffic": int(nbytes * traffic_ratio), "traffic_source": profile,
            "algorithmic_bytes": int(nbytes), "ms": round(ms, 5)}


class Workload:
    """One benchmark configuration resident in HBM: inputs, reusable outputs, and the step that is timed."""

    def __init__(self, G, cfg, rows_mode, rank, dev):
        self.G, self.cfg, self.dev = G, cfg, dev
        self.rows_mode_name = rows_mode
        self.rows_mode = G.ROWS_DENSE if rows_mode == "dense" else G.ROWS_LIVE
        self.flags = G.FLAG_FIXED_BUDGET if cfg.fixed_budget else 0
        seed = replicas.replica_seed(synth.config_seed(cfg), rank)
        self.d = d = synth.make_draft_inputs(cfg, seed, device=str(dev))
        self.c = c = synth.make_cost_inputs(cfg, seed)
        self.kw = dict(l_eff=d.l_eff.to(dev), bonus_token=d.bonus_token.to(dev), ctx_len=d.ctx_len.to(dev))
        self.ck = {k: (v.to(dev) if torch.is_tensor(v) else v) for k, v in cost_kwargs(G, c).items()}
        self.ws = torch.empty(G.cadd_build_workspace_bytes(cfg.batch, cfg.L, cfg.V, cfg.K, cfg.B_max, cfg.R, cfg.torch_dtype),
                              dtype=torch.uint8, device=dev)
        self.tree = G.cadd_build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, workspace=self.ws, flags=self.flags, **self.kw, **self.ck)
        torch.cuda.synchronize()
        self.y = synth.make_target_logits(cfg, seed, d, self.tree.depth.cpu(), device=str(dev))
        self.verdict = G.cadd_verify_tree(self.y, cfg.L, self.tree.n_nodes, self.tree.token_ids, self.tree.parent_idx, self.rows_mode)
        torch.cuda.synchronize()
        n_star = self.tree.n_nodes.cpu()
        es = cfg.elem_bytes
        self.n_star = n_star
        self.build_bytes = int(d.l_eff.clamp(0, cfg.L).sum().item()) * cfg.V * es
        rows_read = cfg.batch * cfg.R if self.rows_mode == G.ROWS_DENSE else int((n_star + 1).sum().item())
        self.verify_bytes = rows_read * cfg.V * es

    def build(self, x=None, extra_flags=0):
        cfg = self.cfg
        self.G.cadd_build_tree(self.d.logits if x is None else x, cfg.K, cfg.B_max, cfg.R, workspace=self.ws, out=self.tree,
                               flags=self.flags | extra_flags, **self.kw, **self.ck)

    def verify(self, y=None, flags=0):
        t = self.tree
        self.G.cadd_verify_tree(self.y if y is None else y, self.cfg.L, t.n_nodes, t.token_ids, t.parent_idx, self.rows_mode,
                                out=self.verdict, flags=flags)

    def step(self):
        self.build()
        self.verify()


def barrier():
    replicas.barrier()
    torch.cuda.synchronize()


def timed_region(w, K, Wm, world):
    """Wm untimed steps, then exactly K steps between one pair of CUDA events on the launching stream, bracketed by
    barrier + synchronize; MAX over ranks.  Returns (total ms, wall seconds)."""
    for _ in range(Wm):
        w.step()
    e_start, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0 = time.perf_counter()
    e_start.record()
    for _ in range(K):
        w.step()
    e_end.record()
    barrier()
    return replicas.max_over_ranks(e_start.elapsed_time(e_end), w.dev), time.perf_counter() - t0


def per_kernel_pass(w, K):
    """K more steps, each kernel of the step launched by a call of its own (the single-kernel flags of the C ABI) with a
    CUDA event on either side, so that every kernel is timed alone on the launching stream.  Kept out of the timed
    region: the events keep a kernel from being set up while the one before it drains."""
    G = w.G
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(5 * K)]
    for i in range(K):
        ev[5 * i].record()
        w.build(extra_flags=G.FLAG_ONLY_TOPK)
        ev[5 * i + 1].record()
        w.build(extra_flags=G.FLAG_ONLY_EXPAND)
        ev[5 * i + 2].record()
        w.verify(flags=G.VERIFY_ONLY_ARGMAX)
        ev[5 * i + 3].record()
        w.verify(flags=G.VERIFY_ONLY_WALK)
        ev[5 * i + 4].record()
    barrier()
    mean = lambda a, b: sum(ev[5 * i + a].elapsed_time(ev[5 * i + b]) for i in range(K)) / K
    steps = sorted(ev[5 * i].elapsed_time(ev[5 * i + 4]) for i in range(K))
    return {"softmax_topk_partial": mean(0, 1), "expand_emit": mean(1, 2), "row_argmax": mean(2, 3), "accept_walk": mean(3, 4),
            "step_mean": mean(0, 4), "step_median": steps[K // 2], "step_min": steps[0]}


def kernel_blocks(w, km):
    """Roofline blocks of the two streaming kernels and the absolute times of the two latency-bound ones."""
    topk = hbm_roofline("softmax_topk_partial", w.build_bytes, km["softmax_topk_partial"], TOPK_TRAFFIC_RATIO,
                        "profiles/softmax_topk_partial_config2_config3.md, scaled by rows")
    argmax = hbm_roofline("row_argmax", w.verify_bytes, km["row_argmax"], ARGMAX_TRAFFIC_RATIO,
                          "profiles/row_argmax_config2.md, scaled by rows")
    return topk, argmax, {k: round(km[k], 5) for k in ("softmax_topk_partial", "expand_emit", "row_argmax", "accept_walk",
                                                         "step_mean", "step_median", "step_min")}


def topk_alone_block(w, dev, iters=20):
    """The softmax/top-K kernel launched alone, back to back, after a pause that lets the clocks recover from the
    30 GB steps before it: this kernel is bound by instruction issue, so its time follows the SM clock (which a long
    streaming step pulls down to the power cap), while the arg-max's does not."""
    G = w.G
    torch.cuda.synchronize()
    time.sleep(0.5)
    for _ in range(3):
        w.build(extra_flags=G.FLAG_ONLY_TOPK)
    sampler = ClockSampler(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0.record()
    for _ in range(iters):
        w.build(extra_flags=G.FLAG_ONLY_TOPK)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    while time.perf_counter() - t0 < 0.35:                 # long enough for a few clock samples
        w.build(extra_flags=G.FLAG_ONLY_TOPK)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    blk = hbm_roofline("softmax_topk_partial (launched alone, back to back)", w.build_bytes, ms, TOPK_TRAFFIC_RATIO,
                       "profiles/softmax_topk_partial_config2_config3.md, scaled by rows")
    blk["launches"] = iters
    blk["sm_mhz"] = clocks.get("sm_mhz")
    return blk


def tree_stats(w):
    n = w.n_star
    return {"n_star_mean": round(float(n.float().mean()), 2), "n_star_max": int(n.max()), "n_star_hist": n_star_histogram(n),
            "accepted_mean": round(float(w.verdict.accepted_len.float().mean().item()), 2)}


def side_workload(G, name, rows_mode, rank, world, dev, K, Wm):
    """Another benchmark configuration measured the same way (timed region + per-kernel pass), reported as an extra key."""
    cfg = synth.CONFIGS[name]
    w = Workload(G, cfg, rows_mode, rank, dev)
    total_ms, _ = timed_region(w, K, Wm, world)
    km = per_kernel_pass(w, K)
    topk, argmax, kms = kernel_blocks(w, km)
    out = {"workload": workload_string(cfg, rows_mode), "value": round(replicas.whole_job_rounds_per_second(K, world, total_ms), 3),
           "unit": UNIT, "steps": K, "ms_per_step": round(total_ms / K, 5), "kernel_ms": kms,
           "roofline_softmax_topk": topk, "roofline_row_argmax": argmax, "trees": tree_stats(w)}
    del w
    torch.cuda.empty_cache()
    return out


def run_ours(args, rank, world):
    from paper_2606_01813_b200 import binding as G
    from paper_2606_01813_b200 import build as cuda_build
    cuda_build.build()                       # no-op when libcadd.so is current; raises if it cannot be built
    local = int(os.environ.get("LOCAL_RANK", 0))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    replicas.init_replicas("nccl", dev)
    cfg = synth.CONFIGS[args.workload]
    if args.batch:
        cfg = synth.scaled(cfg, batch=args.batch)        # reduced case of the same workload (profiling captures)
    w = Workload(G, cfg, args.rows_mode, rank, dev)      # inputs resident in HBM
    d, c, y, tree, verdict, ws, kw, ck = w.d, w.c, w.y, w.tree, w.verdict, w.ws, dict(w.kw, flags=w.flags), w.ck
    rows_mode = w.rows_mode
    kernels_per_step = G.cadd_round_launches(cfg.batch, cfg.L, cfg.V, cfg.K, cfg.B_max, cfg.R, cfg.torch_dtype, rows_mode)

    # ---- device-resident timing ----
    K, Wm = args.steps, max(args.warmup, 3)
    sampler = ClockSampler(dev) if rank == 0 else None
    total_ms, t_wall = timed_region(w, K, Wm, world)
    km = per_kernel_pass(w, K)
    # keep the GPU busy long enough for a few clock samples if the timed region was very short
    if sampler is not None:
        t_end = time.perf_counter() + max(0.0, 0.6 - t_wall)
        while time.perf_counter() < t_end:
            w.step()
        torch.cuda.synchronize()
    clocks = sampler.stop() if sampler is not None else None
    value = replicas.whole_job_rounds_per_second(K, world, total_ms)
    roofline_topk, roofline, kernel_ms = kernel_blocks(w, km)
    try:
        roofline_topk["alone"] = topk_alone_block(w, dev)
    except Exception as ex:
        roofline_topk["alone"] = {"error": str(ex)[:200]}
    verify_bytes = w.verify_bytes
    step = w.step

    # ---- end to end through the public API with HOST buffers ----
    e2e = None
    if not args.no_e2e:
        try:
            e2e = e2e_block(G, w, world, max(1, min(K, args.e2e_steps)))
        except Exception as ex:      # e.g. the host cannot pin a copy of the target logits
            e2e = {"error": str(ex)[:200]}
        torch.cuda.empty_cache()

    # ---- verification under sampling (T = 1) over the same target logits: one draw per row instead of the arg-max ----
    sampled = None
    if not args.no_sampled:
        try:
            sampled = sampled_block(G, cfg, tree, y, rows_mode, verify_bytes, dev, min(K, 10))
        except Exception as ex:
            sampled = {"error": str(ex)[:200]}

    # ---- the same step captured once in a CUDA graph and replayed (launch overhead removed) ----
    graph = None
    if not args.no_graph:
        try:
            ref_nodes, ref_acc = tree.n_nodes.clone(), verdict.accepted_len.clone()
            cg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cg):
                step()
            for _ in range(3):
                cg.replay()
            barrier()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record()
            for _ in range(K):
                cg.replay()
            g1.record()
            barrier()
            gms = replicas.max_over_ranks(g0.elapsed_time(g1), dev)
            same = bool(torch.equal(ref_nodes, tree.n_nodes) and torch.equal(ref_acc, verdict.accepted_len))
            graph = {"ms_per_step": round(gms / K, 5), "value": round(replicas.whole_job_rounds_per_second(K, world, gms), 3),
                     "unit": UNIT, "replays": K, "kernels_per_replay": kernels_per_step, "outputs_match": same}
            del cg
        except Exception as ex:  # capture is an extra measurement: report why it is missing, keep the main line
            graph = {"error": str(ex)[:200]}

    # (the extra measurements below are short; a pause before each lets the clocks recover from the block before it)
    settle = lambda: (torch.cuda.synchronize(), time.sleep(0.3))
    # ---- tree construction fused into the drafter's output projection, next to library GEMM + cadd_build_tree ----
    fused_draft = None
    if args.head_hidden > 0:
        try:
            settle()
            fused_draft = draft_head_block(G, cfg, kw, ck, args.head_hidden, dev, min(K, 10))
        except Exception as ex:
            fused_draft = {"error": str(ex)[:200]}

    # ---- verification fused into the output projection (tensor-core path), next to library GEMM + argmax ----
    fused_head = None
    if args.head_hidden > 0:
        try:
            settle()
            fused_head = head_block(G, cfg, tree, verdict, y, rows_mode, args.head_hidden, dev, min(K, 10))
        except Exception as ex:
            fused_head = {"error": str(ex)[:200]}

    # ---- offline cost fitting on a synthetic 9 x 1024 latency grid (the paper's profiling shape) ----
    cost_fit = None
    if not args.no_fit:
        try:
            settle()
            cost_fit = fit_block(G, dev)
        except Exception as ex:
            cost_fit = {"error": str(ex)[:200]}

    # ---- rounds with a fresh seed each (configuration 5 is defined that way): inputs regenerated outside the timing ----
    fresh = None
    if args.fresh_rounds > 0:
        try:
            fresh = fresh_rounds_block(G, cfg, rank, rows_mode, w.flags, ws, tree, verdict, y, dev, args.fresh_rounds)
        except Exception as ex:
            fresh = {"error": str(ex)[:200]}

    # ---- the oracle timed on this machine's host cores, on a bounded sample (rank 0, N = 1 only) ----
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = oracle_sample(cfg, d, c, y, tree, w.rows_mode == G.ROWS_DENSE, args.cpu_requests)

    # ---- two more of the V = 151936 configurations, measured the same way, as extra keys of the line ----
    others = {}
    for name in [n for n in args.also.split(",") if n and n != "none"]:
        if name == args.workload or args.batch:
            continue
        try:
            settle()
            if name in ("c3", "c4", "c4_stress", "c5"):          # tens of GB each: make room first
                w.y = None
                y = None
                torch.cuda.empty_cache()
            others[name] = side_workload(G, name, args.rows_mode, rank, world, dev, min(K, 50), 3)
        except Exception as ex:
            others[name] = {"error": str(ex)[:200]}

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": round(total_ms / K, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "config": config_block(cfg, args.rows_mode, world),
            "timing": "value: K steps between one pair of CUDA events; roofline blocks and kernel_ms: a second pass of K steps in "
                      "which every kernel is launched by a call of its own with a CUDA event on either side",
            "trees": tree_stats(w),
            "roofline": roofline, "roofline_softmax_topk": roofline_topk, "kernel_ms": kernel_ms,
            "other_workloads": others, "cuda_graph": graph, "fused_head": fused_head, "fused_draft_head": fused_draft,
            "sampled_verify": sampled, "fresh_seed_rounds": fresh, "cost_fit": cost_fit, "e2e": e2e, "cpu_baseline": cpu_baseline,
            "gpu_launches": kernels_per_step * K, "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    replicas.shutdown()


def e2e_block(G, w, world, ke):
    """The same step through the public API with HOST buffers: every step copies the draft and target logits from pinned
    host memory to the device and reads the tree arrays and the verdict back, all inside the timed region."""
    d, y, tree, verdict = w.d, w.y, w.tree, w.verdict
    hx = torch.empty(d.logits.shape, dtype=d.logits.dtype, pin_memory=True)
    hx.copy_(d.logits)
    hy = torch.empty(y.shape, dtype=y.dtype, pin_memory=True)
    hy.copy_(y)
    tree_t = (tree.n_nodes, tree.token_ids, tree.parent_idx, tree.depth)
    out_t = (verdict.accepted_len, verdict.accepted_nodes, verdict.next_bonus)
    h_tree = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in tree_t]
    h_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in out_t]
    dx = torch.empty_like(d.logits)
    dy = y                                   # the resident copy is overwritten with the same bits

    def e2e_step():
        dx.copy_(hx, non_blocking=True)
        w.build(x=dx)
        for h, t in zip(h_tree, tree_t):
            h.copy_(t, non_blocking=True)
        dy.copy_(hy, non_blocking=True)
        w.verify(y=dy)
        for h, t in zip(h_out, out_t):
            h.copy_(t, non_blocking=True)

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(ke):
        e2e_step()
    e1.record()
    barrier()
    ems = replicas.max_over_ranks(e0.elapsed_time(e1), w.dev)
    h2d = hx.numel() * hx.element_size() + hy.numel() * hy.element_size()
    d2h = sum(h.numel() * h.element_size() for h in h_tree + h_out)
    same = bool(torch.equal(h_tree[0], w.n_star))
    return {"value": round(replicas.whole_job_rounds_per_second(ke, world, ems), 3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": ke, "ms_per_step": round(ems / ke, 3), "trees_match_resident_run": same}


def n_star_histogram(n_star):
    """Requests per tree-size bin: 0, 1-3, 4-7, 8-15, ... (powers of two)."""
    edges = [0, 1, 4, 8, 16, 32, 64, 128, 256, 512, 1024, 2049]
    out = {}
    for lo, hi in zip(edges[:-1], edges[1:]):
        cnt = int(((n_star >= lo) & (n_star < hi)).sum())
        if cnt:
            out[str(lo) if hi == lo + 1 else f"{lo}-{hi - 1}"] = cnt
    return out


def measured_peak_tflops():
    try:
        with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"]), "measured (burst)"
    except Exception:
        return 1590.0, "fallback"


def head_block(G, cfg, tree, verdict, y, rows_mode, hidden, dev, iters):
    """cadd_verify_tree_fused_head on synthetic hidden states / weight of the workload's shape, timed alone with CUDA
    events, beside the same work done as a library GEMM that writes the logits plus cadd_verify_tree."""
    g = torch.Generator(device=dev).manual_seed(1234)
    M = cfg.batch * cfg.R
    h = torch.randn(cfg.batch, cfg.R, hidden, device=dev, dtype=torch.bfloat16, generator=g)
    w = torch.randn(cfg.V, hidden, device=dev, dtype=torch.bfloat16, generator=g)
    ws = torch.empty(G.cadd_head_workspace_bytes(cfg.batch, cfg.R, hidden, cfg.V, cfg.L), dtype=torch.uint8, device=dev)
    out = G.cadd_verify_tree_fused_head(h, w, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, rows_mode, workspace=ws)

    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    t_fused = timed(lambda: G.cadd_verify_tree_fused_head(h, w, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, rows_mode,
                                                          workspace=ws, out=out))
    y2 = torch.empty(cfg.batch, cfg.R, cfg.V, device=dev, dtype=torch.bfloat16)   # own buffer: the step's logits stay intact
    t_gemm = timed(lambda: torch.matmul(h.view(M, hidden), w.T, out=y2.view(M, cfg.V)))   # library GEMM, logits written in bf16
    v2 = G.cadd_verify_tree(y2, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, rows_mode)
    t_arg = timed(lambda: G.cadd_verify_tree(y2, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, rows_mode, out=v2))
    # LIVE mode: only rows j <= n*[b] are projected (packed first); with trees of a few nodes the weights' one pass
    # over HBM sets the time
    ws_l = torch.empty(G.cadd_head_workspace_bytes(cfg.batch, cfg.R, hidden, cfg.V, cfg.L, G.ROWS_LIVE), dtype=torch.uint8, device=dev)
    out_l = G.cadd_verify_tree_fused_head(h, w, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, G.ROWS_LIVE, workspace=ws_l)
    t_live = timed(lambda: G.cadd_verify_tree_fused_head(h, w, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, G.ROWS_LIVE,
                                                         workspace=ws_l, out=out_l))
    live_rows = int((tree.n_nodes.clamp(0, cfg.R - 1) + 1).sum().item())
    flops = 2.0 * M * hidden * cfg.V
    peak, kind = measured_peak_tflops()
    ach = flops / (t_fused * 1e-3) / 1e12
    return {"hidden": hidden, "rows": M, "ms": round(t_fused, 4), "flops": flops,
            "live_rows": live_rows, "live_ms": round(t_live, 4), "weight_bytes": cfg.V * hidden * 2,
            "roofline": {"bound": "tensor", "achieved": round(ach, 1), "peak": peak, "peak_kind": f"of {kind}", "unit": "TFLOP/s",
                         "frac": round(ach / peak, 4)},
            "library_gemm_ms": round(t_gemm, 4), "argmax_on_logits_ms": round(t_arg, 4),
            "status_bits": int(out.status.max().item()), "iters": iters}


def draft_head_block(G, cfg, kw, ck, hidden, dev, iters):
    """cadd_build_tree_fused_head on synthetic drafter hidden states / weight of the workload's shape (logits of
    standard deviation 1.5), timed alone, beside a library GEMM that writes bf16 logits plus cadd_build_tree."""
    if cfg.K > 32:
        return {"skipped": "K > 32"}
    g = torch.Generator(device=dev).manual_seed(4321)
    M = cfg.batch * cfg.L
    h = (torch.randn(cfg.batch, cfg.L, hidden, device=dev, generator=g) * (1.5 / hidden ** 0.5)).to(torch.bfloat16)
    w = torch.randn(cfg.V, hidden, device=dev, dtype=torch.bfloat16, generator=g)
    ws = torch.empty(G.cadd_build_head_workspace_bytes(cfg.batch, cfg.L, cfg.V, hidden, cfg.K, cfg.B_max, cfg.R), dtype=torch.uint8, device=dev)
    out = G.cadd_build_tree_fused_head(h, w, cfg.K, cfg.B_max, cfg.R, workspace=ws, **kw, **ck)

    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    t_fused = timed(lambda: G.cadd_build_tree_fused_head(h, w, cfg.K, cfg.B_max, cfg.R, workspace=ws, out=out, **kw, **ck))
    x2 = torch.empty(cfg.batch, cfg.L, cfg.V, device=dev, dtype=torch.bfloat16)
    t_gemm = timed(lambda: torch.matmul(h.view(M, hidden), w.T, out=x2.view(M, cfg.V)))
    ws2 = torch.empty(G.cadd_build_workspace_bytes(cfg.batch, cfg.L, cfg.V, cfg.K, cfg.B_max, cfg.R, torch.bfloat16), dtype=torch.uint8, device=dev)
    o2 = G.cadd_build_tree(x2, cfg.K, cfg.B_max, cfg.R, workspace=ws2, **kw, **ck)
    t_build = timed(lambda: G.cadd_build_tree(x2, cfg.K, cfg.B_max, cfg.R, workspace=ws2, out=o2, **kw, **ck))
    flops = 2.0 * M * hidden * cfg.V
    peak, kind = measured_peak_tflops()
    ach = flops / (t_fused * 1e-3) / 1e12
    return {"hidden": hidden, "rows": M, "ms": round(t_fused, 4), "flops": flops,
            "roofline": {"bound": "tensor", "achieved": round(ach, 1), "peak": peak, "peak_kind": f"of {kind}", "unit": "TFLOP/s",
                         "frac": round(ach / peak, 4)},
            "library_gemm_ms": round(t_gemm, 4), "build_on_logits_ms": round(t_build, 4),
            "status_bits": int(out.status.max().item()), "iters": iters}


def sampled_block(G, cfg, tree, y, rows_mode, verify_bytes, dev, iters):
    """cadd_verify_tree_sampled at temperature 1 on the step's target logits (the same bytes the arg-max reads)."""
    gu = torch.Generator(device="cpu").manual_seed(cfg.index + 99)
    u = torch.rand(cfg.batch, cfg.R, generator=gu, dtype=torch.float64).to(dev)
    out = G.cadd_verify_tree_sampled(y, u, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, rows_mode, temperature=1.0)
    for _ in range(2):
        G.cadd_verify_tree_sampled(y, u, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, rows_mode, temperature=1.0, out=out)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        G.cadd_verify_tree_sampled(y, u, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, rows_mode, temperature=1.0, out=out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    peak, kind = measured_peak_gbs()
    gbs = verify_bytes / (ms * 1e-3) / 1e9
    return {"temperature": 1.0, "ms": round(ms, 4), "achieved_gbs": round(gbs, 1), "frac_of_hbm_peak": round(gbs / peak, 3),
            "peak_kind": kind, "accepted_mean": round(float(out.accepted_len.float().mean().item()), 2)}


def fresh_rounds_block(G, cfg, rank, rows_mode, flags, ws, tree, verdict, y, dev, n_rounds):
    """n_rounds rounds, each on inputs drawn from its own seed (1000 * config + round): draft logits and costs are
    regenerated, the tree is built once untimed so that the target logits can be drawn for it (as the target's forward
    pass would produce them), then one build + verify is timed with CUDA events."""
    times, n_mean, acc_mean = [], [], []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for r in range(n_rounds):
        seed = replicas.replica_seed(synth.config_seed(cfg, r), rank)
        d = synth.make_draft_inputs(cfg, seed, device=str(dev))
        c = synth.make_cost_inputs(cfg, seed)
        kw = dict(l_eff=d.l_eff.to(dev), bonus_token=d.bonus_token.to(dev), ctx_len=d.ctx_len.to(dev), flags=flags)
        ck = {k: (v.to(dev) if torch.is_tensor(v) else v) for k, v in cost_kwargs(G, c).items()}
        G.cadd_build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, workspace=ws, out=tree, **kw, **ck)
        torch.cuda.synchronize()
        synth.make_target_logits(cfg, seed, d, tree.depth.cpu(), device=str(dev), out=y)
        torch.cuda.synchronize()
        e0.record()
        G.cadd_build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, workspace=ws, out=tree, **kw, **ck)
        G.cadd_verify_tree(y, cfg.L, tree.n_nodes, tree.token_ids, tree.parent_idx, rows_mode, out=verdict)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
        n_mean.append(float(tree.n_nodes.float().mean().item()))
        acc_mean.append(float(verdict.accepted_len.float().mean().item()))
        del d
    ts = sorted(times)
    return {"rounds": n_rounds, "value": round(n_rounds / (sum(times) * 1e-3), 3), "unit": UNIT,
            "ms_mean": round(sum(times) / n_rounds, 4), "ms_median": round(ts[n_rounds // 2], 4), "ms_min": round(ts[0], 4),
            "ms_max": round(ts[-1], 4), "n_star_mean": round(sum(n_mean) / n_rounds, 2),
            "accepted_mean": round(sum(acc_mean) / n_rounds, 2)}


def fit_block(G, dev, iters=5):
    """cadd_fit_cost_tables on nine noisy convex latency curves of 1024 points each; absolute time (a small,
    latency-bound problem: one CTA per curve), not a roofline figure."""
    g = torch.Generator(device="cpu").manual_seed(21)
    n = torch.arange(1, 1025, dtype=torch.float64)
    y = torch.stack([18.0 + 2.0 * j + (0.010 + 0.002 * j) * n + (2e-5 + 2e-6 * j) * n * n + 0.004 * torch.clamp(n - 256, min=0)
                     + (0.2 + 0.05 * j) * torch.randn(1024, generator=g, dtype=torch.float64) for j in range(9)]).to(dev)
    fit, nb, st = G.cadd_fit_cost_tables(y)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        G.cadd_fit_cost_tables(y)
    e1.record()
    torch.cuda.synchronize()
    return {"tables": 9, "points": 1024, "ms": round(e0.elapsed_time(e1) / iters, 4), "slope_changes_max": int(nb.max().item()),
            "status_bits": int(st.max().item()), "rmse": round(float(((fit - y) ** 2).mean().sqrt().item()), 5)}


def oracle_sample(cfg, d, c, y, tree, dense, n_req, target_cpu_seconds=15.0):
    """Time the CPU oracle, as it stands, on the first n_req requests of the workload, repeated until about
    target_cpu_seconds of CPU work (wall time x threads) have been spent; then once more on one thread, on fewer
    requests.  The oracle's trees are compared with the CUDA path's on the way (requests that differ, and how many of
    those differ at a decision the oracle itself made with a margin below 1e-6)."""
    from oracle import cadd_oracle as O
    nb = min(n_req, cfg.batch)
    x = d.logits[:nb].cpu()
    yy = y[:nb].cpu()
    mode = O.ROWS_DENSE if dense else O.ROWS_LIVE

    def kwargs(n):
        kw = dict(l_eff=d.l_eff[:n], bonus_token=d.bonus_token[:n], ctx_len=d.ctx_len[:n],
                  flags=O.FLAG_FIXED_BUDGET if cfg.fixed_budget else 0)
        if c.kind == synth.COST_TABLE:
            kw.update(cost_kind=O.COST_TABLE, cost_table=c.table, table_idx=c.table_idx[:n], t_draft=c.t_draft[:n])
        else:
            kw.update(cost_coef=c.coef[:n])
        return kw

    cores = O.num_threads()
    reps, dt = 0, 0.0
    t0 = time.perf_counter()
    while True:
        ot = O.build_tree(x, cfg.K, cfg.B_max, cfg.R, **kwargs(nb))
        O.verify_tree(yy, cfg.L, ot.n_nodes, ot.token_ids, ot.parent_idx, mode)
        reps += 1
        dt = time.perf_counter() - t0
        if dt * cores >= target_cpu_seconds or reps >= 50:
            break
    # the same code on one thread, on a smaller sample (about a third of the CPU work above)
    n1 = max(1, min(nb, int(nb * (target_cpu_seconds / 3.0) / max(dt / reps * cores, 1e-9))))
    O.set_num_threads(1)
    t1 = time.perf_counter()
    o1 = O.build_tree(x[:n1], cfg.K, cfg.B_max, cfg.R, **kwargs(n1))
    O.verify_tree(yy[:n1], cfg.L, o1.n_nodes, o1.token_ids, o1.parent_idx, mode)
    dt1 = time.perf_counter() - t1
    O.set_num_threads(cores)
    g_n, g_tok, g_par = tree.n_nodes[:nb].cpu(), tree.token_ids[:nb].cpu(), tree.parent_idx[:nb].cpu()
    differ = [b for b in range(nb) if not (int(ot.n_nodes[b]) == int(g_n[b]) and torch.equal(ot.token_ids[b], g_tok[b])
                                           and torch.equal(ot.parent_idx[b], g_par[b]))]
    inside = 0
    for b in differ:
        k = min(int(ot.n_nodes[b]), int(g_n[b])) + 1
        rows = [j for j in range(k) if int(ot.token_ids[b, j]) != int(g_tok[b, j]) or int(ot.parent_idx[b, j]) != int(g_par[b, j])]
        margin = float(ot.pop_gap[b, rows[0]]) if rows else float(ot.stop_gap[b])
        inside += margin < 1e-6
    return {"value": round(reps * (nb / cfg.batch) / dt, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{reps} x ({nb} of {cfg.batch} requests of the same workload, one build + verify each), "
                      f"{dt:.2f} s wall on {cores} threads; value scaled to whole rounds",
            "single_thread_value": round((n1 / cfg.batch) / dt1, 5),
            "single_thread_sample": f"1 x ({n1} of {cfg.batch} requests), {dt1:.2f} s on 1 thread; value scaled to whole rounds",
            "trees_match_gpu": not differ, "requests_differing_from_gpu": len(differ), "of_which_inside_oracle_margin_1e-6": int(inside)}


def run_reference(args, rank, world):
    """The reference arm: there is no reference implementation (the paper ships none), so the oracle is
    timed on the host cores, each step a bounded sample of the workload."""
    if rank != 0:
        return
    from oracle import cadd_oracle as O
    O.build()
    cfg = synth.CONFIGS[args.workload]
    nb = min(args.cpu_requests, cfg.batch)
    small = synth.scaled(cfg, batch=nb)
    seed = synth.config_seed(cfg)
    d = synth.make_draft_inputs(small, seed)
    c = synth.make_cost_inputs(small, seed)
    kw = dict(l_eff=d.l_eff, bonus_token=d.bonus_token, ctx_len=d.ctx_len, flags=O.FLAG_FIXED_BUDGET if cfg.fixed_budget else 0)
    if c.kind == synth.COST_TABLE:
        kw.update(cost_kind=O.COST_TABLE, cost_table=c.table, table_idx=c.table_idx, t_draft=c.t_draft)
    else:
        kw.update(cost_coef=c.coef)
    dense = args.rows_mode == "dense"
    ot = O.build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, **kw)
    y = synth.make_target_logits(small, seed, d, ot.depth)

    def step():
        t = O.build_tree(d.logits, cfg.K, cfg.B_max, cfg.R, **kw)
        O.verify_tree(y, cfg.L, t.n_nodes, t.token_ids, t.parent_idx, O.ROWS_DENSE if dense else O.ROWS_LIVE)

    K, Wm = args.steps, args.warmup
    for _ in range(Wm):
        step()
    t0 = time.perf_counter()
    for _ in range(K):
        step()
    dt = time.perf_counter() - t0
    value = K * (nb / cfg.batch) / dt
    sample = f"each step = {nb} of {cfg.batch} requests of the workload (build + verify), value scaled to whole rounds"
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": Wm, "ms_per_step": round(dt / K * 1e3, 3), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_block(cfg, args.rows_mode, world),
            "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_stub(args, rank, world):
    """The launcher and the replica plumbing without a GPU: every rank joins a gloo group, 'steps' are short sleeps,
    rank 0 prints a line with the contract's base keys.  Used by the CPU tests of `--gpus N`."""
    replicas.init_replicas("gloo")
    cpu = torch.device("cpu")
    K, Wm = args.steps, max(args.warmup, 3)
    for _ in range(Wm):
        time.sleep(0.001)
    replicas.barrier()
    t0 = time.perf_counter()
    for _ in range(K):
        time.sleep(0.002 * (1 + rank))                   # the last rank is the slow one
    ms = replicas.max_over_ranks((time.perf_counter() - t0) * 1e3, cpu)
    replicas.barrier()
    if rank == 0:
        cfg = synth.CONFIGS[args.workload]
        print(json.dumps({"metric": METRIC, "value": round(replicas.whole_job_rounds_per_second(K, world, ms), 3), "unit": UNIT,
                          "n_gpus": world, "steps": K, "warmup": Wm, "ms_per_step": round(ms / K, 5), "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "stub (no GPU work)",
                          "config": config_block(cfg, args.rows_mode, world), "gpu_launches": 0}), flush=True)
    replicas.shutdown()


def launch_replicas(n):
    """`python bench.py --gpus N` started by hand (no torchrun): start N copies of this command, one per GPU, with the
    rendezvous variables torchrun would set; rank 0 prints the line.  Returns the worst exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    return max(p.wait() for p in procs)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=sorted(synth.CONFIGS),
                    help="the timed configuration; default: the largest one that fits a GPU (config 5, 30.7 GB per round)")
    ap.add_argument("--also", default="c2,c4_stress",
                    help="comma-separated configurations measured the same way after the main one and reported under "
                         "other_workloads ('none' to skip)")
    ap.add_argument("--rows-mode", default="dense", choices=["dense", "live"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--cpu-requests", type=int, default=32)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (0 = as defined)")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay measurement")
    ap.add_argument("--no-sampled", action="store_true", help="skip the sampling-mode verification measurement")
    ap.add_argument("--fresh-rounds", type=int, default=0,
                    help="also time this many rounds with a fresh seed each (inputs regenerated outside the timed calls)")
    ap.add_argument("--no-fit", action="store_true", help="skip the offline cost-fitting measurement")
    ap.add_argument("--head-hidden", type=int, default=4096,
                    help="hidden size for the fused output-projection verification measurement (0 = skip)")
    ap.add_argument("--stub", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(launch_replicas(args.gpus))           # not under torchrun: become the launcher
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", args.gpus if args.impl == "reference" else 1))
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args, rank, world)
    else:
        args.steps = 100 if args.steps is None else args.steps
        args.warmup = 5 if args.warmup is None else args.warmup
        (run_stub if args.stub else run_ours)(args, rank, world)


if __name__ == "__main__":
    main()
