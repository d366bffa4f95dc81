#!/usr/bin/env python
"""Benchmark of the UBTree draft+verify hot path: drafted-and-verified trees per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

A step is one pass of the whole path over one synthetic batch: ubt_draft_tree (vocabulary log-softmax +
top-k, pair normalisation, tree expansion, mask/positions) followed by ubt_verify_tree (per-node target
pick over [B,N,V] logits and the acceptance walk).  Prints ONE JSON line.  With torchrun (N > 1) every
rank runs the same step on its own batch (weak scaling, no data-path collective) and rank 0 reports the
aggregate; timing is CUDA events, max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import numpy as np
import torch

import ubt_synth as synth

NOMINAL_HBM_GBS = 8000.0          # nominal HBM3e bandwidth of a B200, the figure the 70 % target is stated against
FALLBACK_HBM_GBS = 6650.0         # an earlier measured copy bandwidth, used only without MEASURED_PEAKS.json


def algorithmic_bytes_per_tree(cfg: synth.Config) -> dict:
    """Bytes the method must move per tree: every logit once, the selector scores, every output."""
    e = 2 if cfg.dtype == "bf16" else 4
    mw = (cfg.N + 31) // 32
    draft = cfg.L * cfg.V * e
    target = cfg.N * cfg.V * e
    small = (max(cfg.L - 1, 0) * cfg.k * cfg.k * 4            # bigram scores
             + cfg.L * cfg.k * 8                               # candidates out
             + cfg.N * (6 * 4 + mw * 4) + 4                    # tree arrays + mask + n_nodes
             + (2 * (cfg.L + 1) + 2) * 4)                      # verify outputs
    return {"draft_logits": draft, "target_logits": target, "other": small, "total": draft + target + small}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_tensor_peak():
    """Dense bf16 TFLOP/s of a library product measured on this kind of GPU: the burst figure, for a kernel timed alone."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["bf16_tflops"]), "measured (burst)"
    except Exception:
        return 1590.0, "fallback"


def measure_lm_head(ubt, dev, rows=512, d=4096, V=151936, k=8, reps=10):
    """The LM head fused with step a1 (one tensor-core kernel, logits never stored), timed alone with CUDA events,
    and next to it the unfused route on the same inputs: a library bf16 product that stores the logits, then
    ubt_topk_logprob.  L2: the weight matrix (1.2 GB) is larger than L2 and every launch reads all of it."""
    hd, wd = synth.device_lm_head_inputs(rows, d, V, seed=5, device=dev)
    ids = torch.empty((rows, k), dtype=torch.int32, device=dev)
    lp = torch.empty((rows, k), dtype=torch.float32, device=dev)
    ws = ubt.workspace(ubt.ubt_lm_head_workspace_bytes(rows, d, V, k), dev)
    logits = torch.empty((rows, V), dtype=torch.bfloat16, device=dev)
    ws_t = ubt.workspace(ubt.ubt_draft_workspace_bytes(rows, 1, V, k, 1), dev)

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    def unfused():
        torch.matmul(hd, wd.T, out=logits)
        ubt.ubt_topk_logprob(logits, k, ids, lp, ws_t)

    t_f = timed(lambda: ubt.ubt_lm_head_topk(hd, wd, k, ids, lp, ws))
    t_u = timed(unfused)
    flops = 2.0 * rows * d * V
    peak, kind = measured_tensor_peak()
    return {"kernel": "k_lm_head_topk", "bound": "tensor", "rows": rows, "d": d, "V": V, "k": k, "dtype": "bf16",
            "avg_ms": t_f, "achieved": flops / (t_f * 1e-3) / 1e12, "unit": "TFLOP/s", "peak": peak,
            "peak_source": f"of {kind}", "frac": flops / (t_f * 1e-3) / 1e12 / peak,
            "unfused_ms": t_u, "unfused": "library bf16 product storing the logits + ubt_topk_logprob",
            "launches_per_call": 2, "timeouts": ubt.ubt_debug_ring_timeouts()}


def measure_lm_head_verify(ubt, dev, d=4096, reps=5):
    """Greedy verification straight from the target's hidden states of the tree slots (c3's trees: 32 x 64 slots):
    the LM head fused with the row arg max (ubt_lm_head_topk, k = 1), then the walk on the picks
    (ubt_verify_tree_picks); next to it the unfused route, a library bf16 product that stores the [B, N, V] target
    logits followed by ubt_verify_tree."""
    cfg = synth.CONFIGS["c3"]
    ud, bd, _ = synth.device_inputs(cfg, 1, dev, want_target=False)
    tree = ubt.ubt_draft_tree(ud, bd, cfg.k, cfg.N)
    rows = cfg.B * cfg.N
    hd, wd = synth.device_lm_head_inputs(rows, d, cfg.V, seed=6, device=dev)
    hidden = hd.view(cfg.B, cfg.N, d)
    logits = torch.empty((cfg.B, cfg.N, cfg.V), dtype=torch.bfloat16, device=dev)
    res = ubt.VerifyResult.empty(cfg.B, cfg.L, dev)
    ws_v = ubt.workspace(ubt.ubt_verify_workspace_bytes(cfg.B, cfg.N, cfg.V, "greedy"), dev)

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    def unfused():
        torch.matmul(hd, wd.T, out=logits.view(rows, cfg.V))
        ubt.ubt_verify_tree(tree, logits, "greedy", result=res, ws=ws_v)

    t_f = timed(lambda: ubt.verify_tree_from_hidden(tree, hidden, wd, result=res))
    t_u = timed(unfused)
    flops = 2.0 * rows * d * cfg.V
    peak, kind = measured_tensor_peak()
    return {"kernels": "k_lm_head_topk + k_lm_head_merge + k_walk", "bound": "tensor", "workload": "c3 trees",
            "rows": rows, "d": d, "V": cfg.V, "dtype": "bf16", "avg_ms": t_f,
            "achieved": flops / (t_f * 1e-3) / 1e12, "unit": "TFLOP/s", "peak": peak, "peak_source": f"of {kind}",
            "frac": flops / (t_f * 1e-3) / 1e12 / peak, "unfused_ms": t_u,
            "unfused": "library bf16 product storing the target logits + ubt_verify_tree",
            "logits_bytes_not_written": rows * cfg.V * 2, "timeouts": ubt.ubt_debug_ring_timeouts()}


def recorded_traffic(kernel: str, workload: str):
    """DRAM bytes per launch of `kernel` from the committed ncu summary, if one exists (else None)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            return json.load(f).get(kernel, {}).get(workload)
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.15 and len(r) >= 9] or [r for _, r in self.rows if len(r) >= 9]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        num = lambda s: float(s) if s.replace(".", "", 1).isdigit() else None
        sm = [num(r[1]) for r in rows if num(r[1]) is not None]
        reasons = set()
        for r in rows:
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7),
                              ("sw_power_cap", 8)):
                if r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": num(rows[0][2]),
                "power_w_max": max((num(r[3]) or 0.0) for r in rows), "samples": len(rows),
                "reasons": sorted(reasons)}


def input_seed(rank: int, s: int) -> int:
    """Seed of input set ``s`` on rank ``rank``: every rank streams its own batches (weak scaling)."""
    return 1000 * rank + s


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    return world, rank, local


def max_over_ranks(value: float, world: int, device) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def oracle_pass(cfg, uh, bh, zh, seed, phi=None, psi=None, gate=None, anchor=None, W=0):
    """One oracle draft+verify pass on host arrays; returns (tree, verdict, seconds).  With selector tables the
    bigram scores come from the oracle's selector (the paper's data flow) instead of ``bh``."""
    import oracle
    t0 = time.perf_counter()
    if phi is not None:
        ids, _, _ = oracle.topk_logprob(uh, cfg.k)
        big, anc = oracle.selector_scores(phi, psi, gate, ids, anchor)
        tr = oracle.draft_tree(uh, big.astype(np.float32), cfg.k, cfg.N, W=W, anchor_bigram=anc.astype(np.float32),
                               anchor_tokens=anchor)
    else:
        tr = oracle.draft_tree(uh, bh, cfg.k, cfg.N)
    v = oracle.verify(tr.token_ids, tr.parents, tr.n_nodes, cfg.L, zh, cfg.mode, seed=seed)
    return tr, v, time.perf_counter() - t0


def run_reference(args, cfg, world, rank):
    """The reference arm: the CPU oracle as it stands, on the host cores, on a bounded sample per step."""
    if rank != 0:
        return
    import oracle
    sample = max(1, min(cfg.B, args.ref_trees))
    sub = cfg.replace(B=sample)
    di = synth.draft_inputs(sub, 0)
    z = synth.target_logits(sub, 0)
    for _ in range(args.warmup):
        oracle_pass(sub, di.unigram_logits, di.bigram_scores, z, 0)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_pass(sub, di.unigram_logits, di.bigram_scores, z, 0)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    line = {"impl": "reference", "metric": "draft+verify trees/sec", "value": value, "unit": "trees/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "L": cfg.L, "V": cfg.V, "k": cfg.k, "node_budget": cfg.N,
                       "verify": cfg.mode, "logits": cfg.dtype},
            "cpu_baseline": {"value": value, "unit": "trees/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": f"{sample} of {cfg.B} sequences per step"},
            "e2e": {"value": value, "unit": "trees/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


WORKLOADS_DEFAULT = ("c4", "c3", "c5")     # headline first (the largest single-GPU configuration), then the other two


def kernel_record(name, bytes_per_launch, ms, peak, peak_kind, **extra):
    gbs = bytes_per_launch / (ms * 1e-3) / 1e9 if ms and ms > 0 else None
    rec = {"kernel": name, "algorithmic_bytes": bytes_per_launch, "avg_ms": ms, "gbs": gbs,
           "frac": (gbs / peak) if gbs else None, "peak": peak, "peak_source": f"of {peak_kind}"}
    rec.update(extra)
    return rec


def measure_workload(ubt, args, cfg, paper_flow, world, rank, dev, stream, headline):
    """All device-timed figures of one workload.  Returns (record, state) where state keeps what the headline's
    end-to-end and CPU-baseline legs need."""
    bpt = algorithmic_bytes_per_tree(cfg)
    batch_bytes = bpt["total"] * cfg.B
    # enough distinct batches that one rotation exceeds twice the 126 MB L2
    n_sets = max(2, min(16, -(-4 * 126_000_000 // max(batch_bytes, 1))))
    sets = [synth.device_inputs(cfg, input_seed(rank, s), dev) for s in range(n_sets)]
    tree = ubt.Tree.empty(cfg.B, cfg.N, cfg.L, cfg.k, dev)
    res = ubt.VerifyResult.empty(cfg.B, cfg.L, dev)
    ws_d = ubt.workspace(ubt.ubt_draft_workspace_bytes(cfg.B, cfg.L, cfg.V, cfg.k, cfg.N), dev)
    ws_v = ubt.workspace(ubt.ubt_verify_workspace_bytes(cfg.B, cfg.N, cfg.V, cfg.mode), dev)
    K = args.steps
    mk = lambda: torch.cuda.Event(enable_timing=True)
    ev = [[mk() for _ in range(5)] for _ in range(K)]       # step start, between draft kernels, draft end,
    for row in ev:                                          # verify kernel end, step end
        for e in row:
            e.record(stream)

    sel = {}
    if paper_flow:
        R, W = synth.SELECTOR_RANK, synth.search_width(cfg)
        phi, psi, gate, anchor = synth.device_selector_tables(cfg.V, R, cfg.B, cfg.L, input_seed(rank, 99), dev)
        sel = dict(phi=phi, psi=psi, gate=gate, anchor=anchor, W=W,
                   big=torch.empty((cfg.B, cfg.L - 1, cfg.k, cfg.k), dtype=torch.float32, device=dev),
                   anc=torch.empty((cfg.B, cfg.k), dtype=torch.float32, device=dev))

    def draft(ud, bd, between=None):
        if paper_flow:
            ubt.ubt_topk_logprob(ud, cfg.k, tree.cand_ids, tree.cand_logprob, ws_d, stream=stream)
            if between is not None:
                between.record(stream)
            ubt.ubt_selector_scores(sel["phi"], sel["psi"], sel["gate"], tree.cand_ids, sel["anchor"],
                                    bigram_scores=sel["big"], anchor_bigram=sel["anc"], stream=stream)
            ubt.ubt_build_tree(sel["big"], tree, stream=stream, search_width=sel["W"], anchor_bigram=sel["anc"],
                               anchor_tokens=sel["anchor"])
        else:
            ubt.ubt_draft_tree(ud, bd, cfg.k, cfg.N, tree=tree, ws=ws_d, stream=stream, event_between=between)

    def verify(zd, i, early=False, e_after=None):
        ubt.ubt_verify_tree(tree, zd, cfg.mode, seed=i, temperature=1.0, result=res, ws=ws_v, stream=stream,
                            event_after=e_after, early_start=early)

    def step(i, early=False):
        ud, bd, zd = sets[i % n_sets]
        draft(ud, bd)
        verify(zd, i, early)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    barrier(world)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    time.sleep(0.25)
    t_wall0 = time.time()
    # ---- the timed region: K steps in plain stream order (the verify call reads nothing before the draft call in
    # front of it has completed, as when the target model's forward pass sits between the two)
    e0, e1 = mk(), mk()
    e0.record(stream)
    for i in range(K):
        step(args.warmup + i)
    e1.record(stream)
    torch.cuda.synchronize()
    elapsed_ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    # ---- the same K steps with events between the kernels (an event also keeps a kernel from becoming resident
    # behind the one in front): per-call and per-kernel times
    for i in range(K):
        ud, bd, zd = sets[(args.warmup + i) % n_sets]
        a, b, c, d, e = ev[i]
        a.record(stream)
        draft(ud, bd, between=b)
        c.record(stream)
        verify(zd, args.warmup + i, e_after=d)
        e.record(stream)
    torch.cuda.synchronize()
    # ---- and chained with the opt-in early start of the verify pass (only possible when the target logits do not
    # depend on the tree, as in this benchmark; reported as a secondary figure)
    e2, e3 = mk(), mk()
    e2.record(stream)
    for i in range(K):
        step(args.warmup + i, early=True)
    e3.record(stream)
    torch.cuda.synchronize()
    # ---- the verify call in its path-only form (reads only the target rows a walk visits), timed alone
    for i in range(3):
        ubt.ubt_verify_tree(tree, sets[i % n_sets][2], cfg.mode, seed=i, result=res, ws=ws_v, stream=stream,
                            path_only=True)
    torch.cuda.synchronize()
    e4, e5 = mk(), mk()
    e4.record(stream)
    for i in range(K):
        ubt.ubt_verify_tree(tree, sets[(args.warmup + i) % n_sets][2], cfg.mode, seed=i, result=res, ws=ws_v,
                            stream=stream, path_only=True)
    e5.record(stream)
    torch.cuda.synchronize()
    path_ms = max_over_ranks(e4.elapsed_time(e5), world, dev) / K
    path_len = float(res.accepted_len.float().mean())
    # ... and on targets that agree with the drafted tree (each child's token boosted in its parent's row), so
    # that the walks are several steps long.  Done last: it edits input set 0 in place.
    draft(sets[0][0], sets[0][1])
    torch.cuda.synchronize()
    synth.boost_children_on_device(sets[0][2], tree.token_ids, tree.parents, tree.n_nodes, boost=14.0)
    e6, e7 = mk(), mk()
    e6.record(stream)
    for i in range(K):
        ubt.ubt_verify_tree(tree, sets[0][2], cfg.mode, seed=i, result=res, ws=ws_v, stream=stream, path_only=True)
    e7.record(stream)
    torch.cuda.synchronize()
    path_agree_ms = max_over_ranks(e6.elapsed_time(e7), world, dev) / K
    path_agree_len = float(res.accepted_len.float().mean())
    t_wall1 = time.time()
    barrier(world)
    clocks = sampler.stop(t_wall0, t_wall1)
    chained_ms = max_over_ranks(e2.elapsed_time(e3), world, dev)

    med = statistics.median
    t_a1 = med(r[0].elapsed_time(r[1]) for r in ev)
    t_tree = med(r[1].elapsed_time(r[2]) for r in ev)
    t_draft = med(r[0].elapsed_time(r[2]) for r in ev)
    t_vk = med(r[2].elapsed_time(r[3]) for r in ev)
    t_walk = med(r[3].elapsed_time(r[4]) for r in ev)
    t_verify = med(r[2].elapsed_time(r[4]) for r in ev)

    peak, peak_kind = measured_peak()
    e = 2 if cfg.dtype == "bf16" else 4
    a1_bytes = cfg.B * cfg.L * cfg.V * e
    vk_bytes = cfg.B * cfg.N * cfg.V * e
    tree_bytes = cfg.B * (max(cfg.L - 1, 0) * cfg.k * cfg.k * 4 + cfg.L * cfg.k * 8 + cfg.N * (6 + (cfg.N + 31) // 32) * 4 + 4)
    kernels = [kernel_record("k_lse_topk_ring", a1_bytes, t_a1, peak, peak_kind,
                             traffic=recorded_traffic("k_lse_topk_ring", cfg.name))]
    if paper_flow:
        kernels.append(kernel_record("k_selector_scores+k_build_tree", tree_bytes, t_tree, peak, peak_kind,
                                     note="latency-bound search; bytes are its inputs and outputs"))
    else:
        kernels.append(kernel_record("k_build_tree", tree_bytes, t_tree, peak, peak_kind,
                                     note="latency-bound search (one CTA per sequence); bytes are its inputs and outputs"))
    if cfg.mode == "greedy":
        dominant = kernel_record("k_row_argmax_ring", vk_bytes, t_vk, peak, peak_kind,
                                 traffic=recorded_traffic("k_row_argmax_ring", cfg.name))
    else:
        dominant = kernel_record("k_row_weights_ring+k_row_pick", vk_bytes, t_vk, peak, peak_kind,
                                 traffic=recorded_traffic("k_row_weights_ring+k_row_pick", cfg.name),
                                 note="two passes over every row (maximum, then integer weights); reported against "
                                      "HBM although instruction issue is what limits it")
    kernels.append(dominant)
    kernels.append(kernel_record("k_walk", cfg.B * (2 * (cfg.L + 1) + 2) * 4, t_walk, peak, peak_kind,
                                 note="latency-bound walk of at most L+1 steps"))

    trees_per_s = cfg.B * K * world / (elapsed_ms * 1e-3)
    step_gbs = batch_bytes * K / (elapsed_ms * 1e-3) / 1e9
    launches_per_step = 2 + (2 if cfg.mode == "greedy" else 3)   # top-k, tree | argmax or weights+pick, walk
    if paper_flow:
        launches_per_step += 2                                   # separate merge kernel, selector scores
    rec = {
        "workload": cfg.name, "B": cfg.B, "L": cfg.L, "V": cfg.V, "k": cfg.k, "node_budget": cfg.N,
        "verify": cfg.mode, "logits": cfg.dtype, "input_sets": n_sets,
        "ms_per_step": elapsed_ms / K, "trees_per_s": trees_per_s,
        "bytes_per_tree": bpt["total"], "step_gbs_per_gpu": step_gbs,
        "frac_of_%s_peak" % peak_kind: step_gbs / peak, "frac_of_nominal_8tbs": step_gbs / NOMINAL_HBM_GBS,
        "draft_ms": t_draft, "verify_ms": t_verify,
        "calls_timed_apart_trees_per_s": cfg.B * world / ((t_draft + t_verify) * 1e-3),
        "chained_early_start": {"ms_per_step": chained_ms / K, "trees_per_s": cfg.B * K * world / (chained_ms * 1e-3),
                                "note": "verify pass started while the draft call still ran (ubt_verify_opts.early_start);"
                                        " not reachable when the target logits depend on the tree"},
        "verify_path_only": {"ms_per_call": path_ms, "mean_accepted_len": path_len,
                             "agreeing_targets": {"ms_per_call": path_agree_ms, "mean_accepted_len": path_agree_len},
                             "note": "ubt_verify_opts.path_only: evaluates at most L+1 of the N target rows of a "
                                     "sequence; its time grows with the accepted length (noise targets accept almost "
                                     "nothing; the second figure is on targets boosted towards the drafted tree)"},
        "kernels": kernels, "gpu_launches": launches_per_step * K, "clocks": clocks,
    }
    state = dict(sets=sets, tree=tree, res=res, ws_d=ws_d, ws_v=ws_v, draft=draft, sel=sel, dominant=dominant,
                 launches_per_step=launches_per_step, elapsed_ms=elapsed_ms, bpt=bpt, n_sets=n_sets, clocks=clocks)
    return rec, state


def live_parity(ubt, cfg, paper_flow, st, dev, stream, sample, timed_seconds=0.0):
    """Oracle on the first `sample` sequences of input set 0 (repeated until `timed_seconds` of CPU time have
    passed, for the CPU baseline) and an element-by-element comparison with the CUDA path on the same bytes.
    Returns (parity record, trees done, seconds spent)."""
    from parity import compare_draft, compare_verify, tree_to_numpy
    ud, bd, zd = st["sets"][0]
    sel = st["sel"]
    uh, bh, zh = (synth.to_host_bits(t[:sample]) for t in (ud, bd, zd))
    kw = {}
    if paper_flow:
        kw = dict(phi=synth.to_host_bits(sel["phi"]), psi=synth.to_host_bits(sel["psi"]),
                  gate=sel["gate"][:sample].cpu().numpy(), anchor=sel["anchor"][:sample].cpu().numpy(),
                  W=synth.search_width(cfg))
    done, spent = 0, 0.0
    while True:
        tr, ov, dt = oracle_pass(cfg, uh, bh, zh, 0, **kw)
        done += sample; spent += dt
        if spent >= timed_seconds:
            break
    st["draft"](ud, bd)
    pick = torch.empty((cfg.B, cfg.N), dtype=torch.int32, device=dev)
    ubt.ubt_verify_tree(st["tree"], zd, cfg.mode, seed=0, result=st["res"], ws=st["ws_v"], stream=stream, node_pick=pick)
    torch.cuda.synchronize()
    try:
        g = tree_to_numpy(st["tree"])
        swaps = compare_draft(g, tr, cfg.L, cfg.k, cfg.N, synth.search_width(cfg) if paper_flow else 0, 0.0,
                              kw.get("anchor"), None, rows=list(range(sample)))
        if not swaps:
            compare_verify(st["res"], ov, pick, rows=slice(0, sample))
        rec = {"checked_trees": sample, "near_tie_swaps": len(swaps), "ok": True}
    except AssertionError as ex:
        rec = {"checked_trees": sample, "ok": False, "error": str(ex)[:200]}
    return rec, done, spent


def parity_sample(cfg, paper_flow) -> int:
    """Sequences the oracle checks live: the whole c3 batch, a bounded sample of the multi-GB workloads."""
    if paper_flow:
        return max(1, min(cfg.B, 2))
    return cfg.B if cfg.B * cfg.N * cfg.V <= 32 * 64 * 151_936 else 8


def self_launch(args) -> int:
    """`python bench.py --gpus N` outside a multi-rank launcher: start the N ranks (one per GPU) ourselves."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(synth.CONFIGS) + sorted(synth.NEXT_CONFIGS),
                    help="one workload only; default: c4 (headline), then c3 and c5 in per_workload")
    ap.add_argument("--ref-trees", type=int, default=4, help="sequences per step of the reference arm")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="CPU time budget of the oracle baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-lm-head", action="store_true", help="skip the fused LM head measurement (a 'next' row)")
    ap.add_argument("--lm-head-only", action="store_true", help="only that measurement (profiling captures)")
    ap.add_argument("--batch", type=int, default=0, help="override B of the workload (profiling captures only)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(self_launch(args))
    names = [args.workload] if args.workload else list(WORKLOADS_DEFAULT)
    cfgs = []
    for n in names:
        c = synth.CONFIGS.get(n) or synth.NEXT_CONFIGS[n]
        if args.batch > 0:
            c = c.replace(B=args.batch, name=f"{c.name}-B{args.batch}")
        cfgs.append((c, n in synth.NEXT_CONFIGS))
    cfg, paper_flow = cfgs[0]
    # the paper's own configuration goes through the split entry points, selector scores computed on the device
    if paper_flow:
        args.no_e2e = True          # the host-buffer forms cover the fused call only
    world, rank, local = dist_setup(args.gpus)

    if args.impl == "reference":
        run_reference(args, cfg, world, rank)
        return

    import paper_2609_39972_b200 as ubt          # fails loudly if libubt.so is missing: no CPU fallback
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ubt.load()
    stream = torch.cuda.current_stream()
    if args.lm_head_only:
        if rank == 0:
            print(json.dumps({"next_rows": {"lm_head_topk": measure_lm_head(ubt, dev, reps=max(1, args.steps)),
                                            "lm_head_verify": measure_lm_head_verify(ubt, dev)}}), flush=True)
        return

    # the other workloads first, so that the headline's buffers are the ones kept for the end-to-end legs
    per_workload = {}
    for c, pf in cfgs[1:]:
        rec, st = measure_workload(ubt, args, c, pf, world, rank, dev, stream, headline=False)
        if rank == 0 and not args.no_cpu_baseline:
            rec["parity"], _, _ = live_parity(ubt, c, pf, st, dev, stream, parity_sample(c, pf))
        per_workload[c.name] = rec
        del st
        torch.cuda.empty_cache()
    head, st = measure_workload(ubt, args, cfg, paper_flow, world, rank, dev, stream, headline=True)
    per_workload = {cfg.name: head, **per_workload}
    sets, tree, res, ws_v, draft, sel = st["sets"], st["tree"], st["res"], st["ws_v"], st["draft"], st["sel"]
    launches_per_step, n_sets = st["launches_per_step"], st["n_sets"]
    dom = st["dominant"]
    batch_bytes = st["bpt"]["total"] * cfg.B

    roof = {"bound": "hbm", "kernel": dom["kernel"], "achieved": dom["gbs"], "peak": dom["peak"], "unit": "GB/s",
            "frac": dom["frac"], "peak_source": dom["peak_source"], "traffic": dom.get("traffic"),
            "bytes_per_launch": dom["algorithmic_bytes"], "avg_launch_ms": dom["avg_ms"],
            "timed": "a second pass of the same %d steps with CUDA events recorded by the library around this "
                     "kernel on the launching stream" % args.steps}
    if "note" in dom:
        roof["note"] = dom["note"]
    line = {
        "metric": "draft+verify trees/sec", "value": head["trees_per_s"], "unit": "trees/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": head["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "L": cfg.L, "V": cfg.V, "k": cfg.k, "node_budget": cfg.N,
                   "verify": cfg.mode, "logits": cfg.dtype, "input_sets": n_sets,
                   "order": "plain stream order: draft call, then verify call, nothing overlapped",
                   **({"search_width": synth.search_width(cfg), "selector_rank": synth.SELECTOR_RANK,
                       "flow": "ubt_topk_logprob -> ubt_selector_scores -> ubt_build_tree -> ubt_verify_tree"}
                      if paper_flow else {}),
                   "l2": "inputs larger than L2 (rotation of %d MB)" % (batch_bytes * n_sets // 1_000_000)},
        "hbm": {k: head[k] for k in head if k.startswith("frac_of_") or k in
                ("bytes_per_tree", "step_gbs_per_gpu", "draft_ms", "verify_ms", "calls_timed_apart_trees_per_s",
                 "chained_early_start")},
        "roofline": roof,
        "kernels": head["kernels"],
        "per_workload": per_workload,
        "clocks": st["clocks"],
        "gpu_launches": head["gpu_launches"],
    }

    # ---- a row beyond the timed path: the LM head fused with step a1, timed alone (default run only)
    if rank == 0 and not args.no_lm_head and args.workload is None and args.batch == 0:
        line["next_rows"] = {"lm_head_topk": measure_lm_head(ubt, dev),
                             "lm_head_verify": measure_lm_head_verify(ubt, dev)}
        torch.cuda.empty_cache()

    # ---- end to end through the host-buffer entry points (pinned host inputs, results read back)
    if not args.no_e2e:
        ud, bd, zd = sets[0]
        uh, bh, zh = ud.cpu().pin_memory(), bd.cpu().pin_memory(), zd.cpu().pin_memory()
        tree_h = ubt.Tree.empty(cfg.B, cfg.N, cfg.L, cfg.k, dev, pin=True)
        res_h = ubt.VerifyResult.empty(cfg.B, cfg.L, dev, pin=True)
        code = 1 if cfg.dtype == "bf16" else 0
        dbuf = ubt.workspace(ubt.ubt_draft_host_buffer_bytes(cfg.B, cfg.L, cfg.V, cfg.k, cfg.N, code), dev)
        vbuf = ubt.workspace(ubt.ubt_verify_host_buffer_bytes(cfg.B, cfg.L, cfg.N, cfg.V, code, cfg.mode), dev)

        def e2e_step(i):
            ubt.ubt_draft_tree_host(uh, bh, cfg.k, cfg.N, tree_h, dbuf, stream=stream)
            ubt.ubt_verify_tree_host(tree_h, zh, res_h, vbuf, cfg.mode, seed=i, stream=stream)

        k_e2e = max(3, min(args.steps, 10))
        for i in range(3):
            e2e_step(i)
        torch.cuda.synchronize(); barrier(world)
        t0 = time.perf_counter()
        for i in range(k_e2e):
            e2e_step(i)
        torch.cuda.synchronize()
        dt = max_over_ranks(time.perf_counter() - t0, world, dev)
        mw = (cfg.N + 31) // 32
        h2d = uh.numel() * uh.element_size() + bh.numel() * 4 + zh.numel() * zh.element_size() + cfg.B * (2 * cfg.N + 1) * 4
        d2h = cfg.B * (cfg.N * (6 + mw) * 4 + 4 + cfg.L * cfg.k * 8) + cfg.B * (2 * (cfg.L + 1) + 2) * 4
        line["e2e"] = {"value": cfg.B * k_e2e * world / dt, "unit": "trees/s", "h2d_bytes_per_step": h2d,
                       "d2h_bytes_per_step": d2h, "steps": k_e2e, "gpu_launches": launches_per_step * k_e2e}
        del uh, bh, zh

    # ---- CPU baseline: the oracle as it stands on the host cores, on a bounded sample; doubles as a parity check
    if rank == 0 and not args.no_cpu_baseline:
        import oracle
        sample = parity_sample(cfg, paper_flow)
        par, done, spent = live_parity(ubt, cfg, paper_flow, st, dev, stream, sample, args.cpu_seconds)
        line["cpu_baseline"] = {"value": done / spent, "unit": "trees/s", "cores": oracle.num_threads(),
                                "kind": "oracle", "sample": f"first {sample} of {cfg.B} sequences, repeated for "
                                                            f"{spent:.1f} s ({done} trees)"}
        line["parity"] = par
        per_workload[cfg.name]["parity"] = par

    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
