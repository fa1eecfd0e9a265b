#!/usr/bin/env python
"""Benchmark of the fused Finch step (score + select + compact) on synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c3] [--impl ours|reference]

One "step" is one steady-state finch_step over all layers of the configuration (cache full, one new chunk).
Prints ONE JSON line: candidate KV tokens/s (whole job), ms per step, the HBM roofline of the step, an end-to-end
figure with host buffers, and the fp64 CPU oracle timed on a bounded sample of the same workload.
With N > 1 (launched by torchrun) every rank runs an independent replica; there is no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2408_00167_b200 import workloads as wl  # noqa: E402

METRIC = "candidate_kv_tokens_per_sec"
UNIT = "tokens/s"
FALLBACK_PEAK_GBS = 6650.0
# DRAM bytes (read + write) of one full step from ncu, per configuration: captured on an 8-layer slice and scaled by
# the unit count (profiles/step_kernels_c3_8layers.txt).  Must be set back to None whenever a kernel changes.
TRAFFIC_BYTES = {"c3": 1021440000}
MUFU_PER_CLK_PER_SM = 16   # exp2 results per clock per SM (4 per scheduler)


def peak_hbm():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
    return FALLBACK_PEAK_GBS, "fallback"


def step_counts(cfg: wl.Config, st: dict) -> dict:
    """Candidate tokens and algorithmic ("contract") bytes of one step: K read + kept K/V written."""
    e = 4 if cfg.dtype == "f32" else 2
    chunk_len = np.diff(st["chunk_off"])
    n_cand = st["cache_len"].astype(np.int64) + chunk_len
    kept = np.minimum(st["budget"].astype(np.int64), n_cand)
    rows_read = int(n_cand.sum()) * cfg.n_layers * cfg.n_kv_heads
    rows_written = 2 * int(kept.sum()) * cfg.n_layers * cfg.n_kv_heads
    return dict(tokens=int(n_cand.sum()), contract_bytes=(rows_read + rows_written) * cfg.head_dim * e,
                units=cfg.n_layers * cfg.n_groups * cfg.batch)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled in the background and filtered to a wall-clock window."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc, self.gpu = None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self, t_begin: float, t_end: float) -> dict:
        """Summary of the samples taken between the two time.time() stamps (all samples if none fall inside)."""
        import datetime
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        rows = []
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7 or not f[1].isdigit():
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
            except ValueError:
                ts = None
            rows.append((ts, int(f[1]), int(f[2]), {n for n, v in zip(names, f[3:7]) if v == "Active"}))
        inside = [r for r in rows if r[0] is not None and t_begin <= r[0] <= t_end]
        use = inside or rows
        reasons = set().union(*[r[3] for r in use]) if use else set()
        return {"sm_mhz": statistics.median([r[1] for r in use]) if use else None,
                "sm_max_mhz": use[0][2] if use else None, "reasons": sorted(reasons), "samples": len(use),
                "window": "timed steps" if inside else "whole run (no sample fell inside the timed steps)"}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def aggregate_over_ranks(ms_local: float, tokens_local: int, world: int, backend: str):
    """Replicas only: whole-job time is the slowest rank's, whole-job work is the sum.  Returns (max ms, tokens)."""
    if world == 1:
        return ms_local, tokens_local
    import torch
    import torch.distributed as dist
    dev = "cuda" if backend == "nccl" else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    n = torch.tensor([tokens_local], dtype=torch.int64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item())


def oracle_sample(cfg: wl.Config, target_s: float = 12.0, max_layers: int = 32):
    """Time the fp64 oracle's whole step on whole layers of the same workload until about target_s of CPU work."""
    import oracle
    threads = oracle.max_threads()
    total, layers_done, tokens = 0.0, 0, None
    while layers_done < min(max_layers, cfg.n_layers) and (layers_done == 0 or total < target_s):
        st = wl.steady_state(cfg, [layers_done])
        tokens = step_counts(cfg, st)["tokens"]
        t0 = time.perf_counter()
        oracle.step(cfg.dtype, st["q"], st["cache_k"], st["cache_v"], st["cache_pos"], st["chunk_k"], st["chunk_v"],
                    st["chunk_pos"], n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim,
                    group_mode=cfg.group_mode, q_off=st["q_off"], chunk_off=st["chunk_off"], cache_off=st["cache_off"],
                    cache_len=st["cache_len"], budget=st["budget"], threads=threads)
        total += time.perf_counter() - t0
        layers_done += 1
    step_s = total * cfg.n_layers / layers_done          # units are independent: a whole step is n_layers/sample
    return dict(value=tokens / step_s, unit=UNIT, cores=threads, kind="oracle",
                sample=f"{layers_done} of {cfg.n_layers} layers of {cfg.name} (all heads, full candidates), "
                       f"{total:.1f} s, scaled linearly to a whole step"), step_s


def run_ours(args, cfg: wl.Config):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, str(ROOT / "tests"))
    from paper_2408_00167_b200 import binding as fb
    from paper_2408_00167_b200 import build as fbuild
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    fbuild.build()
    fb.load()

    sampler = ClockSampler(local_rank)
    sampler.start()               # started early: nvidia-smi needs a moment before its first sample
    layers = list(range(cfg.n_layers))
    st = wl.steady_state(cfg, layers)
    counts = step_counts(cfg, st)
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16

    def pinned(a):
        t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if cfg.dtype == "bf16" and a.dtype == np.uint16
                             else np.ascontiguousarray(a))
        t = t.pin_memory()
        return t.view(dt) if a.dtype == np.uint16 else t
    host = {k: pinned(st[k]) for k in ("q", "cache_k", "cache_v", "chunk_k", "chunk_v", "cache_pos", "chunk_pos")}
    dev = {k: v.cuda(non_blocking=True) for k, v in host.items()}
    batch = fb.make_batch(st["q_off"], st["chunk_off"], st["cache_off"], st["cache_len"], st["budget"])
    c = batch.c
    ctx = fb.finch_ctx_create(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                              fb.FINCH_F32 if cfg.dtype == "f32" else fb.FINCH_BF16, cfg.group_mode,
                              max_batch=cfg.batch, max_prompt=c.max_q, max_candidates=c.max_cache + c.max_chunk,
                              device=local_rank)
    G = cfg.n_groups
    out_k, out_v = torch.empty_like(dev["cache_k"]), torch.empty_like(dev["cache_v"])
    out_pos = torch.empty((cfg.n_layers, G, c.total_cache), dtype=torch.int32, device="cuda")
    kept = torch.empty((cfg.n_layers, G, c.total_cache), dtype=torch.int32, device="cuda")
    out_len = torch.empty(cfg.batch, dtype=torch.int32, device="cuda")
    scores = torch.empty((cfg.n_layers, G, c.total_cache + c.total_chunk), dtype=torch.float32, device="cuda")
    ws = torch.empty(fb.finch_workspace_bytes(ctx, batch), dtype=torch.uint8, device="cuda")
    kept_host = torch.empty_like(kept, device="cpu").pin_memory()
    len_host = torch.empty_like(out_len, device="cpu").pin_memory()

    def step():
        fb.finch_step(ctx, dev["q"], dev["cache_k"], dev["cache_v"], dev["cache_pos"], dev["chunk_k"], dev["chunk_v"],
                      dev["chunk_pos"], batch, out_k, out_v, out_pos, kept, out_len, scores, ws)

    def step_e2e():
        # this step's inputs come from pinned host memory through the C ABI's host-buffer call; the cache is
        # carried on the device; the kept positions and lengths come back to the host
        fb.finch_step_host(ctx, host["q"], host["chunk_k"], host["chunk_v"], host["chunk_pos"], dev["q"],
                           dev["chunk_k"], dev["chunk_v"], dev["chunk_pos"], dev["cache_k"], dev["cache_v"],
                           dev["cache_pos"], batch, out_k, out_v, out_pos, kept, out_len, kept_host, len_host, ws)

    def timed(fn, n):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        a.record()
        for _ in range(n):
            fn()
        b.record()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    for _ in range(max(args.warmup, 3)):
        step()
    assert fb.finch_device_status(ctx) == 0
    launches0 = fb.finch_launch_count(ctx)
    t_begin = time.time()
    ms_local = timed(step, args.steps)
    t_end = time.time()
    launches = fb.finch_launch_count(ctx) - launches0
    assert fb.finch_device_status(ctx) == 0
    ms, tokens = aggregate_over_ranks(ms_local, counts["tokens"], world, "nccl")

    # per-phase durations (same kernels, called through the three separate entry points)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    phase = np.zeros(3)
    for _ in range(args.steps):
        ev[0].record()
        fb.finch_score(ctx, dev["q"], dev["cache_k"], dev["chunk_k"], batch, scores, None, ws)
        ev[1].record()
        fb.finch_select(ctx, scores, batch, kept, out_len)
        ev[2].record()
        fb.finch_compact(ctx, kept, out_len, dev["cache_k"], dev["cache_v"], dev["cache_pos"], dev["chunk_k"],
                         dev["chunk_v"], dev["chunk_pos"], batch, out_k, out_v, out_pos)
        ev[3].record()
        torch.cuda.synchronize()
        phase += [ev[i].elapsed_time(ev[i + 1]) for i in range(3)]
    phase /= args.steps
    clocks = sampler.stop(t_begin, t_end)

    step_e2e()
    ms_e2e_local = timed(step_e2e, max(1, min(args.steps, 5)))
    ms_e2e, _ = aggregate_over_ranks(ms_e2e_local, counts["tokens"], world, "nccl")
    e = 4 if cfg.dtype == "f32" else 2
    h2d = sum(host[k].numel() * host[k].element_size() for k in ("q", "chunk_k", "chunk_v", "chunk_pos"))
    d2h = kept_host.numel() * 4 + len_host.numel() * 4
    fb.finch_ctx_destroy(ctx)
    document = document_loop(args, cfg, st, dev) if args.document and world == 1 else None
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    chunk_len = np.diff(st["chunk_off"]).astype(np.int64)
    n_cand = st["cache_len"].astype(np.int64) + chunk_len
    n_q = np.diff(st["q_off"]).astype(np.int64)
    exps = float((n_cand * n_q).sum()) * cfg.n_layers * cfg.n_q_heads   # logits per sweep
    if rank != 0:
        return None
    peak, peak_kind = peak_hbm()
    achieved = counts["contract_bytes"] / (ms_local * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic (seeded Gaussian / Student-t with planted keys)",
        "config": {"workload": f"{cfg.name}: {cfg.n_layers} layers x {cfg.n_q_heads}q/{cfg.n_kv_heads}kv heads, "
                               f"d{cfg.head_dim}, batch {cfg.batch}, {counts['tokens']} candidates per step, "
                               f"steady-state step (cache full)",
                   "l2": "inputs larger than L2 (K+V+outputs per step exceed 126 MB)" if
                   counts["contract_bytes"] > 2.5e8 else "working set fits L2 (latency-bound configuration)",
                   "replicas": "independent replicas, no collective"},
        "clocks": clocks,
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "ms_per_step": ms_e2e},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": TRAFFIC_BYTES.get(cfg.name) if cfg.n_layers == wl.CONFIGS[cfg.name].n_layers else None,
                     "peak_kind": f"of {peak_kind}",
                     "algorithmic_bytes_per_step": counts["contract_bytes"],
                     "kernel": "whole step (score + select + compact launches)"},
        "phases_ms": {"score": float(phase[0]), "select": float(phase[1]), "compact": float(phase[2])},
        # the scoring phase is bound by the exponentials (two sweeps, one exp2 per logit each), not by HBM
        "score_alu": {"bound": "alu", "unit": "Gexp2/s", "achieved": 2 * exps / (phase[0] * 1e-3) / 1e9,
                      "peak": MUFU_PER_CLK_PER_SM * sm_count * (clocks.get("sm_mhz") or 1965) * 1e6 / 1e9,
                      "note": "peak = 16 exp2/clk/SM x SMs x sampled SM clock"},
    }
    line["score_alu"]["frac"] = line["score_alu"]["achieved"] / line["score_alu"]["peak"]
    if document:
        line["document_loop"] = document
    return line


def document_loop(args, cfg: wl.Config, st: dict, dev: dict):
    """Secondary figure: the whole chunk loop of the configuration's documents (every full chunk, empty cache at
    the start), caches resident on the device, budgets by the chosen schedule.  The step-1 chunk's K/V stand in for
    every chunk's data (their distribution is the same); positions advance with the step."""
    import torch
    from paper_2408_00167_b200 import binding as fb
    from paper_2408_00167_b200 import document as doc
    reqs = cfg.requests
    n_steps = min(r.text_len // r.chunk for r in reqs)
    group_mode = cfg.group_mode if args.group_mode < 0 else args.group_mode
    if args.document == "paper":
        per_req = [doc.paper_budgets([r.chunk] * n_steps, sigma=r.text_len / r.budget, k=r.budget) for r in reqs]
    else:
        per_req = [doc.fixed_budgets(n_steps, r.budget) for r in reqs]
    drv = doc.DocumentCompressor(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                                 fb.FINCH_F32 if cfg.dtype == "f32" else fb.FINCH_BF16, [r.budget for r in reqs],
                                 max_prompt=max(r.n_q for r in reqs), max_chunk=max(r.chunk for r in reqs),
                                 group_mode=group_mode)
    chunk_off = st["chunk_off"]
    pos = [dev["chunk_pos"] + step * max(r.chunk for r in reqs) for step in range(n_steps)]

    def loop():
        drv.reset()
        for step in range(n_steps):
            drv.step(dev["q"], st["q_off"], dev["chunk_k"], dev["chunk_v"], pos[step], chunk_off,
                     [per_req[b][step] for b in range(len(reqs))])
    loop()
    assert drv.status() == 0
    reps = 5
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(reps):
        loop()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    assert drv.status() == 0
    drv.close()
    tokens = int(n_steps * np.diff(chunk_off).sum())
    return {"schedule": args.document, "group_mode": "per_layer" if group_mode == 1 else "per_kv_head", "steps": n_steps,
            "document_tokens": tokens, "ms": ms, "tokens_per_s": tokens / (ms * 1e-3),
            "final_cache": [int(r.budget) for r in reqs],
            "note": "whole chunk loop from an empty cache, device-resident caches; one chunk's data reused per step"}


def run_reference(args, cfg: wl.Config):
    """The oracle as it stands, on the host cores, on a bounded sample per step."""
    rank, _, world = dist_env()
    if rank != 0:
        return None
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_sample(cfg, target_s=0.0, max_layers=1)
    vals, secs = [], []
    for _ in range(max(1, min(args.steps, 3))):
        base, step_s = oracle_sample(cfg, target_s=0.0, max_layers=1)
        vals.append(base["value"])
        secs.append(step_s)
    base["value"] = statistics.median(vals)
    base["sample"] = f"1 of {cfg.n_layers} layers of {cfg.name} per step, scaled linearly to a whole step"
    return {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": world,
            "steps": len(vals), "warmup": min(args.warmup, 1), "ms_per_step": statistics.median(secs) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{cfg.name} (oracle, CPU)"}, "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="c3", choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="use only the first LAYERS layers (small profiling runs)")
    ap.add_argument("--document", default="", choices=["", "fixed", "paper"],
                    help="also time the whole chunk loop with this budget schedule (adds a document_loop object)")
    ap.add_argument("--group-mode", type=int, default=-1, choices=[-1, 0, 1],
                    help="selection groups of the document loop: 0 per KV head, 1 per layer (-1: the configuration's)")
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.config]
    if args.layers > 0:
        cfg = wl.scaled(cfg, n_layers=min(args.layers, cfg.n_layers))
    if args.impl == "reference":
        line = run_reference(args, cfg)
    else:
        line = run_ours(args, cfg)
        rank, _, world = dist_env()
        if line is not None and world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"], _ = oracle_sample(cfg)
    if line is not None:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
