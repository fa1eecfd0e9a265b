#!/usr/bin/env python
"""Benchmark of the fused Finch step (score + select + compact) on synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c3] [--impl ours|reference]

One "step" is one steady-state finch_step over all layers of the configuration (cache full, one new chunk).
Prints ONE JSON line: candidate KV tokens/s (whole job), ms per step, the HBM roofline of the step, an end-to-end
figure with host buffers, and the fp64 CPU oracle timed on a bounded sample of the same workload.
The timed region is BLOCKS blocks of K steps each (K = --steps), every block bracketed by a barrier and a device
synchronisation; ms_per_step is the median block's time / K.  Steps alternate between two complete sets of input
and output buffers.
With N > 1 every rank runs an independent replica (no data-path collective): under torchrun the ranks come from the
environment; started directly, `--gpus N` spawns the N ranks itself, one process per GPU.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
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
MUFU_PER_CLK_PER_SM = 16   # exp2 results per clock per SM (4 per scheduler); profiles/exp2_rate.txt
BLOCKS = 25                # timed blocks of --steps steps each; the median block is reported
BUFFER_SETS = 2            # complete input/output buffer sets the steps alternate between
TRAFFIC_FILE = ROOT / "profiles" / "dram_traffic.txt"


def kernel_sources_digest() -> str:
    """SHA-256 over the CUDA sources of the library (names and contents): identifies the kernels a profile was
    taken on, also where no git history is at hand."""
    h = hashlib.sha256()
    csrc = ROOT / "paper_2408_00167_b200" / "csrc"
    for p in sorted(list(csrc.glob("*.cu")) + list(csrc.glob("*.cuh"))):
        h.update(p.name.encode())
        h.update(p.read_bytes())
    return h.hexdigest()


def recorded_traffic(config: str):
    """DRAM bytes (read + write) of one full step of `config` as ncu counted them, from profiles/dram_traffic.txt --
    or None when the file has no entry for the configuration or was captured on other kernel sources.
    Line format:  <config> <bytes per step> <sha256 of the kernel sources> [# comment]"""
    if not TRAFFIC_FILE.exists():
        return None
    digest = kernel_sources_digest()
    for line in TRAFFIC_FILE.read_text().splitlines():
        f = line.split("#")[0].split()
        if len(f) >= 3 and f[0] == config and f[2] == digest:
            return int(f[1])
    return None


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
        import tempfile
        try:
            # into a file, not a pipe: nobody reads before stop(), and a full pipe would stall the sampler for the
            # rest of a long run (its later samples, those of the timed steps, would be missing)
            self.out = tempfile.TemporaryFile(mode="w+")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.out, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self, t_begin: float, t_end: float) -> dict:
        """Summary of the samples taken between the two time.time() stamps (all samples if none fall inside)."""
        import datetime
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            self.proc.wait()
        self.out.seek(0)
        out = self.out.read()
        self.out.close()
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


def launch_replicas(n: int, argv: list, extra_env: dict = None) -> int:
    """Start n ranks of `argv` (a python command line without the interpreter) on this node, one process per GPU,
    with RANK / LOCAL_RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT set as torchrun would; rank 0 inherits stdout.
    Waits for all of them; if one fails the others are terminated (by their own PIDs).  Returns the worst exit code."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), **(extra_env or {}))
        procs.append(subprocess.Popen([sys.executable, *argv], env=env,
                                      stdout=None if rank == 0 else subprocess.DEVNULL))
    worst, pending = 0, set(range(n))
    while pending:
        for rank in sorted(pending):
            rc = procs[rank].poll()
            if rc is None:
                continue
            pending.discard(rank)
            worst = max(worst, abs(rc))
            if rc != 0:                      # a failed rank would leave the others waiting at a barrier
                for other in pending:
                    procs[other].terminate()
        time.sleep(0.05)
    return worst


def oracle_sample(cfg: wl.Config, target_s: float = 12.0, max_layers: int = 32, threads: int = 0):
    """Time the fp64 oracle's whole step on whole layers of the same workload until about target_s of CPU work."""
    import oracle
    threads = threads or oracle.max_threads()
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
    batch = fb.make_batch(st["q_off"], st["chunk_off"], st["cache_off"], st["cache_len"], st["budget"])
    c = batch.c
    ctx = fb.finch_ctx_create(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                              fb.FINCH_F32 if cfg.dtype == "f32" else fb.FINCH_BF16, cfg.group_mode,
                              max_batch=cfg.batch, max_prompt=c.max_q, max_candidates=c.max_cache + c.max_chunk,
                              device=local_rank)
    G = cfg.n_groups

    def buffer_set():
        d = {k: v.cuda(non_blocking=True) for k, v in host.items()}
        d["out_k"], d["out_v"] = torch.empty_like(d["cache_k"]), torch.empty_like(d["cache_v"])
        d["out_pos"] = torch.empty((cfg.n_layers, G, c.total_cache), dtype=torch.int32, device="cuda")
        d["kept"] = torch.empty((cfg.n_layers, G, c.total_cache), dtype=torch.int32, device="cuda")
        d["out_len"] = torch.empty(cfg.batch, dtype=torch.int32, device="cuda")
        d["scores"] = torch.empty((cfg.n_layers, G, c.total_cache + c.total_chunk), dtype=torch.float32, device="cuda")
        return d
    # consecutive steps work on different buffers: nothing a step reads or writes is left in L2 by the step before
    sets = [buffer_set() for _ in range(BUFFER_SETS)]
    dev = sets[0]
    ws = torch.empty(fb.finch_workspace_bytes(ctx, batch), dtype=torch.uint8, device="cuda")
    kept_host = torch.empty_like(dev["kept"], device="cpu").pin_memory()
    len_host = torch.empty_like(dev["out_len"], device="cpu").pin_memory()
    turn = [0]

    def step():
        d = sets[turn[0] % BUFFER_SETS]
        turn[0] += 1
        fb.finch_step(ctx, d["q"], d["cache_k"], d["cache_v"], d["cache_pos"], d["chunk_k"], d["chunk_v"],
                      d["chunk_pos"], batch, d["out_k"], d["out_v"], d["out_pos"], d["kept"], d["out_len"],
                      d["scores"], ws)

    def step_e2e():
        # this step's inputs come from pinned host memory through the C ABI's host-buffer call; the cache is
        # carried on the device; the kept positions and lengths come back to the host
        fb.finch_step_host(ctx, host["q"], host["chunk_k"], host["chunk_v"], host["chunk_pos"], dev["q"],
                           dev["chunk_k"], dev["chunk_v"], dev["chunk_pos"], dev["cache_k"], dev["cache_v"],
                           dev["cache_pos"], batch, dev["out_k"], dev["out_v"], dev["out_pos"], dev["kept"],
                           dev["out_len"], kept_host, len_host, ws)

    def timed(fn, n):
        """n calls of fn between two events, with a barrier and a device synchronisation on both sides."""
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
    block_ms = [timed(step, args.steps) for _ in range(max(1, args.blocks))]
    t_end = time.time()
    launches = (fb.finch_launch_count(ctx) - launches0) // max(1, args.blocks)   # per block of --steps steps
    assert fb.finch_device_status(ctx) == 0
    ms_local = statistics.median(block_ms)
    ms, tokens = aggregate_over_ranks(ms_local, counts["tokens"], world, "nccl")
    clocks = sampler.stop(t_begin, t_end)

    # per-phase durations (same kernels, called through the three separate entry points)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    phase = np.zeros(3)
    for i in range(args.steps):
        d = sets[i % BUFFER_SETS]
        ev[0].record()
        fb.finch_score(ctx, d["q"], d["cache_k"], d["chunk_k"], batch, d["scores"], None, ws)
        ev[1].record()
        fb.finch_select(ctx, d["scores"], batch, d["kept"], d["out_len"])
        ev[2].record()
        fb.finch_compact(ctx, d["kept"], d["out_len"], d["cache_k"], d["cache_v"], d["cache_pos"], d["chunk_k"],
                         d["chunk_v"], d["chunk_pos"], batch, d["out_k"], d["out_v"], d["out_pos"])
        ev[3].record()
        torch.cuda.synchronize()
        phase += [ev[i].elapsed_time(ev[i + 1]) for i in range(3)]
    phase /= args.steps

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
        "timing": {"blocks": max(1, args.blocks), "steps_per_block": args.steps, "statistic": "median block / steps",
                   "block_ms_min": min(block_ms), "block_ms_max": max(block_ms),
                   # time x clock: comparable between runs that saw different SM clocks
                   "kclk_per_step": ms_local * clocks["sm_mhz"] if clocks.get("sm_mhz") else None},
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic (seeded Gaussian / Student-t with planted keys)",
        "config": {"workload": f"{cfg.name}: {cfg.n_layers} layers x {cfg.n_q_heads}q/{cfg.n_kv_heads}kv heads, "
                               f"d{cfg.head_dim}, batch {cfg.batch}, {counts['tokens']} candidates per step, "
                               f"steady-state step (cache full)",
                   "l2": (f"steps alternate between {BUFFER_SETS} complete buffer sets; " +
                          ("inputs larger than L2 (K+V+outputs per step exceed 126 MB)" if
                           counts["contract_bytes"] > 2.5e8 else "one set fits L2 (latency-bound configuration)")),
                   "replicas": "independent replicas, no collective"},
        "clocks": clocks,
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "ms_per_step": ms_e2e},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     # ncu's DRAM bytes of one step, only if they were captured on exactly these kernel sources
                     "traffic": recorded_traffic(cfg.name) if cfg.n_layers == wl.CONFIGS[cfg.name].n_layers else None,
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
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="c3", choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="use only the first LAYERS layers (small profiling runs)")
    ap.add_argument("--blocks", type=int, default=BLOCKS, help="timed blocks of --steps steps (fewer for profiling runs)")
    ap.add_argument("--document", default="", choices=["", "fixed", "paper"],
                    help="also time the whole chunk loop with this budget schedule (adds a document_loop object)")
    ap.add_argument("--group-mode", type=int, default=-1, choices=[-1, 0, 1],
                    help="selection groups of the document loop: 0 per KV head, 1 per layer (-1: the configuration's)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # started directly rather than by torchrun: be the launcher of the N replicas
        sys.exit(launch_replicas(args.gpus, [str(Path(__file__).resolve()), *sys.argv[1:]]))
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
            one, _ = oracle_sample(cfg, target_s=0.0, max_layers=1, threads=1)
            line["cpu_baseline"]["single_thread"] = {"value": one["value"], "unit": UNIT, "cores": 1,
                                                     "sample": one["sample"]}
    if line is not None:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
