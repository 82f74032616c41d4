#!/usr/bin/env python
"""Benchmark of the cached denoising step on one B200 (replicas on N GPUs).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llada8b] [--impl reference]

A "step" is one pass of the whole hot path over one batch: one denoising step
under the dLLM-Cache schedule (full / response-refresh / mixed / adaptive
partial, as the step index decides) followed by the low-confidence transition.
The default workload is the LLaDA-8B-shaped configuration: batch 1, prompt 512,
generation 256 in blocks of 32, 256 steps, K_p = 100, K_r = 6, rho = 0.25,
random-init bf16 weights, uniform random prompt ids (synthetic stand-in for the
paper's benchmark prompts).  `--steps K` times the first K steps of that
schedule (it wraps into a new generation after 256).

Prints ONE JSON line.  value = generated tokens/s with everything resident in
HBM; e2e = the same loop driven through host buffers (token state copied
host->device before and device->host after every step).  --impl reference
times the CPU oracle instead (host cores, bounded sample).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_06295_b200 import synth  # noqa: E402

METRIC = "generated tokens/s, cached denoising steps (dLLM-Cache schedule)"


def schedule_kind(k, K, Kp, Kr):
    rp = (k == K) or (k % Kp == 0)
    rr = (k == K) or (k % Kr == 0)
    return rp, rr, ("full" if rp and rr else "refresh" if rr else "mixed" if rp else "partial")


def block_plan(t, K, R, block_len):
    blocks = R // block_len
    spb = K // blocks
    blk = min(t // spb, blocks - 1)
    i = t - blk * spb
    return blk * block_len, block_len // spb + (1 if i < block_len % spb else 0)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs (read-only query)."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [r.split(",") for r in open(self.path).read().strip().splitlines() if r.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        sm, reasons = [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                out["sm_max_mhz"] = float(r[2])
            except ValueError:
                continue
            for nm, v in zip(names, r[5:9]):
                if v.strip().lower().startswith("active"):
                    reasons.add(nm)
        if sm:
            out["sm_mhz"] = float(np.median(sm))
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        return out


# ----------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ----------------------------------------------------------------------------------------------
def time_oracle(wl, budget_s: float, steps: int | None = None):
    """Times the oracle, as it stands, on the host cores on a bounded sample of
    the workload: the same widths, sequence lengths and schedule, but a
    2-layer model, float32 numpy; per-kind step times are extrapolated to the
    full depth as (t_kind - t_head) * T/2 + t_head, the LM head timed by
    calling the oracle's own projection on the same rows."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import dllm_oracle as O
    cores = len(os.sched_getaffinity(0))
    Tsample = 2
    cfg = wl.model.with_layers(Tsample)
    names = synth.tensor_names(cfg)
    with ThreadPoolExecutor(max_workers=min(8, cores)) as ex:
        w = dict(zip([n for n, _ in names], ex.map(lambda ns: synth.make_tensor(cfg, ns[0], ns[1]), names)))
    orc = O.DLLMOracle(cfg, w, wl.batch, wl.prompt_len, wl.gen_len, dtype=np.float32)
    orc.set_prompt(synth.make_prompt(cfg, wl.batch, wl.prompt_len))
    times = {}
    t_start = time.perf_counter()
    K = wl.steps
    order = []
    for k in range(K, 0, -1):          # first occurrence of each kind, in schedule order
        kind = schedule_kind(k, K, wl.Kp, wl.Kr)[2]
        if kind not in [o[1] for o in order]:
            order.append((k, kind))
    done_steps = 0
    for k, kind in order:
        rp, rr, _ = schedule_kind(k, K, wl.Kp, wl.Kr)
        t0 = time.perf_counter()
        r = orc.step(rp, rr, wl.rho)
        bs, nt = block_plan(K - k, K, wl.gen_len, wl.block_len)
        orc.remask(bs, wl.block_len, nt)
        times[kind] = time.perf_counter() - t0
        done_steps += 1
        if time.perf_counter() - t_start > budget_s and "partial" in times:
            break
    # LM head alone (the oracle's own projection + greedy estimate), to extrapolate depth correctly
    z = O.rmsnorm(r.hidden[0].astype(np.float32), w["norm_f"], cfg.rms_eps)
    t0 = time.perf_counter()
    for _ in range(wl.batch):
        lg = orc._lin(z, "lm_head", "lm_head")
        lg.argmax(-1)
        np.exp(lg - lg.max(-1, keepdims=True)).sum(-1)
    t_head = time.perf_counter() - t0
    T = wl.model.n_layers
    full_depth = {kind: max(t - t_head, 0.0) * (T / Tsample) + t_head for kind, t in times.items()}
    counts = {}
    n_steps = steps if steps is not None else K
    for i in range(n_steps):
        kind = schedule_kind(K - (i % K), K, wl.Kp, wl.Kr)[2]
        counts[kind] = counts.get(kind, 0) + 1
    fallback = full_depth.get("full", max(full_depth.values()))
    total = sum(c * full_depth.get(kind, fallback) for kind, c in counts.items())
    tokens = n_steps * wl.batch * wl.gen_len / K
    return {"tokens_per_s": tokens / total, "cores": cores, "ms_per_step": 1e3 * total / n_steps,
            "per_kind_s_full_depth": {k: round(v, 3) for k, v in full_depth.items()},
            "sample": (f"{Tsample}-layer model at full width ({cfg.d_model}/{cfg.d_ffn}/{cfg.vocab}), B={wl.batch} "
                       f"P={wl.prompt_len} R={wl.gen_len}, float32 numpy, one step of each kind "
                       f"({', '.join(times)}) + LM head timed separately, extrapolated to {T} layers over "
                       f"{n_steps} scheduled steps"),
            "cpu_seconds": round(time.perf_counter() - t_start, 1)}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    t = time_oracle(wl, budget_s=90.0, steps=args.steps)
    line = {"impl": "reference", "metric": METRIC, "value": t["tokens_per_s"], "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(wl, args),
            "cpu_baseline": {"value": t["tokens_per_s"], "unit": "tokens/s", "cores": t["cores"], "kind": "oracle",
                             "sample": t["sample"]},
            "e2e": {"value": t["tokens_per_s"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "per_kind_s": t["per_kind_s_full_depth"]}
    print(json.dumps(line), flush=True)


def aggregate_over_ranks(ms, ms_e2e, world, device):
    """Whole-job time = the slowest replica's device time (max over ranks)."""
    if world <= 1:
        return ms, ms_e2e
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms, ms_e2e], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0]), float(t[1])


def tokens_processed(steps, batch, gen_len, schedule_steps, world):
    """Units all replicas processed: each scheduled step unmasks gen_len / schedule_steps tokens per sequence."""
    return steps * batch * gen_len / schedule_steps * world


def workload_config(wl, args):
    c = wl.model
    return {"workload": f"{wl.name}: {c.n_layers} layers, d={c.d_model}, {c.n_heads}x{c.head_dim} heads "
                        f"({c.n_kv_heads} KV), FFN {c.d_ffn}, vocab {c.vocab}; batch {wl.batch}, prompt "
                        f"{wl.prompt_len}, generation {wl.gen_len} in blocks of {wl.block_len}, {wl.steps} steps",
            "Kp": wl.Kp, "Kr": wl.Kr, "rho": wl.rho, "k_round": "floor",
            "l2": "inputs larger than L2: every step streams all layer weights (>= 14 GB) through the 126 MB L2",
            "replicas": args.gpus}


# ----------------------------------------------------------------------------------------------
# one process per GPU
# ----------------------------------------------------------------------------------------------
def wants_spawn(gpus: int, impl: str, env) -> bool:
    """`--gpus N` given to a plain `python bench.py` (no launcher set WORLD_SIZE): this process starts the N ranks."""
    return gpus > 1 and impl != "reference" and "WORLD_SIZE" not in env


def spawn_ranks(n: int, argv, script=None) -> int:
    """Runs `script` (this file) as n ranks of one node, one per GPU, under torch.distributed.run, rendezvous on
    127.0.0.1 at a free port; returns the launcher's exit code.  Rank 0 prints the JSON line."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
           "127.0.0.1", "--master-port", str(port), script or os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


# ----------------------------------------------------------------------------------------------
# rooflines
# ----------------------------------------------------------------------------------------------
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}      # the figures the target is stated against
TENSOR_CLASSES = {"gemm", "attention", "gemm_v", "gemm_qk", "gemm_o", "gemm_gate_up", "gemm_down", "gemm_lm_head",
                  "attention_mma", "attention_tcgen05"}


def roofline_of(name, rec, peaks):
    """Binding roof of one class of launches from its algorithmic intensity against the ridge of the measured
    peaks (a projection with M activation rows has about M flop per byte): achieved and both fractions."""
    ms, by, fl, n = rec["ms"], rec["bytes"], rec["flops"], rec["launches"]
    if n == 0 or ms <= 0:
        return None
    ridge = peaks["bf16_tflops_sustained"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    tensor = name in TENSOR_CLASSES and by > 0 and fl / by > ridge
    gbs, tfl = by / (ms / 1e3) / 1e9, fl / (ms / 1e3) / 1e12
    out = {"launches": int(n), "avg_us": 1e3 * ms / n, "ms_total": ms, "bytes_per_launch": by / n,
           "flops_per_launch": fl / n, "gbs": gbs, "tflops": tfl, "bound": "tensor" if tensor else "hbm"}
    if tensor:
        out.update(achieved=tfl, unit="TFLOP/s", peak=peaks["bf16_tflops_sustained"],
                   frac=tfl / peaks["bf16_tflops_sustained"], frac_of_nominal=tfl / NOMINAL["bf16_tflops"])
    else:
        out.update(achieved=gbs, unit="GB/s", peak=peaks["hbm_gbs"], frac=gbs / peaks["hbm_gbs"],
                   frac_of_nominal=gbs / NOMINAL["hbm_gbs"])
    return out


def step_roof_ms(per_class, peaks):
    """Roofline time of one step: its launches run one after the other, each at its own binding roof."""
    hbm, tf = peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops_sustained"] * 1e12
    return 1e3 * sum(max(r["bytes"] / hbm, (r["flops"] / tf) if name in TENSOR_CLASSES else 0.0)
                     for name, r in per_class.items())


# dram__bytes_read.sum + dram__bytes_write.sum per projection launch, from an ncu capture of a two-layer case of
# the same kernel scaled to the full depth (every layer streams its own weights); None where no capture of the
# current kernel exists.
TRAFFIC_PER_LAUNCH = {"llada8b": 96.2e6}


# ----------------------------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llada8b", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--rho", type=float, default=None, help="update ratio of the adaptive steps (default: the workload's)")
    ap.add_argument("--rho-sweep", default=None, help="comma list of update ratios timed beside the headline "
                    "(default: 0.1,0.25,0.5 for the batched workload, none otherwise; 'none' to skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-timeline", action="store_true", help="skip the in-graph GEMM figure (a second process)")
    ap.add_argument("--prof-mode", default="graph", choices=["graph", "stream"], help="per-kernel event pairs as "
                    "event-record nodes of the step graphs, or recorded by the host around plain launches")
    ap.add_argument("--full-steps", type=int, default=6, help="timed full-recompute steps for the speedup figure")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (small case for ncu "
                    "captures: same widths, a few GB of weights); the bench line then names the reduced depth")
    ap.add_argument("--no-pdl", action="store_true", help="plain launches instead of programmatic dependent launch")
    ap.add_argument("--compact-cache", action="store_true", help="response-only AttnOut / FFNOut caches")
    ap.add_argument("--ncu-kinds", default="", help="comma list of step kinds (full,refresh,mixed,partial): after "
                    "warm-up run one step of each between cudaProfilerStart/Stop and exit (for "
                    "`ncu --profile-from-start off`); prints no bench line")
    args = ap.parse_args()
    from dataclasses import replace
    wl = synth.WORKLOADS[args.workload]
    if args.layers > 0:
        wl = replace(wl, name=f"{wl.name}-{args.layers}layers", model=wl.model.with_layers(args.layers))
    if args.rho is not None:
        wl = replace(wl, rho=args.rho)
    if args.impl == "reference":
        run_reference(args, wl)
        return
    if wants_spawn(args.gpus, args.impl, os.environ):
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))

    import torch
    import torch.distributed as dist
    from paper_2506_06295_b200 import build as build_mod
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank == 0:
        build_mod.build()
    if world > 1:
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    from paper_2506_06295_b200 import dllm
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    cfg = wl.model
    K, W = args.steps, max(args.warmup, 3)

    model = dllm.Model(cfg, device=dev).random_init_on_device(synth.WEIGHT_SEED + rank)
    ses = dllm.Session(model, wl.batch, wl.prompt_len, wl.gen_len, compact_cache=args.compact_cache)
    prompt = synth.make_prompt(cfg, wl.batch, wl.prompt_len, seed=1 + 1000 * rank)
    ses.set_prompt(prompt)
    if args.no_pdl:
        ses.use_pdl(False)
    stream = ses.stream

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    host_s = [0.0]   # host time spent in the step and transition calls (they only enqueue)

    def run_steps(n, per_step=None):
        for i in range(n):
            k = wl.steps - (i % wl.steps)
            if i and k == wl.steps:
                ses.set_prompt(prompt)          # a new generation starts (a blocking copy from pageable memory)
            t0 = time.perf_counter()
            ses.step_scheduled(k, wl.steps, wl.Kp, wl.Kr, wl.rho)
            bs, nt = block_plan(wl.steps - k, wl.steps, wl.gen_len, wl.block_len)
            ses.remask_low_confidence(bs, wl.block_len, nt)
            host_s[0] += time.perf_counter() - t0
            if per_step:
                per_step(i)

    # warm-up: every step kind W times (also instantiates the CUDA graphs)
    ses.step_full()
    for _ in range(W):
        for rp, rr in ((True, True), (True, False), (False, True), (False, False)):
            ses.step_cached(rp, rr, wl.rho)
    ses.sync()
    ses.set_prompt(prompt)

    if args.ncu_kinds:
        flags = {"full": (True, True), "refresh": (False, True), "mixed": (True, False), "partial": (False, False)}
        ses.step_full()
        ses.sync()
        torch.cuda.profiler.start()
        for kind in args.ncu_kinds.split(","):
            rp, rr = flags[kind]
            ses.step_cached(rp, rr, wl.rho)
            ses.remask_low_confidence(0, wl.block_len, 1)
        ses.sync()
        torch.cuda.profiler.stop()
        print(json.dumps({"ncu_window": args.ncu_kinds.split(","), "launches": ses.launch_count()}))
        return

    # ---- timed region: K steps, everything resident ------------------------------------------
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = ses.launch_count()
    torch.cuda.profiler.start()       # no-op unless a profiler waits for it (`ncu --profile-from-start off`)
    ev0.record(stream)
    host_s[0] = 0.0
    run_steps(K)
    host_enqueue_ms = 1e3 * host_s[0]    # the host only enqueues: it runs ahead of the device
    ev1.record(stream)
    barrier()
    torch.cuda.profiler.stop()
    ms = ev0.elapsed_time(ev1)
    launches = ses.launch_count() - l0
    ses.sync()
    final_tokens = ses.tokens()
    clocks = sampler.stop() if rank == 0 else None

    # ---- per-kind step times and the full-recompute baseline of the same library -------------
    KINDS = {"full": (True, True), "refresh": (False, True), "mixed": (True, False), "partial": (False, False)}

    def time_kind(rp, rr, reps, rho=None):
        rho = wl.rho if rho is None else rho
        ses.step_cached(rp, rr, rho)      # the graph of this (kind, rho) exists before the clock starts
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        a.record(stream)
        for _ in range(reps):
            ses.step_cached(rp, rr, rho)
        b.record(stream)
        torch.cuda.synchronize(dev)
        return a.elapsed_time(b) / reps
    reps = {"full": args.full_steps, "refresh": 16, "mixed": 6, "partial": 16}
    per_kind = {kind: time_kind(*KINDS[kind], reps[kind]) for kind in KINDS}

    def schedule_counts(n_steps):
        counts = {}
        for i in range(n_steps):
            kind = schedule_kind(wl.steps - (i % wl.steps), wl.steps, wl.Kp, wl.Kr)[2]
            counts[kind] = counts.get(kind, 0) + 1
        return counts

    # ---- update-ratio sweep (Fig. 8: throughput against rho), the full-recompute step beside it ------
    sweep = args.rho_sweep if args.rho_sweep is not None else ("0.1,0.25,0.5" if wl.batch > 1 else "none")
    rho_sweep = None
    if sweep != "none":
        rho_sweep = {"full_recompute_ms": per_kind["full"], "refresh_ms": per_kind["refresh"], "points": []}
        whole = schedule_counts(wl.steps)
        for rho in [float(v) for v in sweep.split(",")]:
            t_partial, t_mixed = time_kind(False, False, 8, rho), time_kind(True, False, 3, rho)
            total_ms = (whole.get("full", 0) * per_kind["full"] + whole.get("refresh", 0) * per_kind["refresh"] +
                        whole.get("mixed", 0) * t_mixed + whole.get("partial", 0) * t_partial)
            rho_sweep["points"].append({
                "rho": rho, "partial_ms": t_partial, "mixed_ms": t_mixed,
                "schedule_tokens_per_s": wl.batch * wl.gen_len / (total_ms / 1e3),
                "speedup_vs_full_recompute": wl.steps * per_kind["full"] / total_ms})
        rho_sweep["how"] = ("per-kind step times (CUDA events over graph replays) weighted by the step kinds of the "
                            f"whole {wl.steps}-step schedule; transition launches not included")

    # ---- the same schedule with the prediction restricted to the block each step works on -------
    # (reported beside the headline, never as it: the headline step predicts every response row)
    ses.set_prompt(prompt)
    for k in (wl.steps, wl.steps - 1, wl.steps - 2):        # graphs of the step kinds with a block head
        ses.step_scheduled_block(k, wl.steps, wl.Kp, wl.Kr, wl.rho, 0, wl.block_len)
    ses.set_prompt(prompt)
    barrier()
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b0.record(stream)
    for i in range(K):
        k = wl.steps - (i % wl.steps)
        if i and k == wl.steps:
            ses.set_prompt(prompt)
        bs, nt = block_plan(wl.steps - k, wl.steps, wl.gen_len, wl.block_len)
        ses.step_scheduled_block(k, wl.steps, wl.Kp, wl.Kr, wl.rho, bs, wl.block_len)
        ses.remask_low_confidence(bs, wl.block_len, nt)
    b1.record(stream)
    barrier()
    ms_block = b0.elapsed_time(b1)
    block_tokens = ses.tokens()

    # ---- end to end through host buffers ---------------------------------------------------------
    ses.set_prompt(prompt)
    host_tok = torch.empty((wl.batch, wl.gen_len), dtype=torch.int32).pin_memory()
    host_tok.fill_(cfg.mask_id)
    host_np = host_tok.numpy()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(K):
        k = wl.steps - (i % wl.steps)
        if i and k == wl.steps:
            ses.set_prompt(prompt)
            host_np[...] = cfg.mask_id
        ses.set_response_tokens(host_np)                    # host -> device: this step's token state
        ses.step_scheduled(k, wl.steps, wl.Kp, wl.Kr, wl.rho)
        bs, nt = block_plan(wl.steps - k, wl.steps, wl.gen_len, wl.block_len)
        ses.remask_low_confidence(bs, wl.block_len, nt)
        host_np[...] = ses.tokens()[:, wl.prompt_len:]      # device -> host: the step's result
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)

    # ---- per-kernel times: the same K steps with an event pair around every launch.  The pairs are event-record
    # nodes of each step's graph (or host records around plain launches with --prof-mode stream); launches are
    # serialised and carry no programmatic overlap; each step ends with a synchronisation that reads them back, so
    # the replay's own time is the sum of per-step event pairs, not a span that would include those host gaps.
    if args.prof_mode == "stream":
        ses.use_graphs(False)
    ses.set_prompt(prompt)
    ses.profile(True)
    for k in (wl.steps, wl.steps - 1, wl.steps - 2):        # instantiate the profiling graphs outside the replay
        ses.step_scheduled(k, wl.steps, wl.Kp, wl.Kr, wl.rho)
    ses.profile(False)
    ses.set_prompt(prompt)
    ses.profile(True)
    step_ev = []
    for i in range(K):
        k = wl.steps - (i % wl.steps)
        if i and k == wl.steps:
            ses.set_prompt(prompt)
        a = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ses.step_scheduled(k, wl.steps, wl.Kp, wl.Kr, wl.rho)
        bs, nt = block_plan(wl.steps - k, wl.steps, wl.gen_len, wl.block_len)
        ses.remask_low_confidence(bs, wl.block_len, nt)
        b = torch.cuda.Event(enable_timing=True)
        b.record(stream)
        step_ev.append((a, b))
        if args.prof_mode == "stream" and i % 8 == 7:
            ses.sync()
    ses.sync()
    ms_replay = sum(a.elapsed_time(b) for a, b in step_ev)
    prof = {name: ses.profile_read(i) for i, name in enumerate(dllm.PROF_CLASSES)}
    ses.profile(False)

    # algorithmic bytes / FLOPs of ONE step of each kind (the library's own count), for the per-step fractions
    # and the in-graph figure
    per_kind_work = {}
    for kind, (rp, rr) in KINDS.items():
        ses.profile(True)
        ses.step_cached(rp, rr, wl.rho)
        ses.sync()
        per_kind_work[kind] = {name: ses.profile_read(i) for i, name in enumerate(dllm.PROF_CLASSES[2:], 2)}
        ses.profile(False)
    ses.use_graphs(True)
    partial_gemm_bytes = sum(v["bytes"] for k_, v in per_kind_work["partial"].items() if k_.startswith("gemm"))
    partial_gemm_flops = sum(v["flops"] for k_, v in per_kind_work["partial"].items() if k_.startswith("gemm"))

    # max over ranks
    ms, ms_e2e = aggregate_over_ranks(ms, ms_e2e, world, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    tokens = tokens_processed(K, wl.batch, wl.gen_len, wl.steps, world)
    value = tokens / (ms / 1e3)
    kernels = {name: roofline_of(name, rec, peaks) for name, rec in prof.items()}
    kernels = {k_: v for k_, v in kernels.items() if v is not None}
    # share of the summed event time of all launches ("gemm" and "attention" are sums of classes listed beside
    # them): the figure to hold against the share column of a profiler's launch list of the same command
    kernel_ms = sum(v["ms_total"] for k_, v in kernels.items() if k_ not in ("gemm", "attention"))
    for v in kernels.values():
        v["share_of_kernel_time"] = v["ms_total"] / max(kernel_ms, 1e-9)
    g = kernels["gemm"]
    steps_roof = {}
    for kind, work in per_kind_work.items():
        roof = step_roof_ms(work, peaks)
        steps_roof[kind] = {"ms": per_kind[kind], "roofline_ms": roof, "frac": roof / per_kind[kind],
                            "algorithmic_gb": sum(v["bytes"] for v in work.values()) / 1e9,
                            "algorithmic_tflop": sum(v["flops"] for v in work.values()) / 1e12}
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": workload_config(wl, args),
        "steps_per_s": K * world / (ms / 1e3),
        "step_kinds": schedule_counts(K),
        "ms_per_kind": {k_: round(v, 4) for k_, v in per_kind.items()},
        "speedup_vs_full_recompute": per_kind["full"] / (ms / K),
        "full_recompute_tokens_per_s": wl.batch * wl.gen_len / wl.steps * world / (per_kind["full"] / 1e3),
        "e2e": {"value": tokens / (ms_e2e / 1e3), "unit": "tokens/s",
                "h2d_bytes_per_step": wl.batch * wl.gen_len * 4, "d2h_bytes_per_step": wl.batch * (wl.prompt_len + wl.gen_len) * 4},
        "block_only_prediction": {"value": tokens / (ms_block / 1e3), "unit": "tokens/s", "ms_per_step": ms_block / K,
                                  "same_tokens_as_headline_run": bool((block_tokens == final_tokens).all()),
                                  "what": "dllm_step_scheduled_block: logits, estimate and confidence only for the "
                                          "block the step works on; layers and caches identical"},
        "gpu_launches": int(launches),
        "host_enqueue_ms_per_step": host_enqueue_ms / K,
        "clocks": clocks,
        "roofline": {"kernel": "gemm_bf16_tcgen05_kernel / gemm_bf16_pair_kernel (all projections of the timed steps)",
                     "bound": g["bound"], "achieved": g["achieved"], "peak": g["peak"], "unit": g["unit"],
                     "frac": g["frac"], "frac_of_nominal": g["frac_of_nominal"],
                     "nominal_peak": NOMINAL["bf16_tflops"] if g["bound"] == "tensor" else NOMINAL["hbm_gbs"],
                     "peak_source": peaks["source"] + (" (sustained bf16)" if g["bound"] == "tensor" else " (copy)"),
                     "traffic": TRAFFIC_PER_LAUNCH.get(args.workload) if not args.layers else None,
                     "launches": g["launches"], "avg_launch_us": g["avg_us"],
                     "algorithmic_bytes_per_launch": g["bytes_per_launch"],
                     "algorithmic_flops_per_launch": g["flops_per_launch"],
                     "gemm_share_of_step": g["ms_total"] / max(ms_replay, 1e-9),
                     "gemm_share_of_kernel_time": g["share_of_kernel_time"],
                     "how": "CUDA-event pairs around every launch (" +
                            ("event-record nodes in the step graphs" if args.prof_mode == "graph" else
                             "host records around plain launches") +
                            ", launches serialised, no programmatic overlap) in a replay of the same K steps; "
                            "share = event time of the class / summed per-step event time of that replay; the "
                            "binding roof of a class follows from its algorithmic flop per byte against the ridge "
                            "of the measured peaks"},
        "kernels": kernels,
        "steps_roofline": steps_roof,
        "unmasked_tokens": int((final_tokens[:, wl.prompt_len:] != cfg.mask_id).sum()),
    }
    if rho_sweep is not None:
        line["rho_sweep"] = rho_sweep
    if args.compact_cache:
        line["config"]["cache"] = "response-only AttnOut / FFNOut"
    line["cache_bytes"] = int(ses.cache.numel())
    if world == 1 and not args.no_timeline and not args.layers and args.rho is None:
        line["roofline"]["in_graph"] = in_graph_gemm(args.workload, partial_gemm_bytes, partial_gemm_flops,
                                                     line["roofline"]["bound"], peaks)
    if not args.no_cpu_baseline:
        t = time_oracle(wl, budget_s=25.0, steps=K)
        line["cpu_baseline"] = {"value": t["tokens_per_s"], "unit": "tokens/s", "cores": t["cores"], "kind": "oracle",
                                "sample": t["sample"]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def in_graph_gemm(workload, gemm_bytes, gemm_flops, bound, peaks):
    """GEMM time INSIDE the replayed graph of one adaptive partial step (programmatic dependent launch, warm L2),
    from the device timestamps of the timeline build, in a process of its own after this one has freed nothing it
    needs: achieved = the step's algorithmic GEMM bytes (flops where the class is tensor bound) / the summed
    in-graph durations of its GEMM launches.  Reported beside the event-pair figure, which serialises the
    launches.  None if the run fails."""
    try:
        with tempfile.TemporaryDirectory() as td:
            out = os.path.join(td, "tl.json")
            r = subprocess.run([sys.executable, "-m", "paper_2506_06295_b200.timeline", "--workload", workload,
                                "--kind", "partial", "--no-marks", "--json", out], cwd=ROOT, capture_output=True,
                               text=True, timeout=600)
            if r.returncode != 0:
                return None
            launches = json.load(open(out))
        gemm = [o for o in launches if o["file"].startswith("gemm")]
        us = sum(o["dur_us"] for o in gemm)
        total = launches[-1]["start_us"]
        if bound == "tensor":
            ach, unit, peak, nominal = gemm_flops / (us * 1e-6) / 1e12, "TFLOP/s", peaks["bf16_tflops_sustained"], NOMINAL["bf16_tflops"]
        else:
            ach, unit, peak, nominal = gemm_bytes / (us * 1e-6) / 1e9, "GB/s", peaks["hbm_gbs"], NOMINAL["hbm_gbs"]
        return {"achieved": ach, "unit": unit, "frac": ach / peak,
                "frac_of_nominal": ach / nominal, "gemm_us": us, "gemm_launches": len(gemm),
                "step_us": total, "gemm_share_of_step": us / max(total, 1e-9),
                "how": "one adaptive partial step replayed as a CUDA graph in the timeline build of the library: "
                       "per launch, device time from its predecessor's completion to its own (globaltimer at "
                       "griddepcontrol.wait of every CTA)"}
    except Exception:
        return None


if __name__ == "__main__":
    main()
