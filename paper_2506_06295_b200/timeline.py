"""In-graph timeline of one denoising step, from device timestamps.

    python -m paper_2506_06295_b200.timeline [--workload llada8b] [--kind partial] [--layer 5] [--json out.json]

Builds the timeline variant of the library (libdllm_b200_timeline.so: the same
kernels, each CTA recording the global timer before and after its dependency
wait), replays the CUDA graph of one step of the chosen kind (full, refresh,
mixed, partial) and prints, per kernel launch, the time from the moment its
predecessor had completed to the moment it had completed itself.  Inside a
replayed graph with programmatic dependent launch this is what a kernel costs
the step; event pairs around single launches and profiler runs (serialised,
cold caches) both overstate it.

The timeline library is a separate build; the product library carries no
instrumentation.
"""
from __future__ import annotations

import argparse
import collections
import ctypes as C
import json
import os
import sys

STEMS = ["elementwise", "gemm_simt", "gemm_tcgen05", "attention", "attention_umma"]
KINDS = {"full": (True, True), "refresh": (False, True), "mixed": (True, False), "partial": (False, False)}
RECORD_CAP = 1 << 20


def collect(workload: str, kind: str, marks: bool = True):
    """Runs one step and returns the launches in completion order: dicts with file, grid, block, ctas,
    start_us (predecessor complete), resident_before_us, last_cta_us, dur_us.  marks=False: the marks inside
    the kernels are not recorded (they slow the projections down by several percent)."""
    from . import build as build_mod
    os.environ["DLLM_B200_LIB"] = build_mod.build(timeline=True)
    import torch
    from . import dllm, synth
    wl = synth.WORKLOADS[workload]
    cfg = wl.model
    model = dllm.Model(cfg).random_init_on_device(synth.WEIGHT_SEED)
    ses = dllm.Session(model, wl.batch, wl.prompt_len, wl.gen_len)
    ses.set_prompt(synth.make_prompt(cfg, wl.batch, wl.prompt_len, seed=1))
    rp, rr = KINDS[kind]
    ses.step_full()
    for _ in range(4):      # the graph of this step kind exists and is warm
        ses.step_cached(rp, rr, wl.rho)
    ses.sync()
    bufs = {}
    for st in STEMS:
        setter = getattr(dllm.lib, "dllm_timeline_set_" + st)
        setter.argtypes, setter.restype = [C.c_void_p], C.c_int
        getattr(dllm.lib, "dllm_timeline_count_" + st).restype = C.c_uint
        bufs[st] = torch.zeros(RECORD_CAP * 4, dtype=torch.int64, device=model.device)
        if setter(C.c_void_p(bufs[st].data_ptr())) != 0:
            raise RuntimeError("could not arm the timeline of " + st)
        if getattr(dllm.lib, "dllm_timeline_marks_" + st)(1 if marks else 0) != 0:
            raise RuntimeError("could not switch the marks of " + st)
    torch.cuda.synchronize()
    ses.step_cached(rp, rr, wl.rho)
    ses.sync()
    recs = []
    truncated = False
    for st in STEMS:
        n = getattr(dllm.lib, "dllm_timeline_count_" + st)()
        truncated |= n >= RECORD_CAP
        a = bufs[st].cpu().numpy().reshape(-1, 4)[:n]
        recs += [(int(t1), int(t0), int(tag), st) for tag, t0, t1, _ in a]
        getattr(dllm.lib, "dllm_timeline_set_" + st)(None)
    marks = [r for r in recs if (r[2] >> 60)]
    recs = [r for r in recs if not (r[2] >> 60)]
    recs.sort()
    # CTAs of one launch share (file, grid, block) and are released together; later waves of a large grid are
    # released as earlier CTAs exit, so a gap is allowed inside a launch as long as the signature stays
    launches = []
    for t1, t0, tag, st in recs:
        key = (st, tag)
        size = (tag & 0xffff) * ((tag >> 16) & 0xffff) * ((tag >> 32) & 0xffff)
        if launches and launches[-1]["key"] == key and launches[-1]["n"] < size:
            L = launches[-1]
            L["t0min"], L["t0max"], L["n"] = min(L["t0min"], t0), max(L["t0max"], t0), L["n"] + 1
        else:
            launches.append({"key": key, "t1": t1, "t0min": t0, "t0max": t0, "n": 1})
    base = launches[0]["t1"]
    out = []
    for i, L in enumerate(launches):
        st, tag = L["key"]
        nxt = launches[i + 1]["t1"] if i + 1 < len(launches) else None
        out.append({"file": st, "grid": [tag & 0xffff, (tag >> 16) & 0xffff, (tag >> 32) & 0xffff], "block": tag >> 48,
                    "ctas": L["n"], "start_us": (L["t1"] - base) / 1e3,
                    "resident_before_us": (L["t1"] - L["t0min"]) / 1e3, "last_cta_us": (L["t0max"] - L["t1"]) / 1e3,
                    "dur_us": (nxt - L["t1"]) / 1e3 if nxt is not None else 0.0})
    # marks inside kernels: time after the release of the launch they belong to (same signature, latest release before)
    sig = lambda tag: tag & ((1 << 60) - 1)
    for t1, _t0, tag, st in marks:
        cands = [L for L in launches if L["key"][0] == st and (L["key"][1] & ((1 << 60) - 1)) == sig(tag) and L["t1"] <= t1]
        if cands:
            cands[-1].setdefault("marks", {}).setdefault(tag >> 60, []).append((t1 - cands[-1]["t1"]) / 1e3)
    for o, L in zip(out, launches):
        if "marks" in L:
            o["marks"] = {int(k): [min(v), sum(v) / len(v), max(v)] for k, v in sorted(L["marks"].items())}
    return out, cfg.n_layers, truncated


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--workload", default="llada8b")
    ap.add_argument("--kind", default="partial", choices=sorted(KINDS))
    ap.add_argument("--layer", type=int, default=5, help="layer whose launches are listed one by one")
    ap.add_argument("--json", default=None, help="write every launch to this file")
    ap.add_argument("--no-marks", action="store_true", help="record the launches only, not the marks inside kernels")
    args = ap.parse_args(argv)
    out, n_layers, truncated = collect(args.workload, args.kind, marks=not args.no_marks)
    if args.json:
        with open(args.json, "w") as f:
            json.dump(out, f)
    total = out[-1]["start_us"]
    print(f"{args.workload}, {args.kind} step: {len(out)} launches, {total:.1f} us from the first release to the last"
          + (" (record arrays overflowed: totals are low)" if truncated else ""))
    # launches of one layer: the step starts with one launch (embedding), then n_layers equal groups, then the
    # LM head and the estimate
    per = max(1, (len(out) - 3) // n_layers)
    lo = 1 + args.layer * per
    if not truncated and 0 <= args.layer < n_layers and lo + per < len(out):
        print(f"layer {args.layer} ({per} launches, {out[lo + per]['start_us'] - out[lo]['start_us']:.1f} us):")
        for o in out[lo:lo + per]:
            print(f"  {o['file']:15s} grid {str(tuple(o['grid'])):16s} x {o['block']:4d}  ctas {o['ctas']:5d}  "
                  f"dur {o['dur_us']:8.2f} us  resident {o['resident_before_us']:7.2f} us before release, "
                  f"last CTA in {o['last_cta_us']:+.2f} us")
            for k, (lo_, av, hi) in o.get("marks", {}).items():
                print(f"      mark {k}: min {lo_:6.2f}  mean {av:6.2f}  max {hi:6.2f} us after the release")
    agg = collections.OrderedDict()
    for o in out:
        a = agg.setdefault((o["file"], tuple(o["grid"]), o["block"]), [0, 0.0])
        a[0] += 1
        a[1] += o["dur_us"]
    print("by kernel signature (file, grid, block):")
    for (st, grid, blk), (n, us) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
        print(f"  {st:15s} {str(grid):18s} x {blk:4d}  launches {n:5d}  total {us:10.1f} us  avg {us / n:8.2f}  "
              f"share {100 * us / max(total, 1e-9):5.1f}%")
    return 0


if __name__ == "__main__":
    sys.exit(main())
