#!/usr/bin/env python
"""Benchmark of the ERASE training step on B200: tokens/s (samples/s) of the early-backward
schedule against the serial schedule of the same kernels, on synthetic data.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C4] [--impl reference] [--no-table]

One JSON line on stdout (rank 0).  A "step" is one pass of the whole hot path over one batch:
input staging, every block's forward + local loss, every block's backward, the optimizer.
The headline workload (`value`) is C4, the largest single-GPU configuration; the same line
carries, under `per_config`, the serial and ERASE throughput, gain, MFU and dominant kernel class
of C1, C2, C3 and five points of the C5 saturation sweep (N = 1 only).
With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the
workload on its own GPU (the path has no exchange step on one node: "replicas only"); the value
is the units all ranks processed divided by the slowest rank's time.
"""
import argparse
import atexit
import gc
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_18469_b200 import synth  # noqa: E402

POOL = 8            # distinct pre-staged batches, cycled
MIN_LEG_S = 1.0     # every leg is repeated (K steps per repeat) until this much device time is timed

# dram__bytes_read.sum + dram__bytes_write.sum per launch from ncu captures of the largest member
# of each kernel class (summaries under profiles/).  They sit below the algorithmic bytes where an
# operand or result is still L2-resident.
NCU_DRAM_BYTES = {"C2": {"gemm_fwd": 15.5e6, "gemm_dgrad": 75.4e6, "gemm_wgrad": 71.4e6},
                  "C4": {"gemm_fwd": 565.4e6, "gemm_dgrad": 710.9e6, "gemm_wgrad": 736.5e6}}

# the per-config table of the default run: (label, config name, keyword arguments)
TABLE = [("C1", "C1", {}), ("C2", "C2", {}), ("C3", "C3", {}),
         ("C5 w128 b512", "C5", {"w": 128, "batch": 512}),
         ("C5 w512 b4096", "C5", {"w": 512, "batch": 4096}),
         ("C5 w1024 b32768", "C5", {"w": 1024, "batch": 32768}),
         ("C5 w2048 b4096", "C5", {"w": 2048, "batch": 4096}),
         ("C5 w4096 b4096", "C5", {"w": 4096, "batch": 4096})]


def unit_name(spec):
    return "tokens/s" if spec["input"] == "tokens" else "samples/s"


def units_per_step(spec):
    return spec["batch"] * (spec["seq"] if spec["input"] == "tokens" else 1)


def workload_name(name, spec):
    nb = len(spec["blocks"])
    if spec["input"] == "tokens":
        blk = spec["blocks"][0]
        return (f"{name} LM proxy: {nb} detached pre-LN transformer blocks d{blk['dims'][0]} h{blk['n_heads']} "
                f"ff{blk['dims'][1]} T{spec['seq']} batch{spec['batch']} vocab{spec['vocab']}, local CE heads, AdamW, bf16")
    if spec["input"] == "ctr":
        return f"{name} CTR ranking model: {nb} parallel detached dense subarchitectures, batch {spec['batch']}, local BCE heads, Adam, bf16"
    return f"{name}: {nb} detached MLP blocks w{spec['width']}, batch {spec['batch']}, local BCE heads, SGD, {spec['dtype']}"


# ------------------------------------------------------------------------------------------------
# reference arm / cpu baseline: the oracle as it stands, timed on the host cores
# ------------------------------------------------------------------------------------------------

def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def oracle_sample(cfg_name, spec):
    """A bounded sample of the workload for the oracle (about 10-30 s of CPU work per step) and the
    factor that scales its rate to the whole workload.  Small configs: the full batch, every block.
    C4 and the large sweep points: ONE block of the model (on part of the batch where even that is
    above 2 TFLOP); the blocks all have the same shapes and the oracle's cost is linear in blocks and
    rows, so the full step costs n_blocks x (that block at full batch)."""
    nb = len(spec["blocks"])
    if synth.step_flops(spec) < 2e12:
        return spec, 1.0, "the full batch through every block"
    s = dict(spec)
    s["blocks"] = [dict(spec["blocks"][0])]
    frac = 1
    while frac < 8 and synth.step_flops(s) / frac > 2e12 and spec["batch"] % (2 * frac) == 0:
        frac *= 2
    s["batch"] = spec["batch"] // frac
    return s, 1.0 / nb, (f"1 of the {nb} blocks on {s['batch']} of the {spec['batch']} "
                         f"{'sequences' if spec['input'] == 'tokens' else 'samples'}: extrapolated from 1 of {nb} blocks "
                         f"(rate scaled by 1/{nb})")


def time_oracle(spec, steps, warmup):
    """Times oracle steps on `spec`.  Returns (units/s of this spec, ms/step)."""
    from oracle import erase_oracle as orc
    flat = synth.init_params(spec, 0)
    params = {"input": {}, "blocks": [dict() for _ in spec["blocks"]]}
    for (b, name, _shape, _tr), v in zip(synth.tensor_list(spec), flat):
        (params["input"] if b < 0 else params["blocks"][b])[name] = np.asarray(v, np.float64)
    state = orc.new_opt_state(params)
    batches = [synth.make_batch(spec, 0, index=i) for i in range(min(POOL, steps + warmup))]
    for i in range(warmup):
        _, _, params, state = orc.step(spec, params, state, batches[i % len(batches)])
    t0 = time.perf_counter()
    for i in range(steps):
        _, _, params, state = orc.step(spec, params, state, batches[(warmup + i) % len(batches)])
    dt = time.perf_counter() - t0
    return units_per_step(spec) * steps / dt, 1e3 * dt / steps


def metric_name(spec):
    """One name for both arms: the reference arm times the oracle's step of the same workload."""
    return f"train {unit_name(spec)}, ERASE early-backward schedule (vs serial schedule of the same kernels)"


def run_reference(args, spec, cfg_name):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 3))
    warm = 1 if args.warmup > 0 else 0
    sub, scale, what = oracle_sample(cfg_name, spec)
    val, ms = time_oracle(sub, steps, warm)
    val *= scale
    cores = oracle_threads()
    sample = f"{steps} oracle step(s) after {warm} warm-up, each on {what}; {ms:.0f} ms per sampled step"
    line = {"impl": "reference", "metric": metric_name(spec), "value": val,
            "note": "the CPU oracle's step of the same workload (its results do not depend on the schedule)",
            "unit": unit_name(spec), "n_gpus": args.gpus, "steps": steps, "warmup": warm,
            "ms_per_step": 1e3 * units_per_step(spec) / val,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": workload_name(cfg_name, spec)},
            "cpu_baseline": {"value": val, "unit": unit_name(spec), "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": unit_name(spec), "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# clocks sampled during the timed region
# ------------------------------------------------------------------------------------------------

class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            atexit.register(self._kill)     # never leave the tool running if the bench dies early
        except Exception:
            self.proc = None

    def _kill(self):
        if self.proc and self.proc.poll() is None:
            self.proc.kill()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def summary(self, window=None):
        """Summary of the samples that arrived inside `window` = (t0, t1) of time.time(); the tool
        needs a moment to start, so it is started well before the timed legs and filtered here."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        rows = [r for t, r in list(self.rows) if len(r) >= 7 and (window is None or window[0] <= t <= window[1] + 0.1)]
        scope = "timed legs of the headline workload"
        if not rows:
            rows, scope = [r for _, r in list(self.rows) if len(r) >= 7], "whole run (no sample fell into the timed legs)"
        sm = [float(r[0]) for r in rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in rows if r[1].replace(".", "").isdigit()]
        pw = [float(r[2]) for r in rows if r[2].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i] == "Active" for r in rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "reasons": reasons, "samples": len(sm), "scope": scope}

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "tflops": d["bf16_tflops_sustained"], "tflops_burst": d["bf16_tflops"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops": 1400.0, "tflops_burst": 1590.0, "source": "fallback"}


def progress(what):   # BENCH_PROGRESS=1: which leg is running, on stderr
    if os.environ.get("BENCH_PROGRESS"):
        print(f"[bench {time.strftime('%H:%M:%S')}] {what}", file=sys.stderr, flush=True)


def candidate_schedules(binding, spec, args):
    """ERASE placements of the same kernels (all bit-identical): [(flags without GRAPH, description)]."""
    chain = spec["topo"] == "chain"
    out = [(0, "ERASE, backward released after forward and local loss (the paper's placement)")]
    if args.loss_on_main:
        return out
    if chain and not args.no_split_bwd:
        out.append((binding.SPLIT_BWD, "ERASE, backward released after forward and local loss, parameter-gradient work of each "
                                       "backward on a second stream per block"))
    if chain and not args.no_split_bwd:
        out.append((binding.EARLY_HEAD | binding.SPLIT_BWD,
                    "ERASE, local head+loss+backward of each block released onto side streams after the block body, parameter-gradient "
                    "work of each backward on a second stream per block, one optimizer sweep after the join"))
    f = binding.EARLY_HEAD | binding.BLOCK_OPT
    d = "ERASE, local head+loss+backward+optimizer of each block released onto side streams after the block body"
    if chain and not args.no_split_bwd:
        f |= binding.SPLIT_BWD
        d += ", parameter-gradient work of each backward on a second stream per block"
    if not chain and not args.no_par_fwd:
        f |= binding.PAR_FWD
        d += ", every block's forward on its own side stream too (parallel topology)"
    out.append((f, d))
    return out


def pick_schedule(w, binding, spec, args, n_streams, gflags):
    """Times one short repeat of every candidate placement and returns the fastest (flags, description, trial times)."""
    trials = []
    for f, d in candidate_schedules(binding, spec, args):
        w.warm(n_streams, gflags | f, POOL)
        r = w.leg(n_streams, gflags | f, max(4, min(args.steps, 10)), 2, per_step=False, min_s=0.0, max_repeats=2)
        trials.append((min(r["repeats"]), f, d))
    best = w.rep.agree_on(min(trials))     # data-parallel ranks must all step with one schedule: rank 0's pick
    return gflags | best[1], best[2], {d.split(",")[0] + ("" if f == 0 else f" [flags {f}]"): round(t, 3) for t, f, d in trials}


def schedule_flags(binding, spec, args):
    """(n_streams, graph flags of the serial leg, flags of the ERASE leg, description)."""
    nb = len(spec["blocks"])
    n_streams = args.n_streams if args.n_streams > 0 else nb + 1
    flags = 0 if args.no_graph else binding.GRAPH
    eflags = flags | (0 if args.loss_on_main else (binding.EARLY_HEAD | binding.BLOCK_OPT))
    # chains of blocks: the parameter-gradient work of each B_b goes to a second stream per block
    # (measured faster on C1, C2, C4, C5; not on C3, whose blocks already all run side by side)
    split_bwd = not args.loss_on_main and not args.no_split_bwd and spec["topo"] == "chain"
    if split_bwd:
        eflags |= binding.SPLIT_BWD
    # blocks that all read z_0 (C3): their forwards run side by side as well
    par_fwd = not args.loss_on_main and not args.no_par_fwd and spec["topo"] == "parallel"
    if par_fwd:
        eflags |= binding.PAR_FWD
    desc = ("ERASE, local head+loss+backward+optimizer of each block released onto side streams after the block body"
            + (", parameter-gradient work of each backward on a second stream per block" if split_bwd else "")
            + (", every block's forward on its own side stream too (parallel topology)" if par_fwd else "")
            ) if not args.loss_on_main else "ERASE, backward released after forward and local loss"
    return n_streams, flags, eflags, desc


class Workload:
    """One model with its pool of resident batches; everything that owns torch tensors, events or
    streams is dropped by close() before the model (and its CUDA streams) is destroyed."""

    def __init__(self, torch, binding, spec, rep, data_parallel=False):
        self.torch, self.spec, self.rep = torch, spec, rep
        self.model = binding.Model(spec)
        self.model.set_all(synth.init_params(spec, 0))
        if data_parallel:       # one model over all ranks: same parameters everywhere, each rank its own batches
            rep.attach(self.model, binding.comm_unique_id)
        self.main = torch.cuda.ExternalStream(self.model.main_stream())
        self.host, self.dev = [], []
        for i in range(POOL):
            b = synth.make_batch(spec, 0, index=i + (POOL * rep.rank if data_parallel else 0))
            h = {}
            if spec["input"] == "dense":
                x = torch.from_numpy(b["x"])
                h["x"] = x.to(torch.bfloat16) if spec["dtype"] == "bf16" else x
                h["y"] = torch.from_numpy(b["y"])
            elif spec["input"] == "tokens":
                h["ids"] = torch.from_numpy(b["ids"])
            else:
                h["x"], h["ids"], h["y"] = (torch.from_numpy(b[k]) for k in ("dense", "ids", "y"))
            h = {k: v.contiguous().pin_memory() for k, v in h.items()}
            self.host.append(h)
            self.dev.append({k: v.cuda() for k, v in h.items()})
        torch.cuda.synchronize()

    @staticmethod
    def ptrs(d):
        return {k: d[k].data_ptr() if k in d else None for k in ("x", "ids", "y")}

    def barrier(self):
        self.rep.barrier()
        self.torch.cuda.synchronize()

    def warm(self, ns, fl, n):
        for i in range(n):
            self.model.step(n_streams=ns, flags=fl, **self.ptrs(self.dev[i % POOL]))
        self.model.sync()

    def leg(self, ns, fl, steps, warmup, per_step=True, min_s=MIN_LEG_S, max_repeats=200):
        """Repeats of exactly `steps` steps on resident inputs, each bracketed by a barrier and a
        synchronize, timed with CUDA events on the launching stream (max over ranks), until at least
        `min_s` seconds of device time have been timed.  Returns the list of repeat times (ms), the
        per-step times of the median repeat and the launches of one repeat."""
        torch, model = self.torch, self.model
        self.warm(ns, fl, warmup)
        reps, pers, launches, total = [], [], 0, 0.0
        k = 0
        while (not reps or total < min_s * 1e3) and len(reps) < max_repeats:
            n_ev = steps + 1 if per_step else 2
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_ev)]
            l0 = model.launch_count()
            self.barrier()
            evs[0].record(self.main)
            for i in range(steps):
                model.step(n_streams=ns, flags=fl, **self.ptrs(self.dev[(warmup + k + i) % POOL]))
                if per_step:
                    evs[i + 1].record(self.main)
            if not per_step:
                evs[1].record(self.main)
            model.sync()
            self.barrier()
            ms = self.rep.max_over_ranks(evs[0].elapsed_time(evs[-1]))
            reps.append(ms)
            pers.append(np.array([evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]) if per_step else None)
            launches = model.launch_count() - l0
            total += ms
            k += steps
        med = int(np.argsort(reps)[len(reps) // 2])
        return {"ms": reps[med], "repeats": reps, "per_step": pers[med], "launches": launches}

    def kernel_classes(self, nprof=3):
        """Per-kernel-class attribution from profiled serial steps (CUDA events around every operation)."""
        agg = {}
        for i in range(nprof + 1):
            recs = self.model.profile_step(**self.ptrs(self.dev[i % POOL]))
            if i == 0:
                continue    # warm-up of the profiling path
            for r in recs:
                a = agg.setdefault(r["name"], {"ms": 0.0, "flops": 0.0, "bytes": 0.0, "runs": 0, "launches": 0, "big": {}})
                a["ms"] += r["ms"]; a["flops"] += r["flops"]; a["bytes"] += r["bytes"]
                a["runs"] += 1; a["launches"] += r["launches"]
                b = a["big"].setdefault(r["flops"], {"ms": 0.0, "runs": 0})     # the class's members by size
                b["ms"] += r["ms"]; b["runs"] += 1
        return agg

    def close(self):
        self.host = self.dev = self.main = None
        gc.collect()
        self.torch.cuda.synchronize()
        self.model.close()
        self.torch.cuda.empty_cache()


def roofline_of(agg, peaks, cfg_name):
    top = max(agg, key=lambda k: agg[k]["ms"])
    t = agg[top]
    if top.startswith("gemm") or top.startswith("attention"):
        ach = t["flops"] / (t["ms"] * 1e-3) / 1e12
        roof = {"kernel": top, "bound": "tensor", "achieved": ach, "peak": peaks["tflops"], "unit": "TFLOP/s",
                "frac": ach / peaks["tflops"]}
    else:
        ach = t["bytes"] / (t["ms"] * 1e-3) / 1e9
        roof = {"kernel": top, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"]}
    roof["peak_source"] = peaks["source"] + (" (sustained bf16 GEMM)" if roof["bound"] == "tensor" else " (copy)")
    roof["avg_launch_ms"] = t["ms"] / max(t["launches"], 1)
    tr = NCU_DRAM_BYTES.get(cfg_name, {}).get(top)
    roof["traffic"] = tr
    roof["traffic_note"] = NCU_DRAM_NOTE.get(cfg_name) if tr else None
    tot = sum(x["ms"] for x in agg.values())
    roof["kernel_share"] = {k: round(v["ms"] / tot, 4) for k, v in sorted(agg.items(), key=lambda kv: -kv[1]["ms"])[:8]}
    # the same figure for every tensor-bound class, and for the largest member of each (one launch kind: the local head's GEMM)
    by = {}
    for k, v in agg.items():
        if not k.startswith("gemm") or v["flops"] <= 0:
            continue
        fl, b = max(v["big"].items(), key=lambda kv: kv[0])
        by[k] = {"frac": round(v["flops"] / (v["ms"] * 1e-3) / 1e12 / peaks["tflops"], 4), "share": round(v["ms"] / tot, 4),
                 "largest_launch": {"gflop": round(fl / 1e9, 2), "avg_launch_ms": round(b["ms"] / b["runs"], 4),
                                    "frac": round(fl / (b["ms"] / b["runs"] * 1e-3) / 1e12 / peaks["tflops"], 4)}}
    roof["tensor_classes"] = by
    return roof


NCU_DRAM_NOTE = {"C2": "ncu DRAM bytes of the class's largest GEMM (local head), one launch",
                 "C4": "ncu dram__bytes_read.sum + dram__bytes_write.sum of the class's largest GEMM (the local head's, 8192 x 32768 x 768), "
                       "one full-size launch: profiles/tc_gemm_c4_head_ce_fwd_wgrad_dgrad.md"}


# --sweep: the whole saturation sweep (C5: five widths x three batch sizes) instead of the default table's five points
SWEEP = [("C1", "C1", {}), ("C2", "C2", {}), ("C3", "C3", {})] + [
    (f"C5 w{w} b{b}", "C5", {"w": w, "batch": b}) for w in (128, 512, 1024, 2048, 4096) for b in (512, 4096, 32768)]


def table_entry(torch, binding, rep, label, cfg, kw, args, peaks):
    """Serial and ERASE throughput, gain, MFU and dominant kernel class of one parity-table config."""
    spec = synth.config(cfg, **kw)
    progress(f"table: {label}")
    w = Workload(torch, binding, spec, rep)
    try:
        ns, flags, eflags, _ = schedule_flags(binding, spec, args)
        eflags, _, _ = pick_schedule(w, binding, spec, args, ns, flags)
        units = units_per_step(spec)
        # size one repeat to about a quarter of a second from a short trial run
        w.warm(1, flags, POOL)
        t0 = time.perf_counter()
        w.warm(1, flags, 8)
        est = max((time.perf_counter() - t0) / 8, 1e-5)
        steps = int(min(4000, max(8, math.ceil(0.25 / est))))
        ser = w.leg(1, flags, steps, POOL, per_step=False)
        era = w.leg(ns, eflags, steps, POOL, per_step=False)
        pap = w.leg(ns, flags, steps, POOL, per_step=False, min_s=0.3) if eflags != flags else era
        # F_{b+1} and B_b inside one persistent kernel on a partition of the SMs, where the model qualifies
        per = None
        try:
            per = w.leg(1, flags | binding.PERSISTENT, steps, POOL, per_step=False, min_s=0.5)
        except binding.EraseError as e:
            if e.status != binding.EUNSUPPORTED:
                raise
        agg = w.kernel_classes(2)
        roof = roofline_of(agg, peaks, None)
        flops = synth.step_flops(spec)
        ms_e, ms_s = era["ms"] / steps, ser["ms"] / steps
        return {"config": label, "unit": unit_name(spec), "serial": units / (ms_s * 1e-3), "erase": units / (ms_e * 1e-3),
                "ms_per_step_serial": ms_s, "ms_per_step_erase": ms_e, "gain_pct": 100.0 * (ms_s / ms_e - 1.0),
                "gain_pct_loss_on_main_stream": 100.0 * (ser["ms"] / pap["ms"] - 1.0),
                "persistent": None if per is None else units / (per["ms"] / steps * 1e-3),
                "gain_pct_persistent": None if per is None else 100.0 * (ser["ms"] / per["ms"] - 1.0),
                "steps_per_repeat": steps, "repeats": [len(ser["repeats"]), len(era["repeats"])],
                "mfu_vs_measured_sustained": flops / (ms_e * 1e-3) / (peaks["tflops"] * 1e12),
                "top_class": roof["kernel"], "top_class_bound": roof["bound"], "top_class_frac": roof["frac"],
                "top_class_share": roof["kernel_share"].get(roof["kernel"]), "dtype": spec["dtype"]}
    finally:
        w.close()


def run_gpu(args, spec, cfg_name):
    import torch
    from paper_2608_18469_b200 import binding
    from paper_2608_18469_b200.replicas import Replicas

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    rep = Replicas(backend="nccl", device="cuda")
    rank, world, dist = rep.rank, rep.world, rep.dist
    peaks = measured_peaks()
    nb = len(spec["blocks"])
    if args.data_parallel:
        spec = dict(spec, replicas=world)      # every loss is the mean over the global batch = world x batch
    n_streams, flags, eflags, sched_desc = schedule_flags(binding, spec, args)
    units = units_per_step(spec)

    sampler = ClockSampler(local)
    sampler.start()
    w = Workload(torch, binding, spec, rep, data_parallel=args.data_parallel)
    model = w.model

    # serial first (context), then the ERASE schedule; the clock sampler (started before the model
    # was built) is read over the three timed legs
    progress("choosing the ERASE placement")
    eflags, sched_desc, sched_trials = pick_schedule(w, binding, spec, args, n_streams, flags)
    progress("serial leg")
    t_legs = time.time()
    ser = w.leg(1, flags, args.steps, args.warmup)
    progress("ERASE leg")
    era = w.leg(n_streams, eflags, args.steps, args.warmup)
    progress("ERASE leg, loss on the main stream")
    pap = w.leg(n_streams, flags, args.steps, args.warmup) if eflags != flags else era
    clocks = sampler.summary((t_legs, time.time()))

    # end to end through the C ABI: pinned host batch -> device copy, step, losses back to host
    progress("end-to-end leg")
    stage = {k: torch.empty_like(v) for k, v in w.dev[0].items()}
    h2d = sum(v.numel() * v.element_size() for v in stage.values())
    d2h = nb * 4

    def e2e_step(i):
        with torch.cuda.stream(w.main):
            for k in stage:
                stage[k].copy_(w.host[i % POOL][k], non_blocking=True)
        model.step(n_streams=n_streams, flags=eflags, **w.ptrs(stage))
        return model.losses()

    for i in range(args.warmup):
        e2e_step(i)
    e2e_reps, tot = [], 0.0
    while tot < MIN_LEG_S * 1e3 and len(e2e_reps) < 200:
        w.barrier()
        t0 = time.perf_counter()
        for i in range(args.steps):
            e2e_step(args.warmup + i)
        model.sync()
        w.barrier()
        e2e_reps.append(rep.max_over_ranks(1e3 * (time.perf_counter() - t0)))
        tot += e2e_reps[-1]
    e2e_ms = float(np.median(e2e_reps))

    progress("profiled steps")
    roof = roofline_of(w.kernel_classes(3), peaks, cfg_name)
    stage = None
    w.close()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        progress("cpu baseline (oracle)")
        sub, scale, what = oracle_sample(cfg_name, spec)
        val, ms = time_oracle(sub, 1, 0)
        cpu = {"value": val * scale, "unit": unit_name(spec), "cores": oracle_threads(), "kind": "oracle",
               "sample": f"1 oracle step on {what}; {ms / 1e3:.1f} s"}

    table = None
    if world == 1 and not args.no_table:
        table = []
        for label, cfg, kw in (SWEEP if args.sweep else TABLE):
            try:
                table.append(table_entry(torch, binding, rep, label, cfg, kw, args, peaks))
            except Exception as e:      # one config failing must not lose the headline line
                table.append({"config": label, "error": f"{type(e).__name__}: {e}"[:200]})
    sampler.stop()
    if rank != 0:
        if dist is not None:
            rep.close()
        return

    ser_ms, era_ms, ser_per, era_per = ser["ms"], era["ms"], ser["per_step"], era["per_step"]
    flops = synth.step_flops(spec)
    value = world * units * args.steps / (era_ms * 1e-3)
    serial_value = world * units * args.steps / (ser_ms * 1e-3)
    qps = lambda per: units / (per * 1e-3)
    arena_mb = binding.arena_bytes(spec) / 2 ** 20
    line = {
        "metric": metric_name(spec),
        "value": value, "unit": unit_name(spec), "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": era_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": spec["dtype"], "data": "synthetic",
        "config": {"workload": workload_name(cfg_name, spec), "n_streams": n_streams, "schedule": sched_desc,
                   "schedule_choice": {"how": "one short untimed trial of every placement of the same kernels (bit-identical results); "
                                              "the fastest is the timed ERASE leg", "trial_ms_per_repeat": sched_trials},
                   "cuda_graph": not args.no_graph, "batch_pool": POOL,
                   "repeats": f"each leg = repeats of exactly {args.steps} steps until >= {MIN_LEG_S} s are timed; the median repeat is reported",
                   "l2": f"no flush: the step's working set ({arena_mb:.0f} MiB of stashes, logits, parameters) exceeds the 126 MB L2",
                   "multi_gpu": (f"data parallel: one model on {world} shards of a global batch of {world} x {spec['batch']}, each block's "
                                 "gradients summed over the ranks by one NCCL all-reduce right behind that block's backward, on its stream"
                                 if args.data_parallel else "replicas only" if world > 1 else "single GPU")},
        "serial": {"value": serial_value, "ms_per_step": ser_ms / args.steps, "repeats_ms": [round(x, 3) for x in ser["repeats"]],
                   "p90": float(np.percentile(qps(ser_per), 90)), "median": float(np.median(qps(ser_per)))},
        "erase": {"p90": float(np.percentile(qps(era_per), 90)), "median": float(np.median(qps(era_per))),
                  "repeats_ms": [round(x, 3) for x in era["repeats"]]},
        "gain_pct": 100.0 * (value / serial_value - 1.0),
        "erase_loss_on_main_stream": {"value": world * units * args.steps / (pap["ms"] * 1e-3),
                                      "gain_pct": 100.0 * (ser_ms / pap["ms"] - 1.0),
                                      "note": "the paper's placement: local head and loss run on the main stream before the backward is released"},
        "flops_per_step": flops,
        "mfu": {"vs_measured_sustained": flops * args.steps / (era_ms * 1e-3) / (peaks["tflops"] * 1e12),
                "vs_nominal_2250": flops * args.steps / (era_ms * 1e-3) / 2.25e15},
        "clocks": clocks,
        "e2e": {"value": world * units * args.steps / (e2e_ms * 1e-3), "unit": unit_name(spec),
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(era["launches"]),
        "roofline": roof,
        "cpu_baseline": cpu,
        "per_config": table,
    }
    emit(json.dumps(line))
    if dist is not None:
        rep.close()


_STDOUT_FD = None


def quiet_stdout():
    """Libraries loaded during the run (NCCL prints its version banner) write to file descriptor 1: send it to
    stderr for the duration, so that the JSON line stays the only thing on stdout."""
    global _STDOUT_FD
    sys.stdout.flush()
    _STDOUT_FD = os.dup(1)
    os.dup2(2, 1)


def emit(text):
    sys.stdout.flush()
    if _STDOUT_FD is None:
        print(text, flush=True)
    else:
        os.write(_STDOUT_FD, (text + "\n").encode())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C4")
    ap.add_argument("--w", type=int, default=1024)
    ap.add_argument("--batch", type=int, default=4096)
    ap.add_argument("--n-streams", type=int, default=0, help="0 = n_blocks + 1")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--loss-on-main", action="store_true", help="paper's placement of the local loss")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-table", action="store_true", help="skip the per-config table (C1, C2, C3, five C5 points)")
    ap.add_argument("--sweep", action="store_true",
                    help="per-config table over the whole C5 sweep (15 points, several minutes) instead of five of its points")
    ap.add_argument("--no-par-fwd", action="store_true",
                    help="parallel topology: keep the blocks' forwards on the main stream, one after the other")
    ap.add_argument("--no-split-bwd", action="store_true",
                    help="keep the parameter-gradient work of each B_b on the block's own side stream")
    ap.add_argument("--data-parallel", action="store_true",
                    help="N ranks train ONE model (per-block gradient all-reduce inside the step) instead of N independent "
                         "replicas; runs without graph replay")
    args = ap.parse_args()
    if args.data_parallel:
        args.no_graph = True       # the library offers no graph replay around the exchange
    if args.impl == "ours":
        # at least 3 warm-up steps; with graph replay at least one per pooled batch, so that every
        # (batch pointers, schedule) graph is captured and instantiated before the timed region
        args.warmup = max(args.warmup, 3 if args.no_graph else POOL)
    spec = synth.config(args.config, w=args.w, batch=args.batch)
    if args.impl == "reference":
        run_reference(args, spec, args.config)
    else:
        quiet_stdout()
        run_gpu(args, spec, args.config)


if __name__ == "__main__":
    main()
