#!/usr/bin/env python
"""Benchmark of the ERASE training step on B200: tokens/s (samples/s) of the early-backward
schedule against the serial schedule of the same kernels, on synthetic data.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C2] [--impl reference]

One JSON line on stdout (rank 0).  A "step" is one pass of the whole hot path over one batch:
input staging, every block's forward + local loss, every block's backward, the optimizer.
With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the
workload on its own GPU (the path has no exchange step on one node: "replicas only"); the value
is the units all ranks processed divided by the slowest rank's time.
"""
import argparse
import atexit
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_18469_b200 import synth  # noqa: E402

POOL = 8   # distinct pre-staged batches, cycled

# dram__bytes_read.sum + dram__bytes_write.sum per launch from ncu captures of the largest member
# of each kernel class at C2 (the local head's GEMMs; profiles/tc_gemm_c2_head_fwd_dgrad_wgrad.md).
# They sit below the algorithmic bytes where a 64 MiB operand or result is still L2-resident.
NCU_DRAM_BYTES = {"C2": {"gemm_fwd": 15.5e6, "gemm_dgrad": 75.4e6, "gemm_wgrad": 71.4e6}}


def unit_name(spec):
    return "tokens/s" if spec["input"] == "tokens" else "samples/s"


def units_per_step(spec):
    return spec["batch"] * (spec["seq"] if spec["input"] == "tokens" else 1)


def workload_name(name, spec):
    if name == "C2":
        return "C2 small LM proxy: 4 detached pre-LN transformer blocks d256 h4 ff1024 T256 batch16 vocab8192, CE heads, AdamW"
    return f"{name}: {len(spec['blocks'])} detached blocks, batch {spec['batch']}"


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


def time_oracle(spec, steps, warmup):
    """Times oracle steps (each on one full batch of the workload).  Returns (units/s, ms/step)."""
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
    val, ms = time_oracle(spec, steps, warm)
    cores = oracle_threads()
    sample = f"{steps} full oracle step(s) of the workload's batch ({units_per_step(spec)} {unit_name(spec).split('/')[0]}) after {warm} warm-up"
    line = {"impl": "reference", "metric": metric_name(spec), "value": val,
            "note": "the CPU oracle's step of the same workload (its results do not depend on the schedule)",
            "unit": unit_name(spec), "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": ms,
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

    def stop(self, window=None):
        """Summary of the samples that arrived inside `window` = (t0, t1) of time.time(); the tool
        needs a moment to start, so it is started well before the timed legs and filtered here."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [r for t, r in self.rows if len(r) >= 7 and (window is None or window[0] <= t <= window[1] + 0.1)]
        scope = "timed legs"
        if not rows:
            rows, scope = [r for _, r in self.rows if len(r) >= 7], "whole run (no sample fell into the timed legs)"
        sm = [float(r[0]) for r in rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in rows if r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i] == "Active" for r in rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm), "scope": scope}


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


def run_gpu(args, spec, cfg_name):
    import torch
    from paper_2608_18469_b200 import binding

    from paper_2608_18469_b200.replicas import Replicas
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    rep = Replicas(backend="nccl", device="cuda")
    rank, world, dist = rep.rank, rep.world, rep.dist

    def barrier():
        rep.barrier()
        torch.cuda.synchronize()

    max_over_ranks = rep.max_over_ranks

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
    units = units_per_step(spec)

    sampler = ClockSampler(local)
    sampler.start()
    model = binding.Model(spec)
    model.set_all(synth.init_params(spec, 0))

    def measure():
        """Everything that owns torch tensors, events or streams lives in this scope, so that it
        is released before the model (and its CUDA streams) is destroyed."""
        main = torch.cuda.ExternalStream(model.main_stream())

        # pool of batches resident in HBM, and their pinned host copies for the end-to-end leg
        host, dev = [], []
        for i in range(POOL):
            b = synth.make_batch(spec, 0, index=i)
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
            host.append(h)
            dev.append({k: v.cuda() for k, v in h.items()})
        torch.cuda.synchronize()

        def ptrs(d):
            return {k: d[k].data_ptr() if k in d else None for k in ("x", "ids", "y")}

        def timed(ns, fl, steps, warmup):
            """K steps on resident inputs, per-step CUDA events on the launching stream."""
            for i in range(warmup):
                model.step(n_streams=ns, flags=fl, **ptrs(dev[i % POOL]))
            model.sync()
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
            l0 = model.launch_count()
            barrier()
            evs[0].record(main)
            for i in range(steps):
                model.step(n_streams=ns, flags=fl, **ptrs(dev[(warmup + i) % POOL]))
                evs[i + 1].record(main)
            model.sync()
            barrier()
            total_ms = evs[0].elapsed_time(evs[-1])
            per = np.array([evs[i].elapsed_time(evs[i + 1]) for i in range(steps)])
            return max_over_ranks(total_ms), per, model.launch_count() - l0

        def progress(what):   # BENCH_PROGRESS=1: which leg is running, on stderr
            if os.environ.get("BENCH_PROGRESS"):
                print(f"[bench] {what}", file=sys.stderr, flush=True)

        # serial first (context), then the ERASE schedule; the clock sampler (started before the
        # model was built) is read over the three timed legs
        progress("serial leg")
        t_legs = time.time()
        ser_ms, ser_per, _ = timed(1, flags, args.steps, args.warmup)
        progress("ERASE leg")
        era_ms, era_per, launches = timed(n_streams, eflags, args.steps, args.warmup)
        progress("ERASE leg, loss on the main stream")
        pap_ms, pap_per, _ = timed(n_streams, flags, args.steps, args.warmup) if eflags != flags else (era_ms, era_per, 0)
        clocks = sampler.stop((t_legs, time.time()))
        progress("end-to-end leg")

        # end to end through the C ABI: pinned host batch -> device copy, step, losses back to host
        stage = {k: torch.empty_like(v) for k, v in dev[0].items()}
        h2d = sum(v.numel() * v.element_size() for v in stage.values())
        d2h = nb * 4

        def e2e_step(i):
            with torch.cuda.stream(main):
                for k in stage:
                    stage[k].copy_(host[i % POOL][k], non_blocking=True)
            model.step(n_streams=n_streams, flags=eflags, **ptrs(stage))
            return model.losses()

        for i in range(args.warmup):
            e2e_step(i)
        barrier()
        t0 = time.perf_counter()
        for i in range(args.steps):
            e2e_step(args.warmup + i)
        model.sync()
        barrier()
        e2e_ms = max_over_ranks(1e3 * (time.perf_counter() - t0))

        # per-kernel attribution: profiled serial steps (events around every operation)
        progress("profiled steps")
        agg = {}
        nprof = 3
        for i in range(nprof + 1):
            recs = model.profile_step(**ptrs(dev[i % POOL]))
            if i == 0:
                continue    # warm-up of the profiling path
            for r in recs:
                a = agg.setdefault(r["name"], {"ms": 0.0, "flops": 0.0, "bytes": 0.0, "runs": 0, "launches": 0})
                a["ms"] += r["ms"]; a["flops"] += r["flops"]; a["bytes"] += r["bytes"]
                a["runs"] += 1; a["launches"] += r["launches"]
        top = max(agg, key=lambda k: agg[k]["ms"])
        peaks = measured_peaks()
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
        roof["traffic_note"] = "ncu DRAM bytes of the class's largest GEMM (local head), one launch" if tr else None
        roof["kernel_share"] = {k: round(v["ms"] / sum(x["ms"] for x in agg.values()), 4)
                                for k, v in sorted(agg.items(), key=lambda kv: -kv[1]["ms"])[:8]}

        cpu = None
        if rank == 0 and world == 1 and not args.no_cpu_baseline:
            val, ms = time_oracle(spec, 1, 1)
            cpu = {"value": val, "unit": unit_name(spec), "cores": oracle_threads(), "kind": "oracle",
                   "sample": f"1 full oracle step of the workload's batch ({units} units) after 1 warm-up step; {ms:.0f} ms"}


        return dict(pap_ms=pap_ms, ser_ms=ser_ms, ser_per=ser_per, era_ms=era_ms, era_per=era_per, launches=launches,
                    clocks=clocks, e2e_ms=e2e_ms, h2d=h2d, d2h=d2h, roof=roof, cpu=cpu)

    import gc
    peaks = measured_peaks()
    r = measure()
    gc.collect()
    torch.cuda.synchronize()
    model.close()
    ser_ms, ser_per, era_ms, era_per, launches = r["ser_ms"], r["ser_per"], r["era_ms"], r["era_per"], r["launches"]
    clocks, e2e_ms, h2d, d2h, roof, cpu = r["clocks"], r["e2e_ms"], r["h2d"], r["d2h"], r["roof"], r["cpu"]
    if rank != 0:
        if dist is not None:
            rep.close()
        return
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
        "config": {"workload": workload_name(cfg_name, spec), "n_streams": n_streams,
                   "schedule": ("ERASE, local head+loss+backward+optimizer of each block released onto side streams after the block body"
                                + (", parameter-gradient work of each backward on a second stream per block" if split_bwd else "")
                                + (", every block's forward on its own side stream too (parallel topology)" if par_fwd else ""))
                               if not args.loss_on_main else "ERASE, backward released after forward and local loss",
                   "cuda_graph": not args.no_graph, "batch_pool": POOL,
                   "l2": f"no flush: the step's working set ({arena_mb:.0f} MiB of stashes, logits, parameters) exceeds the 126 MB L2",
                   "multi_gpu": "replicas only" if world > 1 else "single GPU"},
        "serial": {"value": serial_value, "ms_per_step": ser_ms / args.steps,
                   "p90": float(np.percentile(qps(ser_per), 90)), "median": float(np.median(qps(ser_per)))},
        "erase": {"p90": float(np.percentile(qps(era_per), 90)), "median": float(np.median(qps(era_per)))},
        "gain_pct": 100.0 * (value / serial_value - 1.0),
        "erase_loss_on_main_stream": {"value": world * units * args.steps / (r["pap_ms"] * 1e-3),
                                      "gain_pct": 100.0 * (ser_ms / r["pap_ms"] - 1.0),
                                      "note": "the paper's placement: local head and loss run on the main stream before the backward is released"},
        "flops_per_step": flops,
        "mfu": {"vs_measured_sustained": flops * args.steps / (era_ms * 1e-3) / (peaks["tflops"] * 1e12),
                "vs_nominal_2250": flops * args.steps / (era_ms * 1e-3) / 2.25e15},
        "clocks": clocks,
        "e2e": {"value": world * units * args.steps / (e2e_ms * 1e-3), "unit": unit_name(spec),
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "roofline": roof,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        rep.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C2")
    ap.add_argument("--w", type=int, default=1024)
    ap.add_argument("--batch", type=int, default=4096)
    ap.add_argument("--n-streams", type=int, default=0, help="0 = n_blocks + 1")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--loss-on-main", action="store_true", help="paper's placement of the local loss")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-par-fwd", action="store_true",
                    help="parallel topology: keep the blocks' forwards on the main stream, one after the other")
    ap.add_argument("--no-split-bwd", action="store_true",
                    help="keep the parameter-gradient work of each B_b on the block's own side stream")
    args = ap.parse_args()
    if args.impl == "ours":
        # at least 3 warm-up steps; with graph replay at least one per pooled batch, so that every
        # (batch pointers, schedule) graph is captured and instantiated before the timed region
        args.warmup = max(args.warmup, 3 if args.no_graph else POOL)
    spec = synth.config(args.config, w=args.w, batch=args.batch)
    if args.impl == "reference":
        run_reference(args, spec, args.config)
    else:
        run_gpu(args, spec, args.config)


if __name__ == "__main__":
    main()
