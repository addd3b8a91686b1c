"""Print the device-side timeline of one training step (through the C ABI): when each block's
forward F_b and backward B_b started and ended, for the serial schedule and for the ERASE
schedules.  This is the overlap evidence: under ERASE, B_b runs while F_{b+1} does.  The first
three timelines use CUDA events around every phase (no graph replay, so the host's launch rate
shows); the "graph replay" ones use device clock stamps captured into the step's CUDA graph,
i.e. they show the schedule the benchmark times.

  python -m paper_2608_18469_b200.timeline_cli --config C2
"""
import argparse

import numpy as np
import torch

from . import binding, synth


def stage(spec, batch):
    t = {}
    if spec["input"] == "dense":
        x = torch.from_numpy(batch["x"])
        t["x"] = (x.to(torch.bfloat16) if spec["dtype"] == "bf16" else x).cuda()
        t["y"] = torch.from_numpy(batch["y"]).cuda()
    elif spec["input"] == "tokens":
        t["ids"] = torch.from_numpy(batch["ids"]).cuda()
    else:
        t["x"], t["ids"], t["y"] = (torch.from_numpy(batch[k]).cuda() for k in ("dense", "ids", "y"))
    torch.cuda.synchronize()
    return t


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="C2")
    ap.add_argument("--w", type=int, default=1024)
    ap.add_argument("--batch", type=int, default=4096)
    ap.add_argument("--reps", type=int, default=5)
    a = ap.parse_args()
    spec = synth.config(a.config, w=a.w, batch=a.batch)
    nb = len(spec["blocks"])
    m = binding.Model(spec)
    m.set_all(synth.init_params(spec, 0))
    t = stage(spec, synth.make_batch(spec, 0))
    args = {k: v.data_ptr() for k, v in t.items()}
    G = binding.GRAPH | binding.STAMPS
    E = binding.EARLY_HEAD | binding.BLOCK_OPT
    for name, ns, fl in (("serial", 1, 0), ("ERASE, loss on the main stream", nb + 1, 0),
                         ("ERASE, head+loss+backward on side streams", nb + 1, binding.EARLY_HEAD),
                         ("graph replay, serial", 1, G),
                         ("graph replay, ERASE, loss on the main stream", nb + 1, G),
                         ("graph replay, ERASE, head+loss+backward+optimizer on side streams", nb + 1, G | E),
                         ("graph replay, ERASE, as above with the parameter-gradient work on a second stream per block",
                          nb + 1, G | E | binding.SPLIT_BWD),
                         ("graph replay, ERASE, every block's forward on its side stream too (parallel topology only)",
                          nb + 1, G | E | binding.PAR_FWD)):
        if fl & binding.PAR_FWD and spec["topo"] != "parallel":
            continue
        tl = None
        for _ in range(a.reps):          # the last repetition is reported (warm caches, warm clocks)
            m.step(n_streams=ns, flags=fl, **args)
            tl = m.timeline()
        end = max(tl[2 * nb][1], max(tl[nb + b][1] for b in range(nb)))
        how = "device clock stamps inside the CUDA graph" if fl & binding.GRAPH else "event-timed, no graph replay"
        print(f"\n{name}: step {end:.3f} ms ({how})")
        for b in range(nb):
            f0, f1 = tl[b]
            b0, b1 = tl[nb + b]
            ov = ""
            if b + 1 < nb:
                g0, g1 = tl[b + 1]
                ov = f"   B_{b+1} overlaps F_{b+2} for {max(0.0, min(b1, g1) - max(b0, g0)):.3f} ms"
            print(f"  F_{b+1} {f0:7.3f} -> {f1:7.3f}    B_{b+1} {b0:7.3f} -> {b1:7.3f}{ov}")
        print(f"  optimizer {tl[2 * nb][0]:7.3f} -> {tl[2 * nb][1]:7.3f}")
    m.close()


if __name__ == "__main__":
    main()
