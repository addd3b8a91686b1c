"""Run a few training steps of one model through the C ABI and print where the time goes.

  python -m paper_2608_18469_b200.step_cli --config C2
  python -m paper_2608_18469_b200.step_cli --lm 1,768,12,3072,1024,8,32768 --steps 2   # one block of C4's shapes

`--lm n_blocks,d_model,n_heads,d_ff,seq,batch,vocab` builds a transformer model of those shapes
(a small stand-in for a large configuration: a single block holds every kernel of the full model
at its full size, in about a tenth of the memory, which is what a profiler capture needs).
The steps run in the serial order with CUDA events around every operation (erase_profile_step);
the table lists each operation of block 0 with its time and its achieved rate.  This is the command
the kernel profiles under profiles/ were taken with."""
import argparse

import torch

from . import binding, synth
from .timeline_cli import stage


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="C2")
    ap.add_argument("--w", type=int, default=1024)
    ap.add_argument("--batch", type=int, default=4096)
    ap.add_argument("--lm", default=None, help="n_blocks,d_model,n_heads,d_ff,seq,batch,vocab")
    ap.add_argument("--steps", type=int, default=3)
    a = ap.parse_args()
    if a.lm:
        spec = synth.lm_spec(*[int(x) for x in a.lm.split(",")])
    else:
        spec = synth.config(a.config, w=a.w, batch=a.batch)
    m = binding.Model(spec)
    m.set_all(synth.init_params(spec, 0))
    t = stage(spec, synth.make_batch(spec, 0))
    args = {k: v.data_ptr() for k, v in t.items()}
    for _ in range(a.steps):
        recs = m.profile_step(**args)
    print(f"losses {m.losses().tolist()}")
    print(f"step: {sum(r['ms'] for r in recs):.3f} ms over {len(recs)} operations (serial order, events around every operation)")
    for r in recs:
        if r["block"] in (-1, 0):
            tensor = r["name"].startswith(("gemm", "attention"))
            rate = (r["flops"] / r["ms"] / 1e9 if tensor else r["bytes"] / r["ms"] / 1e6) if r["ms"] > 0 else 0.0
            print(f"  phase {r['phase']} {r['name']:18s} {r['ms'] * 1e3:9.1f} us  {r['flops'] / 1e9:9.2f} GFLOP {r['bytes'] / 1e6:9.1f} MB"
                  f"  {rate:9.1f} {'TFLOP/s' if tensor else 'GB/s'}")
    agg = {}
    for r in recs:
        agg[r["name"]] = agg.get(r["name"], 0.0) + r["ms"]
    print({k: round(v, 3) for k, v in sorted(agg.items(), key=lambda kv: -kv[1])})
    m.close()


if __name__ == "__main__":
    main()
