"""Time one GEMM of the library in isolation through the C ABI (erase_gemm).

  python -m paper_2608_18469_b200.gemm_cli --m 4096 --n 8192 --k 256 --layout fwd --engine 1

Layouts are the three the training step uses: fwd (X W^T, both operands contiguous along k),
dgrad (dY W: B contiguous along n), wgrad (dY^T X: both contiguous along m/n, contraction over
the rows).  Prints one JSON line with the CUDA-event time per call and the achieved TFLOP/s.
Inputs are seeded random bf16 values; the output is overwritten every iteration."""
import argparse
import json

import torch

from . import binding


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--m", type=int, default=4096)
    ap.add_argument("--n", type=int, default=8192)
    ap.add_argument("--k", type=int, default=256)
    ap.add_argument("--layout", default="fwd", choices=["fwd", "dgrad", "wgrad"])
    ap.add_argument("--engine", type=int, default=1)
    ap.add_argument("--splits", type=int, default=1)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args()
    torch.manual_seed(0)
    a_mn = a.layout == "wgrad"
    b_mn = a.layout in ("dgrad", "wgrad")
    ta = torch.randn((a.k, a.m) if a_mn else (a.m, a.k), device="cuda").to(torch.bfloat16)
    tb = torch.randn((a.k, a.n) if b_mn else (a.n, a.k), device="cuda").to(torch.bfloat16)
    f32 = a.splits > 1 or a.layout == "wgrad"
    tc = torch.empty((a.m, a.n), device="cuda", dtype=torch.float32 if f32 else torch.bfloat16)
    sa = (1, a.m) if a_mn else (a.k, 1)
    sb = (1, a.n) if b_mn else (a.k, 1)
    torch.cuda.synchronize()

    def call():
        binding.gemm("bf16", a.m, a.n, a.k, ta.data_ptr(), sa[0], sa[1], tb.data_ptr(), sb[0], sb[1],
                     tc.data_ptr(), a.n, c_f32=f32, splits=a.splits, engine=a.engine)

    for _ in range(a.warmup):
        call()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    print(json.dumps({"m": a.m, "n": a.n, "k": a.k, "layout": a.layout, "engine": a.engine, "splits": a.splits,
                      "ms_per_call_incl_host": ms, "tflops": 2.0 * a.m * a.n * a.k / (ms * 1e-3) / 1e12}))


if __name__ == "__main__":
    main()
