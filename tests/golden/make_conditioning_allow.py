"""Writes tests/golden/bf16_conditioning_allow.json.  Calls only the oracle (no GPU, no library).

For every (case, step, tensor) named in ENTRIES it replays the teacher-forced oracle trajectory of
the parity test up to that step and measures how far that tensor's gradient moves when the oracle
itself stores every Linear output and every Linear input-gradient in bfloat16 (relative L2 against
the exact gradient): the sensitivity of that INSTANCE to bf16 storage, whatever the implementation.
The GPU parity harness (tests/gpu_util.py) lets a listed tensor exceed the 2e-2 tolerance only up
to a small multiple of the sensitivity it measures live, under a fixed cap.

    python tests/golden/make_conditioning_allow.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import erase_oracle as orc  # noqa: E402
from paper_2608_18469_b200 import synth  # noqa: E402
from tests import util  # noqa: E402

# (case name as used by tests/test_gpu_parity.py, spec, seed, step, block, tensor, kind, why)
ENTRIES = [
    ("C3", synth.config("C3"), 0, 1, 5, "W0", "weight",
     "after Adam's first (sign) step on labels with 3 % positives the dot block's gradient shrinks 30-fold "
     "(norm 1.40 at step 0, 0.048 at step 1): the many +0.03 and the few -0.97 loss gradients nearly cancel, "
     "so the bf16 rounding of the block output that feeds the fp32 head (forward storage alone: 2.3e-2) is "
     "amplified; the backward storage contributes 1e-3"),
]


def sensitivity(spec, seed, step, block, tensor):
    rnd = lambda a: synth.bf16_round(np.asarray(a, np.float32)).astype(np.float64)
    params = util.structure(spec, synth.init_params(spec, seed))
    state = orc.new_opt_state(params)
    for it in range(step + 1):
        batch = util.operand_batch(spec, synth.make_batch(spec, seed, index=it))
        ops = util.operand_params(spec, params)
        _, g = orc.forward_backward(spec, ops, batch)
        if it == step:
            fwd, bwd = orc.linear_fwd, orc.linear_bwd
            try:
                orc.linear_fwd = lambda x, w, b: rnd(fwd(x, w, b))
                orc.linear_bwd = lambda dy, x, w: (lambda r: (rnd(r[0]), r[1], r[2]))(bwd(dy, x, w))
                _, gp = orc.forward_backward(spec, ops, batch)
            finally:
                orc.linear_fwd, orc.linear_bwd = fwd, bwd
            return synth.rel_l2(gp[block][tensor], g[block][tensor]), float(np.linalg.norm(g[block][tensor]))
        # teacher forcing as in the parity test: optimizer on the fp32 masters, state kept in fp32
        new = {"input": params["input"], "blocks": []}
        ns = {"t": state["t"] + 1, "m": [], "v": []}
        for b, p in enumerate(params["blocks"]):
            np_, nm, nv = {}, {}, {}
            for k in p:
                th, m1, v1 = orc.optimizer_update(spec["opt"], p[k], g[b][k], state["m"][b][k], state["v"][b][k], state["t"] + 1)
                np_[k] = th.astype(np.float32).astype(np.float64)
                nm[k], nv[k] = m1.astype(np.float32).astype(np.float64), v1.astype(np.float32).astype(np.float64)
            new["blocks"].append(np_); ns["m"].append(nm); ns["v"].append(nv)
        params, state = new, ns


def main():
    out = {"about": "bf16 parity: gradient tensors that may exceed 2e-2 relative L2 because the INSTANCE is ill-conditioned "
                    "(a sum over samples that nearly cancels). One entry per (case, step, tensor) with the oracle-measured "
                    "sensitivity of that instance to bf16 storage. Written by tests/golden/make_conditioning_allow.py (oracle "
                    "only). tests/gpu_util.py fails every tensor above 2e-2 that is not listed here; a listed bias may reach "
                    "min(1e-1, 3 x live sensitivity), a listed weight min(5e-2, 1.5 x live sensitivity).",
           "entries": []}
    for case, spec, seed, step, block, tensor, kind, why in ENTRIES:
        s, norm = sensitivity(spec, seed, step, block, tensor)
        out["entries"].append({"case": case, "seed": seed, "step": step, "tensor": f"b{block} {tensor}", "kind": kind,
                               "sensitivity": round(s, 5), "gradient_norm": norm, "why": why})
        print(case, step, block, tensor, s, norm)
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "bf16_conditioning_allow.json"), "w") as f:
        json.dump(out, f, indent=1)
        f.write("\n")


if __name__ == "__main__":
    main()
