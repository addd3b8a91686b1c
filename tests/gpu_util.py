"""GPU-side test helpers: stage synthetic batches on the device (torch owns the memory) and
compare the CUDA library with the oracle.  Imported only by tests marked gpu."""
import numpy as np
import torch

from oracle import erase_oracle as orc
from paper_2608_18469_b200 import binding, synth
from tests import util

TOL = {"f32": 1e-4, "bf16": 2e-2}     # relative L2 PER TENSOR against the fp64 oracle
# Optimizer alone (fp64 update rule applied to the library's own gradient vs the fp32 kernel).  The
# new parameter is the old one plus an update; the kernel rounds the parameter to fp32 (relative
# 6e-8, a few operations: OPT_TOL of its norm) and computes the update with a handful of fp32
# operations (m, v, two bias corrections, sqrt, divide: a few 1e-7 each, 2e-6 observed:
# OPT_TOL_UPDATE of the update's norm).  A tensor that starts at zero (LayerNorm shift) or happens
# to be tiny (a scalar head bias) consists of the update only, every other one is dominated by the
# parameter; any formula mistake shows up at 1e-3 of the update or more.
OPT_TOL = 2e-6
OPT_TOL_UPDATE = 1e-5

# bf16: a hard 2e-2 per tensor, no exceptions.  A gradient is a sum over samples; on some instances that
# sum nearly cancels (a bias gradient on labels drawn independently of the inputs; every gradient of a
# block right after Adam's first sign step on rare positives), and then no implementation that stores
# activations in bf16 keeps 2e-2 RELATIVE to what is left.  The parity cases therefore run on seeds whose
# instances are well conditioned (chosen by scanning seeds; the scan results are in the design notes);
# when a tensor does fail, the message carries the oracle-measured sensitivity of that instance to bf16
# storage (below), so that a conditioning problem can be told from a kernel bug at a glance.


def oracle_bf16_sensitivity(spec, params, batch):
    """Conditioning probe, computed from the oracle alone: the gradients the oracle gives when
    every Linear output (forward) and every Linear input-gradient (backward) is rounded to bf16,
    the places where a bf16 model stores activations.  The distance of these gradients from the
    exact ones measures how strongly this instance amplifies bf16 storage error: a gradient that
    is a sum over samples of terms of both signs (balanced labels, loss gradient summing to ~0)
    can lose most of its leading digits to cancellation, whatever the implementation."""
    rnd = lambda a: synth.bf16_round(np.asarray(a, np.float32)).astype(np.float64)
    fwd, bwd = orc.linear_fwd, orc.linear_bwd
    try:
        orc.linear_fwd = lambda x, w, b: rnd(fwd(x, w, b))
        orc.linear_bwd = lambda dy, x, w: (lambda r: (rnd(r[0]), r[1], r[2]))(bwd(dy, x, w))
        _, g = orc.forward_backward(spec, params, batch)
    finally:
        orc.linear_fwd, orc.linear_bwd = fwd, bwd
    return g


class DevBatch:
    """Device copies of one batch; keeps the torch tensors alive."""

    def __init__(self, spec, batch):
        dev = "cuda"
        self.x = self.ids = self.y = None
        self.t = {}
        if spec["input"] == "dense":
            x = torch.from_numpy(batch["x"])
            self.t["x"] = (x.to(torch.bfloat16) if spec["dtype"] == "bf16" else x).to(dev).contiguous()
            self.t["y"] = torch.from_numpy(batch["y"]).to(dev)
        elif spec["input"] == "tokens":
            self.t["ids"] = torch.from_numpy(batch["ids"]).to(dev)
        else:
            self.t["x"] = torch.from_numpy(batch["dense"]).to(dev)
            self.t["ids"] = torch.from_numpy(batch["ids"]).to(dev)
            self.t["y"] = torch.from_numpy(batch["y"]).to(dev)
        torch.cuda.synchronize()
        for k, v in self.t.items():
            setattr(self, k, v.data_ptr())

    def args(self):
        return dict(x=self.x, ids=self.ids, y=self.y)


def new_model(spec, flat):
    m = binding.Model(spec)
    names = [(b, n, tuple(s), tr) for (b, n, s, tr) in synth.tensor_list(spec)]
    assert m.num_tensors() == len(names)
    for i, want in enumerate(names):
        assert m.tensor_info(i) == want, (i, m.tensor_info(i), want)
    m.set_all(flat)
    return m


def _slots(params, state, b):
    """Parameter and moment containers of block b, or of the trained input tables for b < 0."""
    if b < 0:
        return params["input"], state["m_in"], state["v_in"]
    return params["blocks"][b], state["m"][b], state["v"][b]


def compare_teacher_forced(spec, steps, seed=0, n_streams=2, flags=0, report=None, case=None, init_hook=None, label_p=None):
    """Each step: library and oracle start from the same fp32 parameters and optimizer state;
    losses and every gradient tensor, each on its own, must agree within TOL; the parameters
    after the optimizer must match the update rule applied in fp64 to the library's own gradients.
    `case` names the instance in messages; with `report` (a dict) nothing is asserted: worst errors and
    the list of tensors over the tolerance are collected instead.  `init_hook(values)` may edit the initial parameters in
    place (a dict keyed by (block, tensor name)) before either side sees them; `label_p` overrides the
    probability of a positive label of the synthetic batches."""
    tol = TOL[spec["dtype"]]
    flat = synth.init_params(spec, seed)
    tl = synth.tensor_list(spec)
    if init_hook is not None:           # the test's own change to the drawn initial values, by tensor name
        init_hook({(b, name): v for (b, name, _s, _t), v in zip(tl, flat)})
    tidx = util.trainable_index(spec)
    m = new_model(spec, flat)
    params = util.structure(spec, flat)
    state = orc.new_opt_state(params)
    worst = {}
    try:
        for it in range(steps):
            batch = synth.make_batch(spec, seed, index=it, label_p=label_p)
            db = DevBatch(spec, batch)
            # teacher forcing: library <- oracle state (rounded to fp32, oracle continues from the same)
            if it > 0:
                for i in tidx:
                    b, name, _s, _t = tl[i]
                    pd, md, vd = _slots(params, state, b)
                    p32 = pd[name].astype(np.float32)
                    pd[name] = p32.astype(np.float64)
                    m32 = md[name].astype(np.float32)
                    v32 = vd[name].astype(np.float32)
                    md[name], vd[name] = m32.astype(np.float64), v32.astype(np.float64)
                    m.set_params(i, p32)
                    m.set_opt_state(i, m32, v32, state["t"])
            m.step(n_streams=n_streams, flags=flags, **db.args())
            got_l = m.losses()
            # oracle: forward/backward at the operand values, optimizer on the fp32 masters
            want_l, want_g, want_gin = orc.forward_backward(spec, util.operand_params(spec, params), util.operand_batch(spec, batch),
                                                            want_input=True)
            new_params = {"input": dict(params["input"]), "blocks": []}
            new_state = {"t": state["t"] + 1, "m": [], "v": [], "m_in": dict(state["m_in"]), "v_in": dict(state["v_in"])}
            touched = {k: orc.touched_rows(spec, batch, k) for k in want_gin}
            for k, g in want_gin.items():       # trained input tables: the rows this batch read
                new_params["input"][k], new_state["m_in"][k], new_state["v_in"][k] = orc.optimizer_update_rows(
                    spec["opt"], params["input"][k], g, touched[k], state["m_in"][k], state["v_in"][k], state["t"] + 1)
            for b, p in enumerate(params["blocks"]):
                np_, nm, nv = {}, {}, {}
                for k in p:
                    np_[k], nm[k], nv[k] = orc.optimizer_update(spec["opt"], p[k], want_g[b][k], state["m"][b][k],
                                                                state["v"][b][k], state["t"] + 1)
                new_params["blocks"].append(np_)
                new_state["m"].append(nm)
                new_state["v"].append(nv)
            for b in range(len(want_l)):
                err = abs(got_l[b] - want_l[b]) / max(abs(want_l[b]), 1e-12)
                worst[f"loss{b}"] = max(worst.get(f"loss{b}", 0), err)
                if report is None:
                    assert err <= tol, (it, "loss", b, got_l[b], want_l[b])
            probe = None
            for i in tidx:
                b, name, _s, _t = tl[i]
                g = m.grads(i)
                want = want_gin[name] if b < 0 else want_g[b][name]
                err = synth.rel_l2(g, want)
                key = f"b{b} {name}" if b >= 0 else f"input {name}"
                worst[f"grad {key}"] = max(worst.get(f"grad {key}", 0), err)
                if err > tol:
                    cond = None
                    if spec["dtype"] == "bf16" and b >= 0:      # diagnostic only: how ill-conditioned is this instance?
                        if probe is None:
                            probe = oracle_bf16_sensitivity(spec, util.operand_params(spec, params),
                                                            util.operand_batch(spec, batch))
                        cond = synth.rel_l2(probe[b][name], want)
                    print(f"[parity] case {case} step {it} {key}: err {err:.3e} > {tol:.0e}; oracle bf16 sensitivity of this "
                          f"instance {cond if cond is None else format(cond, '.3e')}")
                    if report is not None:
                        report.setdefault("violations", []).append(
                            {"case": case, "step": it, "tensor": key, "err": float(err),
                             "sensitivity": None if cond is None else float(cond),
                             "norm": float(np.linalg.norm(want))})
                    else:
                        assert err <= tol, (case, it, key, err, tol, "oracle bf16 sensitivity", cond)
                # optimizer alone: update rule in fp64 on the library's gradient
                pd, md, vd = _slots(params, state, b)
                if b < 0:
                    th, _, _ = orc.optimizer_update_rows(spec["opt"], pd[name], g.astype(np.float64), touched[name],
                                                         md[name], vd[name], state["t"] + 1)
                else:
                    th, _, _ = orc.optimizer_update(spec["opt"], pd[name], g.astype(np.float64), md[name], vd[name], state["t"] + 1)
                old = pd[name]
                pbound = OPT_TOL * np.linalg.norm(old) + OPT_TOL_UPDATE * np.linalg.norm(th - old)
                perr = float(np.linalg.norm(m.params(i).astype(np.float64) - th)) / max(pbound, 1e-300)
                worst["param/bound"] = max(worst.get("param/bound", 0), perr)
                if report is None:
                    assert perr <= 1.0, (it, key, perr, pbound)
            params, state = new_params, new_state
    finally:
        m.close()
    if report is not None:
        report.update(worst)
    return worst


def run_steps(spec, flat, batches, n_streams, flags=0, attach=None, orders=None):
    """Free-running steps; returns per-step losses and the final raw state for bit comparison.
    attach(model) runs once before the first step; orders (a list) receives every step's exchange order."""
    m = new_model(spec, flat)
    try:
        if attach is not None:
            attach(m)
        losses = []
        for db in batches:
            m.step(n_streams=n_streams, flags=flags, **db.args())
            losses.append(m.losses().copy())
            if orders is not None:
                orders.append(m.comm_order())
        tidx = util.trainable_index(spec)
        final = {"losses": np.array(losses)}
        for i in tidx:
            final[f"p{i}"] = m.params(i)
            final[f"g{i}"] = m.grads(i)
            mm, vv, t = m.opt_state(i)
            final[f"m{i}"], final[f"v{i}"] = mm, vv
        final["t"] = np.array([t])
        final["launches"] = m.launch_count()
        return final
    finally:
        m.close()
