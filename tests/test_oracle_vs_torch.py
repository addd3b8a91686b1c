"""Library cross-check of the whole oracle: the same detached networks written with torch CPU
modules/functionals in float64, gradients from autograd with ``.detach()`` between blocks and
updates from ``torch.optim``.  This is the special case "the method reduces to library routines":
it pins the forward values, the gradients and the optimizer of the oracle to an implementation
that shares none of its code (F.layer_norm, F.gelu, F.cross_entropy, autograd, torch.optim)."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as TF

from oracle import erase_oracle as orc
from paper_2608_18469_b200 import synth
from tests import util

torch.set_default_dtype(torch.float64)


def _act(kind, u):
    return {"none": lambda t: t, "relu": torch.relu, "gelu": TF.gelu}[kind](u)


def _torch_block(spec, blk, p, zin):
    k = blk["kind"]
    if k in ("mlp", "tower"):
        n_lin = len(blk["dims"]) - 1
        h = zin
        for i in range(n_lin):
            h = TF.linear(h, p[f"W{i}"], p[f"b{i}"])
            if k == "tower" or i < n_lin - 1:
                h = _act(blk["act"], h)
        return h
    if k == "transformer":
        d = blk["dims"][0]
        bt, t, nh = spec["batch"], spec["seq"], blk["n_heads"]
        a = TF.layer_norm(zin, (d,), p["ln1_g"], p["ln1_b"], 1e-5)
        qkv = TF.linear(a, p["Wqkv"], p["bqkv"]).view(bt, t, 3, nh, d // nh)
        q, kk, v = (qkv[:, :, i].transpose(1, 2) for i in range(3))
        o = TF.scaled_dot_product_attention(q, kk, v, is_causal=True)
        o = o.transpose(1, 2).reshape(bt * t, d)
        h = zin + TF.linear(o, p["Wproj"], p["bproj"])
        m = TF.layer_norm(h, (d,), p["ln2_g"], p["ln2_b"], 1e-5)
        return h + TF.linear(TF.gelu(TF.linear(m, p["W1"], p["b1"])), p["W2"], p["b2"])
    if k == "cross":
        x = zin
        for i in range(blk["n_cross"]):
            x = zin * TF.linear(x, p[f"Wc{i}"], p[f"bc{i}"]) + x
        return x
    if k == "dot":
        e, ns = spec["emb_dim"], spec["n_sparse"]
        nb = zin.shape[0]
        proj = TF.linear(zin[:, ns * e:], p["Wd"], p["bd"])
        vec = torch.cat([proj[:, None, :], zin[:, :ns * e].view(nb, ns, e)], dim=1)
        gram = torch.bmm(vec, vec.transpose(1, 2))
        feats = [gram[:, i, j] for i in range(ns + 1) for j in range(i)]
        f = torch.cat([torch.stack(feats, dim=1), proj], dim=1)
        f = TF.pad(f, (0, blk["dims"][0] - f.shape[1]))
        n_lin = len(blk["dims"]) - 1
        for i in range(n_lin):
            f = _act(blk["act"], TF.linear(f, p[f"W{i}"], p[f"b{i}"]))
        return f
    raise ValueError(k)


def _torch_step(spec, tparams, z0, target, optim):
    """forward with detach between blocks, ONE backward on the summed loss (Eq. 2), optimizer."""
    losses = []
    z = z0
    for blk, p in zip(spec["blocks"], tparams):
        zin = (z0 if spec["topo"] == "parallel" else z).detach()
        z = _torch_block(spec, blk, p, zin)
        if blk["head"] == "goodness":       # BCE on the goodness score G = sum_j z_j^2, threshold bh (Section 2.1)
            losses.append(TF.binary_cross_entropy_with_logits((z * z).sum(dim=1) + p["bh"][0], target))
            continue
        s = TF.linear(z, p["Wh"], p["bh"])
        if blk["head"] == "bce":
            losses.append(TF.binary_cross_entropy_with_logits(s[:, 0], target))
        else:
            losses.append(TF.cross_entropy(s, target))
    optim.zero_grad()
    sum(losses).backward()
    grads = [{k: v.grad.detach().numpy().copy() for k, v in p.items()} for p in tparams]
    optim.step()
    return [float(l.detach()) for l in losses], grads


def _run(spec, steps, seed=0):
    flat = synth.init_params(spec, seed)
    params = util.structure(spec, flat)
    # perturb LN gain/shift and everything else a little so nothing sits at a special point
    rng = np.random.default_rng(11)
    for p in params["blocks"]:
        for k in p:
            p[k] = p[k] + 0.02 * rng.standard_normal(p[k].shape)
    tparams = [{k: torch.tensor(v, requires_grad=True) for k, v in p.items()} for p in params["blocks"]]
    allp = [v for p in tparams for v in p.values()]
    o = spec["opt"]
    if o["kind"] == "sgd":
        optim = torch.optim.SGD(allp, lr=o["lr"])
    elif o["kind"] == "adam":
        optim = torch.optim.Adam(allp, lr=o["lr"], betas=(o["beta1"], o["beta2"]), eps=o["eps"])
    else:
        optim = torch.optim.AdamW(allp, lr=o["lr"], betas=(o["beta1"], o["beta2"]), eps=o["eps"],
                                  weight_decay=o["wd"])
    state = orc.new_opt_state(params)
    for it in range(steps):
        batch = synth.make_batch(spec, seed, index=it)
        z0, target = orc.stage_input(spec, params["input"], batch)   # staging is pinned separately
        tt = torch.tensor(target) if target.dtype.kind == 'f' else torch.tensor(target, dtype=torch.long)
        tl, tg = _torch_step(spec, tparams, torch.tensor(z0), tt, optim)
        ol, og, params, state = orc.step(spec, params, state, batch)
        assert np.allclose(ol, tl, rtol=1e-12, atol=1e-13), (it, ol, tl)
        for b in range(len(tg)):
            for k in tg[b]:
                assert synth.rel_l2(og[b][k], tg[b][k]) < 1e-10, (it, b, k)
                # Parameters agree to 1e-12, plus what the optimizer makes of the (<= 1e-10) difference
                # between the two gradients: Adam's update lr*m^/(sqrt(v^)+eps) has slope up to lr/eps
                # where the gradient is mathematically zero and both sides hold rounding noise of
                # ~1e-17 (the key bias of attention: softmax does not see it); SGD's slope is lr.
                want = tparams[b][k].detach().numpy()
                slope = o["lr"] if o["kind"] == "sgd" else o["lr"] / o["eps"]
                bound = 1e-12 * np.linalg.norm(want) + 2.0 * slope * np.linalg.norm(og[b][k] - tg[b][k])
                assert np.linalg.norm(params["blocks"][b][k] - want) <= bound, (it, b, k)


@pytest.mark.parametrize("name", list(util.tiny_specs()))
def test_tiny_instances_three_steps(name):
    spec = util.tiny_specs()[name]
    _run(spec, steps=3)


@pytest.mark.parametrize("optk", ["sgd", "adam", "adamw"])
def test_mid_size_mlp_all_optimizers(optk):
    o = {"kind": optk, "lr": 1e-2, "wd": 0.05, "beta1": 0.9, "beta2": 0.999, "eps": 1e-8}
    spec = synth.mlp_spec(32, 64, 3, 40, "gelu", "f32", opt=o)
    _run(spec, steps=4)


def test_mid_size_lm():
    spec = synth.lm_spec(2, 32, 4, 64, 16, 3, 50, dtype="f32")
    _run(spec, steps=2)


def test_mid_size_ctr():
    spec = synth.ctr_spec(batch=32, n_dense=13, n_sparse=5, table_rows=50, emb_dim=8,
                          tower=(24, 16, 8), n_cross=3, dtype="f32")
    _run(spec, steps=2)


def test_config1_ten_steps_full_size():
    """The tiny fp32 MLP workload at its stated size, ten steps from seed 0."""
    _run(synth.config("C1"), steps=10)
