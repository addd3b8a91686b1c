"""Pins for the CPU oracle: finite differences, stop-gradient invariants, closed forms,
conservation laws, optimizer closed forms.  None of these re-types the oracle's own formulas
as the expectation: each compares against mathematics fixed elsewhere (a limit, a hand-worked
value, an invariant)."""
import copy
import json
import math
import os

import numpy as np
import pytest

from oracle import erase_oracle as orc
from paper_2608_18469_b200 import synth
from tests import util

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _setup(spec, seed=0, **kw):
    flat = synth.init_params(spec, seed, **kw)
    return util.structure(spec, flat), synth.make_batch(spec, seed)


# ---------------------------------------------------------------- finite differences

@pytest.mark.parametrize("name", list(util.tiny_specs()))
def test_gradients_match_central_differences(name):
    """d l_b / d theta_b from the oracle's backward equals the central difference of the
    forward-only loss l_b, for every scalar of every trainable tensor."""
    spec = util.tiny_specs()[name]
    params, batch = _setup(spec, seed=3)
    # move away from symmetric / degenerate points (LN gain 1, shift 0)
    rng = np.random.default_rng(5)
    for p in params["blocks"]:
        for k in p:
            p[k] = p[k] + 0.05 * rng.standard_normal(p[k].shape)
    _, grads = orc.forward_backward(spec, params, batch)
    h = 1e-5
    worst = 0.0
    for b, p in enumerate(params["blocks"]):
        for k in p:
            fd = np.zeros_like(p[k])
            it = np.nditer(p[k], flags=["multi_index"])
            for _ in it:
                idx = it.multi_index
                old = p[k][idx]
                p[k][idx] = old + h
                lp = orc.forward_only(spec, params, batch)[b]
                p[k][idx] = old - h
                lm = orc.forward_only(spec, params, batch)[b]
                p[k][idx] = old
                fd[idx] = (lp - lm) / (2 * h)
            err = synth.rel_l2(grads[b][k], fd)
            worst = max(worst, err)
            assert err <= 1e-6, (name, b, k, err)
    assert worst > 0.0


# ---------------------------------------------------------------- detachment (Eq. 1)

@pytest.mark.parametrize("name", ["mlp_relu", "lm"])
def test_later_blocks_do_not_touch_earlier_gradients(name):
    spec = util.tiny_specs()[name]
    params, batch = _setup(spec, seed=1)
    _, g0 = orc.forward_backward(spec, params, batch)
    p2 = copy.deepcopy(params)
    for k in p2["blocks"][-1]:
        p2["blocks"][-1][k] = p2["blocks"][-1][k] + 0.3
    _, g1 = orc.forward_backward(spec, p2, batch)
    for b in range(len(spec["blocks"]) - 1):
        for k in g0[b]:
            assert np.array_equal(g0[b][k], g1[b][k])
    # chain: an earlier block's parameters do change a later block's gradient (through z)
    p3 = copy.deepcopy(params)
    p3["blocks"][0]["Wh"] = p3["blocks"][0]["Wh"] + 0.3      # head only: z_1 unchanged
    _, g3 = orc.forward_backward(spec, p3, batch)
    assert all(np.array_equal(g0[1][k], g3[1][k]) for k in g0[1])
    first = "W0" if name == "mlp_relu" else "W2"
    p4 = copy.deepcopy(params)
    p4["blocks"][0][first] = p4["blocks"][0][first] + 0.3
    _, g4 = orc.forward_backward(spec, p4, batch)
    assert any(not np.array_equal(g0[1][k], g4[1][k]) for k in g0[1])


def test_parallel_blocks_are_mutually_independent():
    spec = util.tiny_specs()["ctr"]
    params, batch = _setup(spec, seed=2)
    l0, g0 = orc.forward_backward(spec, params, batch)
    for victim in range(len(spec["blocks"])):
        p2 = copy.deepcopy(params)
        for k in p2["blocks"][victim]:
            p2["blocks"][victim][k] = p2["blocks"][victim][k] + 0.2
        l1, g1 = orc.forward_backward(spec, p2, batch)
        for b in range(len(spec["blocks"])):
            if b != victim:
                assert l0[b] == l1[b]
                assert all(np.array_equal(g0[b][k], g1[b][k]) for k in g0[b])


def test_stop_gradient_is_a_cut_not_independence():
    """l_2 really depends on theta_1 (finite difference non-zero) yet the oracle assigns block 1
    no gradient from l_2: block 1's gradient equals the gradient of l_1 alone."""
    spec = util.tiny_specs()["mlp_relu"]
    params, batch = _setup(spec, seed=4)
    _, grads = orc.forward_backward(spec, params, batch)
    h = 1e-5
    w = params["blocks"][0]["W1"]
    old = w[0, 0]
    w[0, 0] = old + h
    lp = orc.forward_only(spec, params, batch)
    w[0, 0] = old - h
    lm = orc.forward_only(spec, params, batch)
    w[0, 0] = old
    d_l1 = (lp[0] - lm[0]) / (2 * h)
    d_l2 = (lp[1] - lm[1]) / (2 * h)
    assert abs(d_l2) > 1e-6                       # the dependence exists ...
    assert abs(grads[0]["W1"][0, 0] - d_l1) <= 1e-8 * max(1, abs(d_l1))   # ... and is cut
    assert abs(grads[0]["W1"][0, 0] - (d_l1 + d_l2)) > 1e-7


def test_forward_losses_equal_undetached_forward():
    for name, spec in util.tiny_specs().items():
        params, batch = _setup(spec, seed=6)
        l0, _ = orc.forward_backward(spec, params, batch)
        assert np.allclose(l0, orc.forward_only(spec, params, batch), rtol=0, atol=1e-15)


# ---------------------------------------------------------------- closed forms

def test_one_layer_bce_worked_example():
    """Logistic regression on X=[[1,2],[3,-1]], y=[1,0] from w=0,b=0 with SGD lr 1e-2: values
    worked by hand (tests/golden/bce_logistic.json)."""
    gold = json.load(open(os.path.join(GOLD, "bce_logistic.json")))
    # a 'cross' block with no cross layers passes x0 through: the head sees x0.
    spec = {"dtype": "f32", "input": "dense", "topo": "chain", "batch": 2, "width": 2,
            "blocks": [{"kind": "cross", "dims": [2], "n_cross": 0, "act": "none",
                        "head": "bce", "head_out": 1}],
            "opt": {"kind": "sgd", "lr": 1e-2, "wd": 0.0, "beta1": 0.9, "beta2": 0.999, "eps": 1e-8}}
    params = {"input": {}, "blocks": [{"Wh": np.zeros((1, 2)), "bh": np.zeros(1)}]}
    batch = {"x": np.array(gold["X"], float), "y": np.array(gold["y"], float)}
    state = orc.new_opt_state(params)
    for stp in gold["steps"]:
        losses, grads, params, state = orc.step(spec, params, state, batch)
        assert abs(losses[0] - stp["loss"]) < 5e-10
        if "grad_w" in stp:
            assert np.allclose(grads[0]["Wh"][0], stp["grad_w"], atol=5e-9, rtol=0)
            assert abs(grads[0]["bh"][0] - stp["grad_b"]) < 5e-10
        if "w_after" in stp:
            assert np.allclose(params["blocks"][0]["Wh"][0], stp["w_after"], atol=1e-12, rtol=0)


def test_goodness_head_closed_forms():
    """Section 2.1's goodness objective, pinned by hand: with z = (3, 4) the score is G = 25; with
    the threshold at 25 (bh = -25) the logit is 0, so a single row costs ln 2, ds = (1/2 - y)/N
    and dz = 2 ds z; one positive and one negative row with the same z cancel exactly in dbh."""
    z = np.array([[3.0, 4.0], [3.0, 4.0]])
    p = {"bh": np.array([-25.0])}
    y = np.array([1.0, 0.0])
    loss, dz, g = orc.goodness_head(p, z, y)
    assert abs(loss - math.log(2.0)) < 1e-15
    assert np.allclose(dz, [[-1.5, -2.0], [1.5, 2.0]], atol=1e-15)      # 2 * (+-1/4) * z
    assert abs(g["bh"][0]) < 1e-16 and set(g) == {"bh"}
    # far above / below the threshold the loss is the margin itself (softplus -> identity / 0)
    big, _, _ = orc.goodness_head({"bh": np.array([0.0])}, np.array([[30.0, 40.0]]), np.array([0.0]))
    assert abs(big - 2500.0) < 1e-9
    small, dz0, _ = orc.goodness_head({"bh": np.array([-5000.0])}, np.array([[30.0, 40.0]]), np.array([0.0]))
    assert small < 1e-100
    assert np.all(np.abs(dz0) < 1e-100)


@pytest.mark.parametrize("name", list(util.tiny_specs()))
def test_zero_heads_give_ln2_or_lnV_and_zero_body_gradients(name):
    spec = util.tiny_specs()[name]
    if any(blk["head"] == "goodness" for blk in spec["blocks"]):
        pytest.skip("the goodness head has no weights to zero: its closed forms are pinned separately")
    params, batch = _setup(spec, seed=0, zero_heads=True)
    losses, grads = orc.forward_backward(spec, params, batch)
    for b, blk in enumerate(spec["blocks"]):
        want = math.log(2.0) if blk["head"] == "bce" else math.log(blk["head_out"])
        assert abs(losses[b] - want) < 1e-14
        for k, g in grads[b].items():
            if k not in ("Wh", "bh"):
                assert np.all(g == 0.0), (b, k)
        n = spec["batch"] * (spec.get("seq", 1) if spec["input"] == "tokens" else 1)
        if blk["head"] == "bce":
            y = batch["y"]
            assert np.allclose(grads[b]["bh"][0], np.sum(0.5 - y) / n, atol=1e-15)
        else:
            tgt = batch["ids"][:, 1:].reshape(-1)
            want_b = np.full(blk["head_out"], 1.0 / blk["head_out"]) - np.bincount(
                tgt, minlength=blk["head_out"]) / n
            assert np.allclose(grads[b]["bh"], want_b, atol=1e-15)


def test_transformer_with_zero_output_projections_is_identity():
    spec = util.tiny_specs()["lm"]
    params, batch = _setup(spec, seed=7)
    for p in params["blocks"]:
        for k in ("Wproj", "bproj", "W2", "b2"):
            p[k] = np.zeros_like(p[k])
        p["Wh"] = params["blocks"][0]["Wh"]
        p["bh"] = params["blocks"][0]["bh"]
    losses, _ = orc.forward_backward(spec, params, batch)
    assert abs(losses[0] - losses[1]) < 1e-15     # z_1 = z_0 => same head, same loss


def test_identity_cross_stack_reduces_to_logistic_regression_on_x0():
    spec = util.tiny_specs()["ctr"]
    params, batch = _setup(spec, seed=8)
    b = 3                                           # first cross block
    assert spec["blocks"][b]["kind"] == "cross"
    for k in params["blocks"][b]:
        if k.startswith(("Wc", "bc")):
            params["blocks"][b][k] = np.zeros_like(params["blocks"][b][k])
    losses, grads = orc.forward_backward(spec, params, batch)
    x0, y = orc.stage_input(spec, params["input"], batch)
    s = x0 @ params["blocks"][b]["Wh"][0] + params["blocks"][b]["bh"][0]
    sig = 1.0 / (1.0 + np.exp(-s))
    assert abs(losses[b] + np.mean(y * np.log(sig) + (1 - y) * np.log(1 - sig))) < 1e-14
    assert np.allclose(grads[b]["Wh"][0], x0.T @ (sig - y) / len(y), atol=1e-15)


# ---------------------------------------------------------------- conservation laws

def test_softmax_ce_rows_of_gradient_sum_to_zero_and_uniform_case():
    rng = np.random.default_rng(0)
    logits = rng.standard_normal((7, 11)) * 3
    t = rng.integers(0, 11, 7)
    loss, d = orc.softmax_ce(logits, t)
    assert np.allclose(d.sum(axis=1), 0.0, atol=1e-16)
    # brute force, no max subtraction
    brute = np.mean([math.log(sum(math.exp(v) for v in row)) - row[ti] for row, ti in zip(logits, t)])
    assert abs(loss - brute) < 1e-13
    # shift invariance
    loss2, d2 = orc.softmax_ce(logits + 100.0, t)
    assert abs(loss - loss2) < 1e-12 and np.allclose(d, d2, atol=1e-14)


def test_bce_matches_probability_form_and_is_stable():
    rng = np.random.default_rng(1)
    s = rng.standard_normal(9) * 4
    y = (rng.random(9) < 0.5).astype(float)
    loss, ds = orc.bce_with_logits(s, y)
    p = 1 / (1 + np.exp(-s))
    assert abs(loss + np.mean(y * np.log(p) + (1 - y) * np.log(1 - p))) < 1e-13
    assert np.allclose(ds, (p - y) / 9, atol=1e-16)
    big, _ = orc.bce_with_logits(np.array([800.0, -800.0]), np.array([1.0, 0.0]))
    assert big == 0.0
    big2, _ = orc.bce_with_logits(np.array([800.0]), np.array([0.0]))
    assert big2 == 800.0


def test_layernorm_invariants():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((5, 8)) * 2 + 1
    g, b = np.ones(8), np.zeros(8)
    y, cache = orc.layernorm_fwd(x, g, b)
    assert np.allclose(y.mean(axis=1), 0, atol=1e-15)
    assert np.allclose((y ** 2).mean(axis=1), x.var(axis=1) / (x.var(axis=1) + 1e-5), atol=1e-14)
    dy = rng.standard_normal((5, 8))
    dx, dg, db = orc.layernorm_bwd(dy, cache, g)
    assert np.allclose(dx.sum(axis=1), 0, atol=1e-14)             # shift invariance of LN
    # orthogonal to x-hat up to the eps in the variance: the residue is r*(dy.x-hat)*eps/(var+eps)
    xh, r = cache
    resid = r[:, 0] * (dy * xh).sum(axis=1) * (1e-5 / (x.var(axis=1) + 1e-5))
    assert np.allclose((dx * xh).sum(axis=1), resid, atol=1e-14)
    assert np.all(np.abs((dx * xh).sum(axis=1)) < 1e-4)
    assert np.allclose(db, dy.sum(axis=0))


def test_attention_is_causal_and_rows_of_ds_sum_to_zero():
    rng = np.random.default_rng(3)
    q, k, v = (rng.standard_normal((2, 2, 6, 4)) for _ in range(3))
    o, p = orc.causal_attention_fwd(q, k, v)
    assert np.allclose(p.sum(axis=-1), 1.0, atol=1e-15)
    assert np.all(np.triu(p[0, 0], k=1) == 0.0)
    k2, v2, q2 = k.copy(), v.copy(), q.copy()
    k2[:, :, 4:], v2[:, :, 4:], q2[:, :, 4:] = 9.0, -9.0, 5.0   # perturb the future
    o2, _ = orc.causal_attention_fwd(q2, k2, v2)
    assert np.array_equal(o[:, :, :4], o2[:, :, :4])
    # first position attends only to itself
    assert np.allclose(o[:, :, 0], v[:, :, 0], atol=1e-15)
    # uniform scores: position i averages v[0..i]
    o3, _ = orc.causal_attention_fwd(np.zeros_like(q), k, v)
    assert np.allclose(o3[0, 0, 3], v[0, 0, :4].mean(axis=0), atol=1e-15)
    # brute-force one (batch, head) with python loops
    dh = 4
    for i in range(6):
        w = [math.exp(sum(q[1, 1, i, c] * k[1, 1, j, c] for c in range(dh)) / 2.0) for j in range(i + 1)]
        want = sum(wj * v[1, 1, j] for j, wj in enumerate(w)) / sum(w)
        assert np.allclose(o[1, 1, i], want, atol=1e-13)
    do = rng.standard_normal(o.shape)
    dq, dk, dv = orc.causal_attention_bwd(do, q, k, v, p)
    dp = do @ np.swapaxes(v, -1, -2)
    ds = p * (dp - (dp * p).sum(-1, keepdims=True))
    assert np.allclose(ds.sum(axis=-1), 0.0, atol=1e-14)


def test_gelu_and_relu_known_values():
    u = np.array([-1.0, 0.0, 1.0, 2.0])
    # Phi(1) = 0.8413447460685429, Phi(2) = 0.9772498680518208 (standard normal table)
    want = np.array([-1.0 * (1 - 0.8413447460685429), 0.0, 0.8413447460685429, 2 * 0.9772498680518208])
    assert np.allclose(orc.act_fwd("gelu", u), want, atol=1e-15)
    assert np.array_equal(orc.act_bwd("relu", np.array([-1.0, 0.0, 2.0]), np.ones(3)), [0.0, 0.0, 1.0])
    assert abs(orc.act_bwd("gelu", np.array([0.0]), np.ones(1))[0] - 0.5) < 1e-16


def test_bias_gradient_is_column_sum_and_dw_is_outer_product_sum():
    rng = np.random.default_rng(4)
    x, w, dy = rng.standard_normal((5, 3)), rng.standard_normal((4, 3)), rng.standard_normal((5, 4))
    dx, dw, db = orc.linear_bwd(dy, x, w)
    want_dw = sum(np.outer(dy[n], x[n]) for n in range(5))
    assert np.allclose(dw, want_dw, atol=1e-14) and np.allclose(db, dy.sum(0))
    assert np.allclose(dx[2], sum(dy[2, o] * w[o] for o in range(4)), atol=1e-14)
    assert np.allclose(orc.linear_fwd(x, w, np.arange(4.0))[1, 2], x[1] @ w[2] + 2.0)


def test_ctr_input_packing_layout():
    spec = util.tiny_specs()["ctr"]
    params, batch = _setup(spec, seed=9)
    z0, y = orc.stage_input(spec, params["input"], batch)
    e, ns, nd = spec["emb_dim"], spec["n_sparse"], spec["n_dense"]
    assert z0.shape == (spec["batch"], spec["width"])
    n, t = 1, 2
    assert np.array_equal(z0[n, t * e:(t + 1) * e], params["input"][f"table{t}"][batch["ids"][n, t]])
    assert np.array_equal(z0[:, ns * e:ns * e + nd], batch["dense"].astype(np.float64))
    assert np.all(z0[:, ns * e + nd:] == 0)


def test_token_input_and_shifted_targets():
    spec = util.tiny_specs()["lm"]
    params, batch = _setup(spec, seed=9)
    z0, tgt = orc.stage_input(spec, params["input"], batch)
    ids = batch["ids"]
    assert np.array_equal(tgt, ids[:, 1:].reshape(-1))
    r = 1 * spec["seq"] + 2
    assert np.array_equal(z0[r], params["input"]["tok_emb"][ids[1, 2]] + params["input"]["pos_emb"][2])


def test_dot_interaction_features_brute_force():
    spec = util.tiny_specs()["ctr"]
    params, batch = _setup(spec, seed=10)
    blk, p = spec["blocks"][5], params["blocks"][5]
    x0, _ = orc.stage_input(spec, params["input"], batch)
    _, (dense_pad, vec, ii, jj, cache) = orc.block_forward(spec, blk, p, x0)
    feats = cache[0][0]                             # input of the first tower layer
    e, ns = spec["emb_dim"], spec["n_sparse"]
    n = 2
    proj = p["Wd"] @ x0[n, ns * e:] + p["bd"]
    vs = [proj] + [x0[n, t * e:(t + 1) * e] for t in range(ns)]
    want = [float(vs[i] @ vs[j]) for i in range(ns + 1) for j in range(i)] + list(proj)
    assert np.allclose(feats[n, :len(want)], want, atol=1e-14)
    assert np.all(feats[n, len(want):] == 0)


# ---------------------------------------------------------------- optimizer

def test_optimizer_closed_forms():
    g = np.array([0.5, -0.75])
    th = np.array([1.0, -2.0])
    z = np.zeros(2)
    sgd = {"kind": "sgd", "lr": 1e-2}
    assert np.allclose(orc.optimizer_update(sgd, th, g, z, z, 1)[0], [0.995, -1.9925], atol=1e-16)
    adam = {"kind": "adam", "lr": 1e-3, "beta1": 0.9, "beta2": 0.999, "eps": 1e-8, "wd": 0.0}
    # first Adam step is -lr * g / (|g| + eps)
    t1, m1, v1 = orc.optimizer_update(adam, th, g, z, z, 1)
    assert np.allclose(t1 - th, -1e-3 * g / (np.abs(g) + 1e-8), atol=1e-18)
    assert np.allclose(t1 - th, [-0.001, 0.001], atol=1e-10)
    # constant gradient: the update stays -lr*sign(g) (up to eps) at every t
    cur, m, v = th, z, z
    for t in range(1, 6):
        nxt, m, v = orc.optimizer_update(adam, cur, g, m, v, t)
        assert np.allclose(nxt - cur, -1e-3 * np.sign(g), atol=1e-9)
        cur = nxt
    adamw = dict(adam, kind="adamw", wd=1e-2)
    tw, _, _ = orc.optimizer_update(adamw, th, g, z, z, 1)
    assert np.allclose(tw, th * (1 - 1e-3 * 1e-2) - 1e-3 * g / (np.abs(g) + 1e-8), atol=1e-16)


def test_label_independence_sanity():
    """Labels independent of inputs: BCE near the constant predictor's entropy (NE near 1)."""
    p = 0.03
    h = -(p * math.log(p) + (1 - p) * math.log(1 - p))
    assert abs(h - 0.134742) < 1e-6
    spec = synth.ctr_spec(batch=2048, table_rows=500, tower=(32, 16, 8))
    flat = synth.init_params(spec, 0, zero_heads=True)
    params = util.structure(spec, flat)
    batch = synth.make_batch(spec, 0)
    # constant predictor at the label rate through the head bias
    for pb in params["blocks"]:
        pb["bh"] = np.array([math.log(p / (1 - p))])
    losses, _ = orc.forward_backward(spec, params, batch)
    rate = batch["y"].mean()
    want = -(rate * math.log(p) + (1 - rate) * math.log(1 - p))
    assert np.allclose(losses, want, atol=1e-12)
