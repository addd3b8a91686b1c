"""CPU oracle for one training step of a network of detached blocks with local losses.

TEST INFRASTRUCTURE ONLY.  This file is the plain definition the CUDA library is
checked against.  It shares no code with the CUDA path, imports nothing from the
package, and may be imported only by the tests, the smoke check and the
benchmark's cpu-baseline leg.  Everything is float64 numpy; matmul, erf and exp
are the only library primitives; there is no blocking, fusion or reordering.

What it computes (paper Section 2.1, Eq. 1, and Section 2.2, Eq. 2):

  z_0 = x (the input embedding);   z_b = f_b(sg[z_{b-1}]; theta_b),  b = 1..B
  l_b = loss(head_b(z_b), target)            (local loss on the undetached z_b)
  g_b = d l_b / d theta_b                    (within block b only: sg has zero Jacobian,
                                              so nothing reaches z_{b-1} or other blocks)
  theta_b <- optimizer(theta_b, g_b)

Optionally the model ends with the UNDETACHED REMAINDER of Section 2.2 (Eq. 2): a main network
(block kind "main", always last) that reads u = [z_0 | sg[z_1] | ... | sg[z_B]] (z_0 only with
"reads_input"), a tower Linear-act-...-Linear-act with its own head, whose loss is L_main.  Its
backward is the usual one: it trains the main network's own parameters and, through the
undetached z_0 columns of u, the producer of z_0 -- the embedding tables (spec["train_input"]):
d L_main / d table_t[r] is the sum of the z_0-gradient slices of every sample whose id in
column t is r (a scatter-add; repeated ids add up).  The sg[z_b] columns pass nothing back, and
the detached blocks still see z_0 through sg (Eq. 1), so the tables receive gradient from L_main
alone.  Tables are updated on the rows the batch touched only (untouched rows keep their values
and moments; the bias correction uses the global step count).

ERASE itself is only a schedule of this computation (early backward per block on
side streams), so it has no separate oracle: every schedule must reproduce these
numbers.  With all lambda_i = 1 and no L_main, g is also the gradient of Eq. 2's
aggregate objective with each z_{b-1} held constant inside block b.

The paper does not fix f_b, the heads, the losses or the optimizer; the readings
used here (mean reductions, exact-erf GELU, biased-variance LayerNorm with eps
1e-5, pre-LN transformer, full-rank DCN-v2 cross layers, strict-lower-triangle
dot interaction, PyTorch-convention Adam/AdamW; heads: Linear + mean BCE with
logits, Linear + mean softmax cross-entropy, or Section 2.1's example itself,
BCE on the goodness score G_b = sum_j z_bj^2 with a trainable threshold) are the
ones listed in the design notes of this repository.

Pins (tests/test_oracle_*.py): central finite differences on every parameter of
every block kind; torch CPU autograd in float64 with .detach() between blocks;
the stop-gradient invariants; hand-derived closed forms for one-layer logistic
regression, zero heads (ln 2, ln V), identity cross layers, the goodness head
at and far from its threshold; conservation laws of softmax, LayerNorm and
attention; Adam's first step.

Parameter containers: ``params = {"input": {name: array}, "blocks": [{name: array}, ...]}``.
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf

F = np.float64


# ----------------------------------------------------------------------------
# elementary layers: forward value and reverse-mode rule, each as its definition
# ----------------------------------------------------------------------------

def linear_fwd(x, w, b):
    """Y = X W^T + b   (W is [out, in])."""
    return x @ w.T + b


def linear_bwd(dy, x, w):
    """dX = dY W ; dW = dY^T X ; db = column sums of dY."""
    return dy @ w, dy.T @ x, dy.sum(axis=0)


def act_fwd(kind, u):
    if kind == "none":
        return u
    if kind == "relu":
        return np.maximum(u, 0.0)
    if kind == "gelu":                                   # exact form: u * Phi(u)
        return u * 0.5 * (1.0 + erf(u / np.sqrt(2.0)))
    raise ValueError(kind)


def act_bwd(kind, u, dy):
    if kind == "none":
        return dy
    if kind == "relu":                                   # derivative 0 at exactly 0
        return dy * (u > 0.0)
    if kind == "gelu":                                   # Phi(u) + u * phi(u)
        cdf = 0.5 * (1.0 + erf(u / np.sqrt(2.0)))
        pdf = np.exp(-0.5 * u * u) / np.sqrt(2.0 * np.pi)
        return dy * (cdf + u * pdf)
    raise ValueError(kind)


def bce_with_logits(s, y):
    """Mean over rows of softplus(s) - y*s (stable form); gradient (sigmoid(s) - y)/N."""
    n = s.shape[0]
    loss = np.mean(np.maximum(s, 0.0) - s * y + np.log1p(np.exp(-np.abs(s))))
    sig = np.where(s >= 0, 1.0 / (1.0 + np.exp(-np.abs(s))),
                   np.exp(-np.abs(s)) / (1.0 + np.exp(-np.abs(s))))
    return loss, (sig - y) / n


def softmax_ce(logits, t):
    """Mean over rows of logsumexp(row) - row[t]; gradient (softmax - onehot)/N."""
    n = logits.shape[0]
    mx = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - mx)
    se = e.sum(axis=1, keepdims=True)
    lse = (mx + np.log(se))[:, 0]
    loss = np.mean(lse - logits[np.arange(n), t])
    d = e / se
    d[np.arange(n), t] -= 1.0
    return loss, d / n


LN_EPS = 1e-5


def layernorm_fwd(x, g, b):
    mu = x.mean(axis=1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=1, keepdims=True)     # biased variance
    r = 1.0 / np.sqrt(var + LN_EPS)
    xh = (x - mu) * r
    return xh * g + b, (xh, r)


def layernorm_bwd(dy, cache, g):
    xh, r = cache
    gg = dy * g
    dx = r * (gg - gg.mean(axis=1, keepdims=True) - xh * (gg * xh).mean(axis=1, keepdims=True))
    return dx, (dy * xh).sum(axis=0), dy.sum(axis=0)


def causal_attention_fwd(q, k, v):
    """q, k, v: [batch, heads, T, dh].  S = QK^T/sqrt(dh), masked j<=i, P = softmax, O = PV."""
    dh = q.shape[-1]
    t = q.shape[-2]
    s = q @ np.swapaxes(k, -1, -2) / np.sqrt(dh)
    mask = np.tril(np.ones((t, t), dtype=bool))
    s = np.where(mask, s, -np.inf)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    return p @ v, p


def causal_attention_bwd(do, q, k, v, p):
    dh = q.shape[-1]
    dv = np.swapaxes(p, -1, -2) @ do
    dp = do @ np.swapaxes(v, -1, -2)
    ds = p * (dp - (dp * p).sum(axis=-1, keepdims=True))
    dq = ds @ k / np.sqrt(dh)
    dk = np.swapaxes(ds, -1, -2) @ q / np.sqrt(dh)
    return dq, dk, dv


# ----------------------------------------------------------------------------
# input staging: z_0 = x
# ----------------------------------------------------------------------------

def stage_input(spec, inp, batch):
    """Returns (z0 [rows, width], target).  Frozen inputs sit under sg[z_0]: no gradient."""
    kind = spec["input"]
    if kind == "dense":
        return np.asarray(batch["x"], F), np.asarray(batch["y"], F)
    if kind == "tokens":
        ids = np.asarray(batch["ids"])
        tin, tgt = ids[:, :-1], ids[:, 1:]
        t = tin.shape[1]
        z0 = np.asarray(inp["tok_emb"], F)[tin] + np.asarray(inp["pos_emb"], F)[None, :t, :]
        return z0.reshape(-1, z0.shape[-1]), tgt.reshape(-1)
    if kind == "ctr":
        ids = np.asarray(batch["ids"])
        nb = ids.shape[0]
        cols = [np.asarray(inp[f"table{t}"], F)[ids[:, t]] for t in range(spec["n_sparse"])]
        dense = np.asarray(batch["dense"], F)
        pad = spec["width"] - spec["n_sparse"] * spec["emb_dim"] - spec["n_dense"]
        z0 = np.concatenate(cols + [dense, np.zeros((nb, pad), F)], axis=1)
        return z0, np.asarray(batch["y"], F)
    raise ValueError(kind)


# ----------------------------------------------------------------------------
# blocks: body forward/backward.  backward returns parameter gradients only;
# the gradient with respect to the block input is never formed into z_{b-1}.
# ----------------------------------------------------------------------------

def _mlp_fwd(blk, p, z, act_last, prefix="W", bprefix="b"):
    n_lin = len(blk["dims"]) - 1
    cache = []
    h = z
    for i in range(n_lin):
        u = linear_fwd(h, p[f"{prefix}{i}"], p[f"{bprefix}{i}"])
        use_act = act_last or i < n_lin - 1
        y = act_fwd(blk["act"], u) if use_act else u
        cache.append((h, u, use_act))
        h = y
    return h, cache


def _mlp_bwd(blk, p, cache, dz, grads, prefix="W", bprefix="b", need_dx=False):
    d = dz
    for i in reversed(range(len(cache))):
        h, u, use_act = cache[i]
        du = act_bwd(blk["act"], u, d) if use_act else d
        dx, dw, db = linear_bwd(du, h, p[f"{prefix}{i}"])
        grads[f"{prefix}{i}"], grads[f"{bprefix}{i}"] = dw, db
        d = dx
    return d if need_dx else None


def _split_heads(x, bt, t, h):
    return x.reshape(bt, t, h, -1).transpose(0, 2, 1, 3)


def _merge_heads(x):
    bt, h, t, dh = x.shape
    return x.transpose(0, 2, 1, 3).reshape(bt * t, h * dh)


def _transformer_fwd(spec, blk, p, z):
    d = blk["dims"][0]
    bt, t, h = spec["batch"], spec["seq"], blk["n_heads"]
    a, c1 = layernorm_fwd(z, p["ln1_g"], p["ln1_b"])
    qkv = linear_fwd(a, p["Wqkv"], p["bqkv"])
    q, k, v = (_split_heads(qkv[:, i * d:(i + 1) * d], bt, t, h) for i in range(3))
    o4, prob = causal_attention_fwd(q, k, v)
    o = _merge_heads(o4)
    hres = z + linear_fwd(o, p["Wproj"], p["bproj"])
    m, c2 = layernorm_fwd(hres, p["ln2_g"], p["ln2_b"])
    u = linear_fwd(m, p["W1"], p["b1"])
    g = act_fwd("gelu", u)
    zout = hres + linear_fwd(g, p["W2"], p["b2"])
    return zout, (a, c1, q, k, v, prob, o, m, c2, u, g)


def _transformer_bwd(spec, blk, p, cache, dz, grads):
    a, c1, q, k, v, prob, o, m, c2, u, g = cache
    bt, t, h = spec["batch"], spec["seq"], blk["n_heads"]
    dg, grads["W2"], grads["b2"] = linear_bwd(dz, g, p["W2"])
    du = act_bwd("gelu", u, dg)
    dm, grads["W1"], grads["b1"] = linear_bwd(du, m, p["W1"])
    dln2, grads["ln2_g"], grads["ln2_b"] = layernorm_bwd(dm, c2, p["ln2_g"])
    dh = dz + dln2                                         # residual: z' = h + MLP(LN2(h))
    do, grads["Wproj"], grads["bproj"] = linear_bwd(dh, o, p["Wproj"])
    dq, dk, dv = causal_attention_bwd(_split_heads(do, bt, t, h), q, k, v, prob)
    dqkv = np.concatenate([_merge_heads(dq), _merge_heads(dk), _merge_heads(dv)], axis=1)
    da, grads["Wqkv"], grads["bqkv"] = linear_bwd(dqkv, a, p["Wqkv"])
    _dx, grads["ln1_g"], grads["ln1_b"] = layernorm_bwd(da, c1, p["ln1_g"])
    # _dx + dh would be d l_b / d z_{b-1}: discarded, the input is detached.


def _cross_fwd(blk, p, x0):
    xl = x0
    cache = []
    for i in range(blk["n_cross"]):
        u = linear_fwd(xl, p[f"Wc{i}"], p[f"bc{i}"])
        cache.append(xl)
        xl = x0 * u + xl                                    # x_{l+1} = x0 (.) (W x_l + b) + x_l
    return xl, cache


def _cross_bwd(blk, p, x0, cache, dz, grads):
    d = dz
    for i in reversed(range(blk["n_cross"])):
        tt = d * x0                                         # through the Hadamard factor u
        dx, grads[f"Wc{i}"], grads[f"bc{i}"] = linear_bwd(tt, cache[i], p[f"Wc{i}"])
        d = dx + d                                          # skip path; d/dx0 discarded (detached)


def _dot_fwd(spec, blk, p, x0):
    e, ns = spec["emb_dim"], spec["n_sparse"]
    nb = x0.shape[0]
    dense_pad = x0[:, ns * e:]                              # the 16 padded dense columns
    proj = linear_fwd(dense_pad, p["Wd"], p["bd"])          # [nb, e]
    vec = np.concatenate([proj[:, None, :], x0[:, :ns * e].reshape(nb, ns, e)], axis=1)
    gram = vec @ np.swapaxes(vec, 1, 2)                     # [nb, 27, 27]
    ii, jj = np.tril_indices(ns + 1, k=-1)                  # strict lower triangle, row-major
    feats = np.concatenate([gram[:, ii, jj], proj], axis=1)
    width = blk["dims"][0]
    feats = np.concatenate([feats, np.zeros((nb, width - feats.shape[1]), F)], axis=1)
    out, cache = _mlp_fwd(blk, p, feats, act_last=True)
    return out, (dense_pad, vec, ii, jj, cache)


def _dot_bwd(spec, blk, p, cache_all, dz, grads):
    dense_pad, vec, ii, jj, cache = cache_all
    e = spec["emb_dim"]
    nb, nv, _ = vec.shape
    dfeat = _mlp_bwd(blk, p, cache, dz, grads, need_dx=True)
    npair = ii.shape[0]
    dgram = np.zeros((nb, nv, nv), F)
    dgram[:, ii, jj] = dfeat[:, :npair]
    dvec = (dgram + np.swapaxes(dgram, 1, 2)) @ vec         # G = V V^T
    dproj = dvec[:, 0, :] + dfeat[:, npair:npair + e]       # vector 0 is the dense projection
    _dx, grads["Wd"], grads["bd"] = linear_bwd(dproj, dense_pad, p["Wd"])
    # rows 1.. of dvec belong to the frozen embedding rows: discarded.


def block_forward(spec, blk, p, zin):
    k = blk["kind"]
    if k == "mlp":
        return _mlp_fwd(blk, p, zin, act_last=False)
    if k == "tower":
        return _mlp_fwd(blk, p, zin, act_last=True)
    if k == "transformer":
        return _transformer_fwd(spec, blk, p, zin)
    if k == "cross":
        return _cross_fwd(blk, p, zin)
    if k == "dot":
        return _dot_fwd(spec, blk, p, zin)
    raise ValueError(k)


def block_backward(spec, blk, p, zin, cache, dz, grads):
    k = blk["kind"]
    if k in ("mlp", "tower"):
        _mlp_bwd(blk, p, cache, dz, grads)
    elif k == "transformer":
        _transformer_bwd(spec, blk, p, cache, dz, grads)
    elif k == "cross":
        _cross_bwd(blk, p, zin, cache, dz, grads)
    elif k == "dot":
        _dot_bwd(spec, blk, p, cache, dz, grads)
    else:
        raise ValueError(k)


def goodness_head(p, z, target):
    """Section 2.1: binary cross-entropy applied to the goodness score G_b = sum_j z_bj^2.
    The logit is s_n = G_n + bh (bh: trainable scalar, minus the threshold); labels 1 = positive.
    dG/dz = 2 z, so dz = 2 ds z; the threshold's gradient is sum_n ds_n."""
    s = np.sum(z * z, axis=1) + p["bh"][0]
    loss, ds = bce_with_logits(s, target)
    return loss, 2.0 * ds[:, None] * z, {"bh": np.array([ds.sum()])}


def head_loss(blk, p, z, target):
    """Local head applied to z_b and its loss.  Returns loss, dz, {Wh, bh grads}."""
    if blk["head"] == "goodness":
        return goodness_head(p, z, target)
    s = linear_fwd(z, p["Wh"], p["bh"])
    if blk["head"] == "bce":
        loss, ds = bce_with_logits(s[:, 0], target)
        ds = ds[:, None]
    elif blk["head"] == "ce":
        loss, ds = softmax_ce(s, target)
    else:
        raise ValueError(blk["head"])
    dz, dwh, dbh = linear_bwd(ds, z, p["Wh"])
    return loss, dz, {"Wh": dwh, "bh": dbh}


# ----------------------------------------------------------------------------
# the step
# ----------------------------------------------------------------------------

def main_input(blk, z0, outs):
    """u = [z_0 | sg[z_1] | ... | sg[z_B]]: the value only; which columns pass a gradient back is
    decided in the backward (the z_0 columns, and only with reads_input)."""
    return np.concatenate(([z0] if blk.get("reads_input") else []) + outs, axis=1)


def input_gradients(spec, batch, dz0):
    """Gradient of the producer of z_0 from dz0 = d L_main / d z_0 [rows, width].
    ctr   : table_t[r] receives the sum over the samples n with ids[n, t] = r of dz0[n, t*e:(t+1)*e]
    tokens: tok_emb[r] receives the rows of dz0 whose input token is r; pos_emb[t] the sum over sequences
    dense : z_0 is data, nothing to train."""
    kind = spec["input"]
    if kind == "ctr":
        ids = np.asarray(batch["ids"])
        e = spec["emb_dim"]
        out = {}
        for t in range(spec["n_sparse"]):
            g = np.zeros((spec["table_rows"], e), F)
            for n in range(ids.shape[0]):                    # the scatter-add, written out
                g[ids[n, t]] += dz0[n, t * e:(t + 1) * e]
            out[f"table{t}"] = g
        return out
    if kind == "tokens":
        ids = np.asarray(batch["ids"])[:, :-1]
        bt, t = ids.shape
        d3 = dz0.reshape(bt, t, -1)
        gt = np.zeros((spec["vocab"], d3.shape[-1]), F)
        for b in range(bt):
            for i in range(t):
                gt[ids[b, i]] += d3[b, i]
        return {"tok_emb": gt, "pos_emb": d3.sum(axis=0)}
    return {}


def forward_backward(spec, params, batch, want_input=False):
    """Losses l_1..l_B (then L_main) and gradients (a dict per block) for one batch.
    With want_input a third value: {name: gradient} of the trainable input tables (from L_main)."""
    inp = params.get("input", {})
    z0, target = stage_input(spec, inp, batch)
    losses, grads, outs = [], [], []
    ginput = {}
    z = z0
    for blk, p64 in zip(spec["blocks"], params["blocks"]):
        p = {k: np.asarray(v, F) for k, v in p64.items()}
        if blk["kind"] == "main":                               # the undetached remainder: usual backward
            u = main_input(blk, z0, outs)
            zout, cache = _mlp_fwd(blk, p, u, act_last=True)
            loss, dz, g = head_loss(blk, p, zout, target)
            du = _mlp_bwd(blk, p, cache, dz, g, need_dx=True)
            if blk.get("reads_input") and spec.get("train_input"):
                ginput = input_gradients(spec, batch, du[:, :z0.shape[1]])   # the sg[z_b] columns pass nothing back
            losses.append(float(loss))
            grads.append(g)
            continue
        zin = z0 if spec["topo"] == "parallel" else z       # value of sg[z_{b-1}]
        zout, cache = block_forward(spec, blk, p, zin)
        loss, dz, g = head_loss(blk, p, zout, target)
        block_backward(spec, blk, p, zin, cache, dz, g)
        losses.append(float(loss))
        grads.append(g)
        outs.append(zout)
        z = zout                                            # passed on detached
    return (losses, grads, ginput) if want_input else (losses, grads)


def forward_only(spec, params, batch):
    """Per-block losses with no notion of detachment (sg is the identity going forward)."""
    inp = params.get("input", {})
    z0, target = stage_input(spec, inp, batch)
    out = []
    z = z0
    outs = []
    for blk, p64 in zip(spec["blocks"], params["blocks"]):
        p = {k: np.asarray(v, F) for k, v in p64.items()}
        if blk["kind"] == "main":
            zm, _ = _mlp_fwd(blk, p, main_input(blk, z0, outs), act_last=True)
            s = linear_fwd(zm, p["Wh"], p["bh"])
            out.append(float(bce_with_logits(s[:, 0], target)[0] if blk["head"] == "bce" else softmax_ce(s, target)[0]))
            continue
        zin = z0 if spec["topo"] == "parallel" else z
        z, _ = block_forward(spec, blk, p, zin)
        outs.append(z)
        if blk["head"] == "goodness":
            out.append(float(goodness_head(p, z, target)[0]))
            continue
        s = linear_fwd(z, p["Wh"], p["bh"])
        if blk["head"] == "bce":
            out.append(float(bce_with_logits(s[:, 0], target)[0]))
        else:
            out.append(float(softmax_ce(s, target)[0]))
    return out


def new_opt_state(params):
    return {"t": 0,
            "m": [{k: np.zeros_like(np.asarray(v, F)) for k, v in p.items()} for p in params["blocks"]],
            "v": [{k: np.zeros_like(np.asarray(v, F)) for k, v in p.items()} for p in params["blocks"]],
            "m_in": {k: np.zeros_like(np.asarray(v, F)) for k, v in params.get("input", {}).items()},
            "v_in": {k: np.zeros_like(np.asarray(v, F)) for k, v in params.get("input", {}).items()}}


def optimizer_update_rows(opt, theta, g, touched, m, v, t):
    """The same update on the rows `touched` (boolean mask) only: untouched rows keep their
    values and moments.  t is the global step count."""
    th2, m2, v2 = optimizer_update(opt, theta[touched], g[touched], m[touched], v[touched], t)
    theta, m, v = theta.copy(), m.copy(), v.copy()
    theta[touched], m[touched], v[touched] = th2, m2, v2
    return theta, m, v


def touched_rows(spec, batch, name):
    """Rows of input table `name` that the batch reads."""
    ids = np.asarray(batch["ids"])
    if spec["input"] == "ctr":
        mask = np.zeros(spec["table_rows"], bool)
        mask[ids[:, int(name[5:])]] = True
        return mask
    if name == "tok_emb":
        mask = np.zeros(spec["vocab"], bool)
        mask[ids[:, :-1].ravel()] = True
        return mask
    return np.ones(spec["seq"], bool)


def optimizer_update(opt, theta, g, m, v, t):
    """One tensor's update; t counts from 1.  Returns new (theta, m, v).

    sgd   : theta - lr g
    adam  : m = b1 m + (1-b1) g ; v = b2 v + (1-b2) g^2 ;
            theta - lr (m/(1-b1^t)) / (sqrt(v/(1-b2^t)) + eps)
    adamw : the same after the decoupled shrink theta (1 - lr wd)
    """
    lr = opt["lr"]
    if opt["kind"] == "sgd":
        return theta - lr * g, m, v
    b1, b2, eps = opt["beta1"], opt["beta2"], opt["eps"]
    if opt["kind"] == "adamw":
        theta = theta * (1.0 - lr * opt["wd"])
    elif opt["kind"] != "adam":
        raise ValueError(opt["kind"])
    m = b1 * m + (1.0 - b1) * g
    v = b2 * v + (1.0 - b2) * g * g
    mhat = m / (1.0 - b1 ** t)
    vhat = v / (1.0 - b2 ** t)
    return theta - lr * mhat / (np.sqrt(vhat) + eps), m, v


def step(spec, params, state, batch):
    """One training step.  Returns (losses, grads, new_params, new_state); inputs untouched."""
    losses, grads, ginput = forward_backward(spec, params, batch, want_input=True)
    t = state["t"] + 1
    new_p = {"input": dict(params.get("input", {})), "blocks": []}
    new_s = {"t": t, "m": [], "v": [], "m_in": dict(state.get("m_in", {})), "v_in": dict(state.get("v_in", {}))}
    for k, g in ginput.items():                                 # trainable input tables: the rows this batch touched
        th, m1, v1 = optimizer_update_rows(spec["opt"], np.asarray(params["input"][k], F), g, touched_rows(spec, batch, k),
                                           np.asarray(state["m_in"][k], F), np.asarray(state["v_in"][k], F), t)
        new_p["input"][k], new_s["m_in"][k], new_s["v_in"][k] = th, m1, v1
    for b, p in enumerate(params["blocks"]):
        np_, nm, nv = {}, {}, {}
        for k in p:
            np_[k], nm[k], nv[k] = optimizer_update(spec["opt"], np.asarray(p[k], F), grads[b][k],
                                                    state["m"][b][k], state["v"][b][k], t)
        new_p["blocks"].append(np_)
        new_s["m"].append(nm)
        new_s["v"].append(nv)
    return losses, grads, new_p, new_s
