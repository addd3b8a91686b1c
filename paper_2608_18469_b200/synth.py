"""Seeded synthetic workloads: model specs, tensor lists, initial parameters, batches.

This module holds NO arithmetic of the method (no forward, loss, gradient or
optimizer maths).  It only names shapes and draws random numbers, so that the
CPU oracle and the CUDA library can be fed identical bits without sharing any
code with each other.  Everything is drawn with numpy ``Generator(PCG64(seed))``.

A *spec* is a plain dict::

    {"dtype": "f32"|"bf16", "input": "dense"|"tokens"|"ctr",
     "topo": "chain"|"parallel", "batch": int,
     "width": int,                      # dense: input width
     "seq": int, "vocab": int,          # tokens
     "n_dense", "n_sparse", "table_rows", "emb_dim",   # ctr
     "train_input": bool,               # ctr with a main block: the tables are trained (by L_main)
     "blocks": [ {"kind": "mlp"|"tower"|"transformer"|"cross"|"dot"|"main",
                  "dims": [...], "act": "none"|"relu"|"gelu",
                  "n_heads": int, "n_cross": int, "head": "bce"|"ce"|"goodness",
                  "head_out": int}, ... ],
     "opt": {"kind": "sgd"|"adam"|"adamw", "lr", "beta1", "beta2", "eps", "wd"}}

Block kinds (detached blocks of Eq. 1; the local head is part of the block):
  mlp          Linear(d0->d1) act Linear(d1->d2) ... (no activation after the last)
  tower        the same with the activation after every Linear
  transformer  pre-LN block, dims = [d_model, d_ff]
  cross        n_cross DCN-v2 layers of width dims[0]
  dot          Linear(16->emb_dim) on the padded dense features, pairwise dots of
               the 27 vectors, then a tower over dims (dims[0] = padded feature count)
  main         (last block only) the undetached remainder of Eq. 2: a tower over
               [z_0 | sg[z_1] | .. | sg[z_B]] (z_0 with "reads_input") with loss L_main
"""
from __future__ import annotations

import math

import numpy as np

ADAM_DEFAULT = {"beta1": 0.9, "beta2": 0.999, "eps": 1e-8}


def _opt(kind, lr, wd=0.0):
    o = {"kind": kind, "lr": lr, "wd": wd}
    o.update(ADAM_DEFAULT)
    return o


# ----------------------------------------------------------------------------
# the five workloads (shapes of the paper's MNIST-MLP, NanoChat and CTR models)
# ----------------------------------------------------------------------------

def mlp_spec(width, hidden, n_blocks, batch, act, dtype, opt=None, head="bce"):
    blk = {"kind": "mlp", "dims": [width, hidden, width], "act": act,
           "head": head, "head_out": 1}
    return {"dtype": dtype, "input": "dense", "topo": "chain", "batch": batch,
            "width": width, "blocks": [dict(blk) for _ in range(n_blocks)],
            "opt": opt or _opt("sgd", 1e-2)}


def lm_spec(n_blocks, d_model, n_heads, d_ff, seq, batch, vocab, dtype="bf16", opt=None):
    blk = {"kind": "transformer", "dims": [d_model, d_ff], "act": "gelu",
           "n_heads": n_heads, "head": "ce", "head_out": vocab}
    return {"dtype": dtype, "input": "tokens", "topo": "chain", "batch": batch,
            "seq": seq, "vocab": vocab, "width": d_model,
            "blocks": [dict(blk) for _ in range(n_blocks)],
            "opt": opt or _opt("adamw", 1e-3, 1e-2)}


def ctr_spec(batch=4096, n_dense=13, n_sparse=26, table_rows=100000, emb_dim=64,
             tower=(1024, 512, 256), n_cross=3, dtype="bf16", opt=None):
    # x0 = [n_sparse*emb_dim embedding columns | n_dense dense | zero pad to a multiple of 16]
    dense_pad = (n_dense + 15) // 16 * 16
    w0 = n_sparse * emb_dim + dense_pad
    n_vec = n_sparse + 1
    n_feat = n_vec * (n_vec - 1) // 2 + emb_dim
    n_feat_pad = (n_feat + 7) // 8 * 8
    blocks = []
    for _ in range(3):
        blocks.append({"kind": "tower", "dims": [w0, *tower], "act": "relu",
                       "head": "bce", "head_out": 1})
    for _ in range(2):
        blocks.append({"kind": "cross", "dims": [w0], "n_cross": n_cross, "act": "none",
                       "head": "bce", "head_out": 1})
    blocks.append({"kind": "dot", "dims": [n_feat_pad, *tower], "act": "relu",
                   "head": "bce", "head_out": 1})
    return {"dtype": dtype, "input": "ctr", "topo": "parallel", "batch": batch,
            "n_dense": n_dense, "n_sparse": n_sparse, "table_rows": table_rows,
            "emb_dim": emb_dim, "width": w0, "blocks": blocks,
            "opt": opt or _opt("adam", 1e-3)}


def block_out_width(blk):
    return blk["dims"][0] if blk["kind"] in ("cross", "transformer") else blk["dims"][-1]


def with_main(spec, tower=(256, 128), reads_input=True, train_input=True, act="relu"):
    """The same model followed by the undetached remainder of Eq. 2: a main tower (activation after
    every Linear) over u = [z_0 | sg[z_1] | ... | sg[z_B]] with its own BCE head, loss L_main and the
    usual end-of-step backward; with train_input its gradient reaches the input tables through the
    z_0 columns of u.  Dense and CTR inputs (the head needs labels)."""
    s = dict(spec)
    width = (spec["width"] if reads_input else 0) + sum(block_out_width(b) for b in spec["blocks"])
    main = {"kind": "main", "dims": [width, *tower], "act": act, "head": "bce", "head_out": 1,
            "reads_input": bool(reads_input)}
    s["blocks"] = [dict(b) for b in spec["blocks"]] + [main]
    s["train_input"] = bool(train_input and reads_input and spec["input"] == "ctr")
    return s


def config(name, **kw):
    """The named workloads C1..C5 (C5 takes w= and batch=)."""
    if name == "C1":
        return mlp_spec(64, 256, 2, 256, "relu", "f32")
    if name == "C2":
        return lm_spec(4, 256, 4, 1024, 256, 16, 8192)
    if name == "C3":
        return ctr_spec()
    if name == "C4":
        return lm_spec(12, 768, 12, 3072, 1024, 8, 32768)
    if name == "C5":
        w, batch = kw.get("w", 1024), kw.get("batch", 4096)
        return mlp_spec(w, 4 * w, 8, batch, "gelu", "bf16")
    raise KeyError(name)


C5_WIDTHS = (128, 512, 1024, 2048, 4096)
C5_BATCHES = (512, 4096, 32768)


# ----------------------------------------------------------------------------
# tensor list: (block index or -1 for frozen inputs, name, shape, trainable)
# This order is the library's tensor index order.
# ----------------------------------------------------------------------------

def tensor_list(spec):
    out = []
    tin = bool(spec.get("train_input"))     # the main network's backward reaches the input tables
    if spec["input"] == "tokens":
        out.append((-1, "tok_emb", (spec["vocab"], spec["width"]), False))
        out.append((-1, "pos_emb", (spec["seq"], spec["width"]), False))
    elif spec["input"] == "ctr":
        for t in range(spec["n_sparse"]):
            out.append((-1, f"table{t}", (spec["table_rows"], spec["emb_dim"]), tin))
    for b, blk in enumerate(spec["blocks"]):
        k, dims = blk["kind"], blk["dims"]
        if k in ("mlp", "tower", "main"):
            for i, (a, o) in enumerate(zip(dims, dims[1:])):
                out.append((b, f"W{i}", (o, a), True))
                out.append((b, f"b{i}", (o,), True))
            d_out = dims[-1]
        elif k == "transformer":
            d, ff = dims
            out += [(b, "ln1_g", (d,), True), (b, "ln1_b", (d,), True),
                    (b, "Wqkv", (3 * d, d), True), (b, "bqkv", (3 * d,), True),
                    (b, "Wproj", (d, d), True), (b, "bproj", (d,), True),
                    (b, "ln2_g", (d,), True), (b, "ln2_b", (d,), True),
                    (b, "W1", (ff, d), True), (b, "b1", (ff,), True),
                    (b, "W2", (d, ff), True), (b, "b2", (d,), True)]
            d_out = d
        elif k == "cross":
            w = dims[0]
            for i in range(blk["n_cross"]):
                out.append((b, f"Wc{i}", (w, w), True))
                out.append((b, f"bc{i}", (w,), True))
            d_out = w
        elif k == "dot":
            e = spec["emb_dim"]
            out.append((b, "Wd", (e, 16), True))
            out.append((b, "bd", (e,), True))
            for i, (a, o) in enumerate(zip(dims, dims[1:])):
                out.append((b, f"W{i}", (o, a), True))
                out.append((b, f"b{i}", (o,), True))
            d_out = dims[-1]
        else:
            raise ValueError(k)
        if blk["head"] != "goodness":                  # the goodness head has no weights, only its threshold bh
            out.append((b, "Wh", (blk["head_out"], d_out), True))
        out.append((b, "bh", (blk["head_out"],), True))
    return out


def _followed_by_activation(blk, name):
    """True if this Linear weight feeds an activation (sets the init gain)."""
    k = blk["kind"]
    if not (name.startswith("W") and name[1:].isdigit()):
        return False
    i = int(name[1:])
    if k == "mlp":
        return blk["act"] != "none" and i < len(blk["dims"]) - 2
    if k in ("tower", "dot", "main"):
        return blk["act"] != "none"
    if k == "transformer":
        return name == "W1"
    return False


def init_params(spec, seed=0, zero_heads=False):
    """Initial fp32 values, drawn in tensor-index order.

    Linear W ~ U(-a, a) with a = sqrt(3 g / in): g = 2 when the Linear feeds a ReLU/GELU, else 1,
    so that the second moment of the activations is roughly kept from layer to layer (with the
    smaller 1/sqrt(in) bound an 8-deep stack without residuals or norms collapses every sample
    onto the same bias-driven vector, and the gradients become differences of nearly equal sums);
    Linear b ~ U(-1/sqrt(in), 1/sqrt(in)); LayerNorm gain 1, shift 0; CTR tables N(0, (1/8)^2);
    token embedding N(0, 1); position embedding N(0, 0.1^2); the goodness head's threshold bh = minus
    half the width of z_b (the sum of squares of a unit-variance z_b is about that width).
    Returns a list of float32 arrays aligned with ``tensor_list(spec)``.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    vals = []
    fan_in = fan_out = None
    for (b, name, shape, _tr) in tensor_list(spec):
        if name == "tok_emb":
            v = rng.standard_normal(shape)
        elif name == "pos_emb":
            v = 0.1 * rng.standard_normal(shape)
        elif name.startswith("table"):
            v = 0.125 * rng.standard_normal(shape)
        elif name.endswith("_g"):
            v = np.ones(shape)
        elif name.endswith("_b") and name.startswith("ln"):
            v = np.zeros(shape)
        elif len(shape) == 2:                       # Linear weight [out, in]
            fan_in, fan_out = shape[1], shape[0]
            gain = 2.0 if _followed_by_activation(spec["blocks"][b], name) else 1.0
            bound = math.sqrt(3.0 * gain / fan_in)
            v = rng.uniform(-bound, bound, shape)
            if zero_heads and name == "Wh":
                v = np.zeros(shape)
        else:                                       # Linear bias
            bound = 1.0 / math.sqrt(fan_in)
            v = rng.uniform(-bound, bound, shape)
            if name == "bh" and b >= 0 and spec["blocks"][b]["head"] == "goodness":
                v = np.full(shape, -0.5 * fan_out)
            if zero_heads and name == "bh":
                v = np.zeros(shape)
        vals.append(np.ascontiguousarray(v, dtype=np.float32))
    return vals


# ----------------------------------------------------------------------------
# batches
# ----------------------------------------------------------------------------

def bf16_round(a):
    """Round float32 values to the nearest bfloat16 (ties to even), returned as float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return r.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(a):
    """float32 array (already bf16-representable or not) -> uint16 bfloat16 bit patterns (RNE)."""
    return (bf16_round(a).view(np.uint32) >> 16).astype(np.uint16)


_ZIPF_CACHE = {}


def _zipf_cdf(n, s):
    key = (n, s)
    if key not in _ZIPF_CACHE:
        p = np.arange(1, n + 1, dtype=np.float64) ** (-s)
        _ZIPF_CACHE[key] = np.cumsum(p / p.sum())
    return _ZIPF_CACHE[key]


def make_batch(spec, seed=0, index=0, label_p=None):
    """One batch as a dict of numpy arrays (what the caller would stage on the device).

    dense  : x [batch, width] float32 ~ N(0,1) (rounded to bf16 values when dtype is bf16),
             y [batch] float32 ~ Bernoulli(p), p = 0.5
    tokens : ids [batch, seq+1] int32 ~ U{0..vocab-1}; inputs ids[:, :seq], targets ids[:, 1:]
    ctr    : dense [batch, n_dense] float32 = log1p(exp(N(0,1))) (a lognormal(0,1) through log1p),
             ids [batch, n_sparse] int32, each column bounded Zipf(s=1.1) ranks mapped through a
             fixed per-table permutation; y ~ Bernoulli(0.03)
    """
    rng = np.random.Generator(np.random.PCG64([seed, 1000 + index]))
    nb = spec["batch"]
    if spec["input"] == "dense":
        x = rng.standard_normal((nb, spec["width"])).astype(np.float32)
        if spec["dtype"] == "bf16":
            x = bf16_round(x)
        p = 0.5 if label_p is None else label_p
        y = (rng.random(nb) < p).astype(np.float32)
        return {"x": x, "y": y}
    if spec["input"] == "tokens":
        ids = rng.integers(0, spec["vocab"], (nb, spec["seq"] + 1), dtype=np.int64).astype(np.int32)
        return {"ids": ids}
    if spec["input"] == "ctr":
        dense = np.log1p(np.exp(rng.standard_normal((nb, spec["n_dense"])))).astype(np.float32)
        rows = spec["table_rows"]
        cdf = _zipf_cdf(rows, 1.1)
        ids = np.empty((nb, spec["n_sparse"]), dtype=np.int32)
        for t in range(spec["n_sparse"]):
            rank = np.minimum(np.searchsorted(cdf, rng.random(nb)), rows - 1)
            perm = np.random.Generator(np.random.PCG64([7, t])).permutation(rows)
            ids[:, t] = perm[rank]
        p = 0.03 if label_p is None else label_p
        y = (rng.random(nb) < p).astype(np.float32)
        return {"dense": dense, "ids": ids, "y": y}
    raise ValueError(spec["input"])


# ----------------------------------------------------------------------------
# algorithmic FLOPs of one step (2*m*n*k per matmul; causal attention at its
# lower-triangular half; no dgrad into a detached block input)
# ----------------------------------------------------------------------------

def step_flops(spec):
    nb = spec["batch"] * (spec.get("seq", 1) if spec["input"] == "tokens" else 1)

    def lin(i, o):
        return 2 * nb * i * o

    total = 0
    for blk in spec["blocks"]:
        k, dims = blk["kind"], blk["dims"]
        if k == "main":                      # the usual backward: the first layer's dgrad is needed too
            f = sum(lin(a, o) for a, o in zip(dims, dims[1:])) + lin(dims[-1], blk["head_out"])
            total += 3 * f
        elif k in ("mlp", "tower"):
            f = sum(lin(a, o) for a, o in zip(dims, dims[1:])) + lin(dims[-1], blk["head_out"])
            total += f + 2 * f - lin(dims[0], dims[1])
        elif k == "transformer":
            d, ff = dims
            t, bt, h = spec["seq"], spec["batch"], blk["n_heads"]
            dh = d // h
            linf = lin(d, 3 * d) + lin(d, d) + lin(d, ff) + lin(ff, d)
            att = 2 * 2 * bt * h * (t * (t + 1) // 2) * dh
            head = lin(d, blk["head_out"])
            total += 3 * (linf + att + head)
        elif k == "cross":
            w = dims[0]
            f = blk["n_cross"] * lin(w, w) + lin(w, 1)
            total += f + 2 * f - lin(w, w)
        elif k == "dot":
            e, nv = spec["emb_dim"], spec["n_sparse"] + 1
            f0 = lin(16, e) + 2 * nb * nv * nv * e
            f = sum(lin(a, o) for a, o in zip(dims, dims[1:])) + lin(dims[-1], 1)
            total += f0 + f + 2 * f + 2 * (2 * nb * nv * nv * e) + lin(16, e)
    return total


def rel_l2(a, b):
    """||a-b||2 / max(||b||2, 1e-12*sqrt(n)) in float64 (the parity metric)."""
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    den = max(float(np.linalg.norm(b)), 1e-12 * math.sqrt(max(b.size, 1)))
    return float(np.linalg.norm(a - b)) / den
