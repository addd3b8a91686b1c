"""Helpers shared by the tests: flat tensor list <-> the oracle's parameter containers."""
import numpy as np

from paper_2608_18469_b200 import synth


def structure(spec, flat):
    """Flat list (tensor-index order) -> {"input": {...}, "blocks": [{...}]} in float64."""
    out = {"input": {}, "blocks": [dict() for _ in spec["blocks"]]}
    for (b, name, _shape, _tr), v in zip(synth.tensor_list(spec), flat):
        (out["input"] if b < 0 else out["blocks"][b])[name] = np.asarray(v, np.float64)
    return out


def flatten_blocks(spec, per_block):
    """List of per-block dicts -> flat list over the trainable tensors, tensor-index order."""
    return [per_block[b][name] for (b, name, _s, tr) in synth.tensor_list(spec) if tr]


def trainable_index(spec):
    return [i for i, (_b, _n, _s, tr) in enumerate(synth.tensor_list(spec)) if tr]


def tiny_specs():
    """One tiny instance per block kind (a few rows, a few columns), chain or parallel."""
    s = {}
    s["mlp_relu"] = synth.mlp_spec(4, 6, 2, 3, "relu", "f32")
    s["mlp_gelu"] = synth.mlp_spec(4, 6, 3, 3, "gelu", "f32")
    s["lm"] = synth.lm_spec(2, 4, 2, 6, 3, 2, 5, dtype="f32")
    s["ctr"] = synth.ctr_spec(batch=3, n_dense=2, n_sparse=3, table_rows=7, emb_dim=4,
                              tower=(6, 5, 4), n_cross=2, dtype="f32")
    s["mlp_goodness"] = synth.mlp_spec(4, 6, 2, 5, "relu", "f32", head="goodness")
    s["tower_goodness"] = synth.mlp_spec(4, 6, 2, 5, "gelu", "f32", head="goodness")
    for blk in s["tower_goodness"]["blocks"]:
        blk["kind"] = "tower"       # the activation also follows the last Linear: z_b = act(u)
    return s


def operand_params(spec, params):
    """The parameter values the bf16 path actually multiplies with.

    A bf16 model keeps fp32 master parameters and feeds its GEMMs bf16 roundings of the weight
    matrices (refreshed by the optimizer).  Those roundings are the operands ("bf16 operands,
    fp32 accumulation"), so parity evaluates the oracle at the same operand values; gradients are
    then applied to the fp32 masters.  Biases, LayerNorm parameters and the 1-wide BCE head vector
    are consumed in fp32 and stay unrounded.  fp32 models are returned unchanged.
    """
    if spec["dtype"] != "bf16":
        return params
    inp = params["input"]
    if spec["input"] == "ctr":      # x0 is stored in bf16: the frozen table rows are operands too
        inp = {k: synth.bf16_round(v.astype(np.float32)).astype(np.float64) for k, v in inp.items()}
    out = {"input": inp, "blocks": []}
    for blk, p in zip(spec["blocks"], params["blocks"]):
        q = {}
        for k, v in p.items():
            if v.ndim == 2 and not (k == "Wh" and blk["head"] == "bce"):
                q[k] = synth.bf16_round(v.astype(np.float32)).astype(np.float64)
            else:
                q[k] = v
        out["blocks"].append(q)
    return out


def operand_batch(spec, batch):
    """The batch as the bf16 path sees it: CTR dense features are packed into the bf16 x0."""
    if spec["dtype"] == "bf16" and spec["input"] == "ctr":
        return dict(batch, dense=synth.bf16_round(batch["dense"]))
    return batch
