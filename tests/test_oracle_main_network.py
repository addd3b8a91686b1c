"""Pins for the undetached remainder of Eq. 2 in the oracle: a main network over
[z_0 | sg[z_1] | ... | sg[z_B]] with loss L_main, trained by the usual backward, whose gradient
reaches the embedding tables through the z_0 columns (a scatter-add by id).  Pinned against
central finite differences, torch autograd (index lookups, .detach(), one backward on the summed
loss of Eq. 2), a hand-worked case with a repeated id, and the stop-gradient invariants."""
import copy

import numpy as np
import pytest
import torch
import torch.nn.functional as TF

from oracle import erase_oracle as orc
from paper_2608_18469_b200 import synth
from tests import util
from tests.test_oracle_vs_torch import _torch_block

torch.set_default_dtype(torch.float64)


def _ctr(batch=6, rows=4, seed=0, opt=None):
    base = synth.ctr_spec(batch=batch, n_dense=2, n_sparse=3, table_rows=rows, emb_dim=4, tower=(6, 5, 4), n_cross=2,
                          dtype="f32", opt=opt)
    spec = synth.with_main(base, tower=(7, 5))
    params = util.structure(spec, synth.init_params(spec, seed))
    rng = np.random.default_rng(seed + 1)
    for p in params["blocks"]:
        for k in p:
            p[k] = p[k] + 0.05 * rng.standard_normal(p[k].shape)
    return spec, params, synth.make_batch(spec, seed)


def test_main_network_and_table_gradients_match_central_differences():
    """L_main's gradient w.r.t. every scalar of the main network and of every table entry; with 6
    samples on 4-row tables most rows are hit by several samples (repeated ids)."""
    spec, params, batch = _ctr()
    B = len(spec["blocks"]) - 1
    ids = batch["ids"]
    assert any(len(set(ids[:, t])) < ids.shape[0] for t in range(ids.shape[1]))     # repeated ids present
    _, grads, gin = orc.forward_backward(spec, params, batch, want_input=True)
    h = 1e-5

    def fd_of(arr):
        fd = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = arr[i]
            arr[i] = old + h
            lp = orc.forward_only(spec, params, batch)[B]
            arr[i] = old - h
            lm = orc.forward_only(spec, params, batch)[B]
            arr[i] = old
            fd[i] = (lp - lm) / (2 * h)
        return fd

    for k in params["blocks"][B]:
        assert synth.rel_l2(grads[B][k], fd_of(params["blocks"][B][k])) <= 1e-6, k

    # Tables: sg[z_b] is a CONSTANT for the backward, so the reference is the central difference of
    # L_main with the block outputs held at their base values while z_0 follows the tables.
    blk, pm = spec["blocks"][B], params["blocks"][B]
    z0_base, target = orc.stage_input(spec, params["input"], batch)
    outs = []
    for b in range(B):
        outs.append(orc.block_forward(spec, spec["blocks"][b], params["blocks"][b], z0_base)[0])

    def lmain_frozen():
        z0, _ = orc.stage_input(spec, params["input"], batch)
        zm, _ = orc._mlp_fwd(blk, pm, orc.main_input(blk, z0, outs), act_last=True)
        return orc.head_loss(blk, pm, zm, target)[0]

    def fd_frozen(arr):
        fd = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = arr[i]
            arr[i] = old + h
            lp = lmain_frozen()
            arr[i] = old - h
            lm = lmain_frozen()
            arr[i] = old
            fd[i] = (lp - lm) / (2 * h)
        return fd

    untouched = 0
    for t in range(spec["n_sparse"]):
        name = f"table{t}"
        fd = fd_frozen(params["input"][name])
        total = fd_of(params["input"][name])                   # the derivative THROUGH the blocks as well: a different number
        assert synth.rel_l2(total, fd) > 1e-3
        assert synth.rel_l2(gin[name], fd) <= 1e-6, name
        mask = orc.touched_rows(spec, batch, name)
        assert np.all(gin[name][~mask] == 0.0)                  # rows no sample reads get exactly nothing
        untouched += int((~mask).sum())
    assert untouched > 0


def test_tables_receive_gradient_from_the_main_loss_alone():
    """The detached blocks read z_0 through sg (Eq. 1): their local losses DO depend on the tables
    (a finite difference shows it) but contribute nothing to the table gradient."""
    spec, params, batch = _ctr(seed=2)
    B = len(spec["blocks"]) - 1
    _, _, gin = orc.forward_backward(spec, params, batch, want_input=True)
    r, c = int(batch["ids"][0, 0]), 1
    h = 1e-5
    tab = params["input"]["table0"]
    old = tab[r, c]
    tab[r, c] = old + h
    lp = orc.forward_only(spec, params, batch)
    tab[r, c] = old - h
    lm = orc.forward_only(spec, params, batch)
    tab[r, c] = old
    fd = (np.array(lp) - np.array(lm)) / (2 * h)
    assert abs(fd[:B]).max() > 1e-4                            # local losses move with the table entry ...
    assert abs(gin["table0"][r, c] - fd.sum()) > 1e-5          # ... but they are not in the table's gradient


def test_main_network_does_not_reach_into_the_detached_blocks():
    spec, params, batch = _ctr(seed=3)
    B = len(spec["blocks"]) - 1
    _, g0 = orc.forward_backward(spec, params, batch)
    p2 = copy.deepcopy(params)
    for k in p2["blocks"][B]:
        p2["blocks"][B][k] = p2["blocks"][B][k] + 0.3
    _, g1 = orc.forward_backward(spec, p2, batch)
    for b in range(B):
        for k in g0[b]:
            assert np.array_equal(g0[b][k], g1[b][k])
    # the other way round the VALUE passes (sg is the identity forward): block parameters change L_main's gradients
    p3 = copy.deepcopy(params)
    p3["blocks"][0]["W0"] = p3["blocks"][0]["W0"] + 0.3
    _, g3 = orc.forward_backward(spec, p3, batch)
    assert not np.array_equal(g0[B]["W0"], g3[B]["W0"])


def test_repeated_id_adds_up_by_hand():
    """Two samples with the same id: the table row's gradient is the sum of their z_0-gradient
    slices.  Main network = one Linear(4 -> 1) with ReLU on a 1-table, 1-block-free model is not
    expressible here, so the check is on the scatter itself with a prescribed dz0."""
    spec = {"input": "ctr", "n_sparse": 2, "emb_dim": 2, "table_rows": 3}
    batch = {"ids": np.array([[1, 0], [1, 2], [0, 2]], dtype=np.int32)}
    dz0 = np.array([[1.0, 2.0, 10.0, 20.0, 9.0],
                    [3.0, 4.0, 30.0, 40.0, 9.0],
                    [5.0, 6.0, 50.0, 60.0, 9.0]])             # the last column (a dense feature) trains nothing
    g = orc.input_gradients(spec, batch, dz0)
    assert np.array_equal(g["table0"], np.array([[5.0, 6.0], [4.0, 6.0], [0.0, 0.0]]))      # row 1: samples 0 and 1
    assert np.array_equal(g["table1"], np.array([[10.0, 20.0], [0.0, 0.0], [80.0, 100.0]]))  # row 2: samples 1 and 2


@pytest.mark.parametrize("optk", ["sgd", "adam"])
def test_against_torch_autograd_with_index_lookups(optk):
    """x0 = cat(table_t[ids[:, t]], dense, pad); blocks on x0.detach(); main on cat(x0, z_b.detach());
    ONE backward on L_main + sum_b l_b (Eq. 2, all lambda 1).  torch's dense optimizers move
    untouched rows only when their gradient history is non-zero, so the first step (zero history)
    is comparable for every optimizer: untouched rows stay, touched rows follow the dense rule."""
    opt = {"kind": optk, "lr": 1e-2, "wd": 0.0, "beta1": 0.9, "beta2": 0.999, "eps": 1e-8}
    spec, params, batch = _ctr(batch=7, rows=5, seed=4, opt=opt)
    B = len(spec["blocks"]) - 1
    tin = {k: torch.tensor(v, requires_grad=True) for k, v in params["input"].items()}
    tpar = [{k: torch.tensor(v, requires_grad=True) for k, v in p.items()} for p in params["blocks"]]
    ids = torch.tensor(batch["ids"], dtype=torch.long)
    dense = torch.tensor(batch["dense"], dtype=torch.float64)
    y = torch.tensor(batch["y"], dtype=torch.float64)
    pad = spec["width"] - spec["n_sparse"] * spec["emb_dim"] - spec["n_dense"]
    x0 = torch.cat([tin[f"table{t}"][ids[:, t]] for t in range(spec["n_sparse"])] + [dense, torch.zeros(len(y), pad)], dim=1)
    losses, outs = [], []
    for blk, p in zip(spec["blocks"][:B], tpar[:B]):
        z = _torch_block(spec, blk, p, x0.detach())
        outs.append(z)
        losses.append(TF.binary_cross_entropy_with_logits(TF.linear(z, p["Wh"], p["bh"])[:, 0], y))
    u = torch.cat([x0] + [z.detach() for z in outs], dim=1)
    main = dict(spec["blocks"][B], kind="tower")
    zm = _torch_block(spec, main, tpar[B], u)
    losses.append(TF.binary_cross_entropy_with_logits(TF.linear(zm, tpar[B]["Wh"], tpar[B]["bh"])[:, 0], y))
    allp = list(tin.values()) + [v for p in tpar for v in p.values()]
    optim = torch.optim.SGD(allp, lr=opt["lr"]) if optk == "sgd" else torch.optim.Adam(allp, lr=opt["lr"], betas=(0.9, 0.999), eps=1e-8)
    optim.zero_grad()
    sum(losses).backward()
    ol, og, gin = orc.forward_backward(spec, params, batch, want_input=True)
    assert np.allclose(ol, [float(l.detach()) for l in losses], rtol=1e-12, atol=1e-13)
    for b in range(B + 1):
        for k in og[b]:
            assert synth.rel_l2(og[b][k], tpar[b][k].grad.numpy()) < 1e-10, (b, k)
    for k in gin:
        assert synth.rel_l2(gin[k], tin[k].grad.numpy()) < 1e-10, k
    optim.step()
    _, _, newp, _ = orc.step(spec, params, orc.new_opt_state(params), batch)
    for k in gin:
        want = tin[k].detach().numpy()
        assert np.linalg.norm(newp["input"][k] - want) <= 1e-9 * np.linalg.norm(want) + 1e-12, k
        mask = orc.touched_rows(spec, batch, k)
        assert np.array_equal(newp["input"][k][~mask], params["input"][k][~mask])


def test_sparse_adam_first_step_closed_form_and_untouched_rows_keep_their_state():
    """Adam's first step on a touched row is -lr g / (|g| + eps); a row nobody reads keeps value and
    moments; on a later step the bias correction uses the GLOBAL step count."""
    opt = {"kind": "adam", "lr": 1e-3, "wd": 0.0, "beta1": 0.9, "beta2": 0.999, "eps": 1e-8}
    theta = np.array([[1.0, -2.0], [3.0, 4.0], [5.0, 6.0]])
    g = np.array([[0.5, -0.75], [0.0, 0.0], [2.0, 1.0]])
    touched = np.array([True, False, True])
    z = np.zeros_like(theta)
    th, m, v = orc.optimizer_update_rows(opt, theta, g, touched, z, z, 1)
    assert np.allclose(th[0], theta[0] - 1e-3 * np.sign(g[0]), atol=1e-10)
    assert np.array_equal(th[1], theta[1]) and np.array_equal(m[1], z[1]) and np.array_equal(v[1], z[1])
    # step 5 touching only the middle row, whose history is empty: the update is lr * (0.1 g / (1 - 0.9^5)) / (sqrt(0.001 g^2 / (1 - 0.999^5)) + eps)
    g2 = np.array([[0.0, 0.0], [0.3, -0.3], [0.0, 0.0]])
    th2, m2, v2 = orc.optimizer_update_rows(opt, th, g2, np.array([False, True, False]), m, v, 5)
    mh = 0.1 * 0.3 / (1 - 0.9 ** 5)
    vh = 0.001 * 0.09 / (1 - 0.999 ** 5)
    assert np.allclose(th2[1], th[1] - 1e-3 * np.array([1, -1]) * mh / (np.sqrt(vh) + 1e-8), atol=1e-12)
    assert np.array_equal(th2[0], th[0]) and np.array_equal(m2[2], m[2])
