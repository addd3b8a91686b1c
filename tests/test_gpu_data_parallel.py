"""Data-parallel replicas through the C ABI on one GPU.

What one GPU can show: (1) a model built for R replicas produces, on its shard, exactly its share
of the global sums -- the shares of the R shards add up to the oracle's losses and gradients on the
union batch; (2) with a communicator attached (a world of one: NCCL really runs, the sum over one
replica changes nothing) every schedule enqueues one exchange per block behind that block's
backward, in an order fixed by the schedule, and stays bit-identical to the model without one."""
import numpy as np
import pytest

from oracle import erase_oracle as orc
from paper_2608_18469_b200 import binding, synth
from tests import util

pytestmark = pytest.mark.gpu


def _gu():
    from tests import gpu_util
    return gpu_util


def _shard(spec, batch, r, world):
    per = spec["batch"] // world
    return {k: v[r * per:(r + 1) * per] for k, v in batch.items()}


@pytest.mark.parametrize("name", ["mlp_f32", "ctr_f32", "lm_f32", "lm_bf16"])
def test_shares_of_two_shards_add_up_to_the_oracle_on_the_union_batch(name):
    gu = _gu()
    full = {"mlp_f32": synth.mlp_spec(64, 128, 3, 96, "gelu", "f32"),
            "ctr_f32": synth.ctr_spec(batch=64, table_rows=50, tower=(64, 32, 16), dtype="f32"),
            "lm_f32": synth.lm_spec(2, 64, 2, 128, 24, 4, 96, dtype="f32"),
            "lm_bf16": synth.lm_spec(2, 128, 2, 256, 64, 8, 512)}[name]      # the softmax head fused into its GEMM
    tol = gu.TOL[full["dtype"]]
    world = 2
    local = dict(full, batch=full["batch"] // world, replicas=world)
    flat = synth.init_params(full, 3)
    batch = synth.make_batch(full, 3)
    want_l, want_g = orc.forward_backward(full, util.operand_params(full, util.structure(full, flat)), util.operand_batch(full, batch))
    tl = synth.tensor_list(full)
    tidx = util.trainable_index(full)
    m = gu.new_model(local, flat)
    try:
        db = gu.DevBatch(local, _shard(full, batch, 0, world))
        with pytest.raises(binding.EraseError) as e:         # built for two replicas, no communicator, no flag
            m.step(n_streams=2, **db.args())
        assert e.value.status == binding.ESTATE
        loss = np.zeros(len(full["blocks"]))
        grads = {i: 0.0 for i in tidx}
        for r in range(world):
            db = gu.DevBatch(local, _shard(full, batch, r, world))
            m.step(n_streams=len(full["blocks"]) + 1, flags=binding.LOCAL_GRADS | binding.NO_OPT, **db.args())
            loss += m.losses().astype(np.float64)
            for i in tidx:
                grads[i] = grads[i] + m.grads(i).astype(np.float64)
            assert m.comm_order() == []                       # nothing was exchanged
        np.testing.assert_allclose(loss, want_l, rtol=tol)
        for i in tidx:
            b, tname, _s, _t = tl[i]
            assert synth.rel_l2(grads[i], want_g[b][tname]) <= tol, (b, tname)
    finally:
        m.close()


@pytest.mark.parametrize("name", ["ctr", "c5"])
def test_a_communicator_of_one_runs_the_exchange_and_changes_no_bit(name):
    gu = _gu()
    spec = {"ctr": synth.ctr_spec(batch=256, table_rows=500, tower=(128, 64, 32)),
            "c5": synth.config("C5", w=128, batch=512)}[name]
    nb = len(spec["blocks"])
    flat = synth.init_params(spec, 5)
    batches = [gu.DevBatch(spec, synth.make_batch(spec, 5, index=i)) for i in range(3)]
    plain = gu.run_steps(spec, flat, batches, n_streams=1)
    uid = binding.comm_unique_id()
    assert len(uid) == binding.COMM_ID_BYTES and any(uid)

    def attach(m):
        m.comm_init(0, 1, binding.comm_unique_id())

    backward_order = list(range(nb - 1, -1, -1)) + [-1]
    forward_order = list(range(nb)) + [-1]
    cases = [(1, 0, backward_order), (2, 0, forward_order), (nb + 1, 0, forward_order),
             (nb + 1, binding.EARLY_HEAD | binding.BLOCK_OPT | binding.SPLIT_BWD, forward_order),
             (nb + 1, binding.PAR_FWD | binding.BLOCK_OPT, forward_order)]
    if name == "c5":
        cases.append((1, binding.PERSISTENT, forward_order))
    for ns, fl, order in cases:
        orders = []
        got = gu.run_steps(spec, flat, batches, n_streams=ns, flags=fl, attach=attach, orders=orders)
        for k in plain:
            if k != "launches":
                assert got[k].tobytes() == plain[k].tobytes(), (ns, fl, k)
        assert orders == [order] * len(batches), (ns, fl, orders)


def test_communicator_rules():
    gu = _gu()
    spec = synth.mlp_spec(64, 128, 2, 32, "relu", "f32")
    flat = synth.init_params(spec, 1)
    db = gu.DevBatch(spec, synth.make_batch(spec, 1))
    m = gu.new_model(spec, flat)
    try:
        uid = binding.comm_unique_id()
        with pytest.raises(binding.EraseError) as e:     # the spec says one replica
            m.comm_init(0, 2, uid)
        assert e.value.status == binding.EINVAL
        with pytest.raises(binding.EraseError) as e:
            m.comm_init(1, 1, uid)
        assert e.value.status == binding.EINVAL
        m.comm_init(0, 1, uid)
        with pytest.raises(binding.EraseError) as e:     # only one communicator per model
            m.comm_init(0, 1, binding.comm_unique_id())
        assert e.value.status == binding.ESTATE
        with pytest.raises(binding.EraseError) as e:     # no graph replay around the exchange
            m.step(n_streams=2, flags=binding.GRAPH, **db.args())
        assert e.value.status == binding.EUNSUPPORTED
        m.step(n_streams=2, flags=binding.GRAPH | binding.LOCAL_GRADS, **db.args())
        assert m.comm_order() == []
        m.step(n_streams=2, **db.args())
        assert m.comm_order() == [0, 1, -1]
        assert np.isfinite(m.losses()).all()
    finally:
        m.close()
    # sparse table gradients are not exchanged: a trained-table model takes a communicator of one only
    tspec = dict(synth.with_main(synth.ctr_spec(batch=64, table_rows=50, tower=(64, 32, 16)), tower=(64, 32)), replicas=2)
    tm = gu.new_model(tspec, synth.init_params(tspec, 2))
    try:
        with pytest.raises(binding.EraseError) as e:
            tm.comm_init(0, 2, binding.comm_unique_id())
        assert e.value.status == binding.EUNSUPPORTED
    finally:
        tm.close()
