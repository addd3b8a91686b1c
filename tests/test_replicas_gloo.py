"""The N > 1 paths on CPU, two gloo ranks.  Independent replicas: barrier + MAX over ranks, whole-job
rate = units of all ranks / slowest rank's time.  Data-parallel replicas: the host-side part (shards,
the communicator id reaching every rank, one schedule for all) and the recipe itself, checked on the
oracle: each rank's share of the global means, summed over the ranks, is the single-process result."""
import os
import socket

import pytest
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2608_18469_b200.replicas import Replicas
    r = Replicas(backend="gloo", device="cpu")
    r.barrier()
    local_ms = 10.0 if rank == 0 else 25.0          # rank 1 is the straggler
    rate, ms = r.whole_job_rate(units_per_rank_step=4096, steps=5, local_ms=local_ms)
    mx = r.max_over_ranks(rank + 1.5)
    r.barrier()
    out.put((rank, rate, ms, mx))
    r.close()


def test_two_ranks_report_the_slowest_time_and_the_aggregate_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, rate, ms, mx in res:
        assert ms == 25.0 and mx == 2.5
        assert rate == pytest.approx(2 * 4096 * 5 / 25e-3)


def test_single_process_needs_no_process_group():
    os.environ.pop("WORLD_SIZE", None)
    os.environ.pop("RANK", None)
    from paper_2608_18469_b200.replicas import Replicas
    r = Replicas(backend="gloo")
    r.barrier()
    assert r.world == 1 and r.max_over_ranks(3.0) == 3.0
    assert r.whole_job_rate(100, 2, 4.0) == (100 * 2 / 4e-3, 4.0)
    r.close()


class _FakeModel:
    """Stands in for binding.Model: records what the communicator set-up was given."""

    def __init__(self):
        self.got = None

    def comm_init(self, rank, world, uid):
        self.got = (rank, world, uid)


def _dp_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import numpy as np
    import torch
    from oracle import erase_oracle as orc
    from paper_2608_18469_b200 import synth
    from paper_2608_18469_b200.replicas import Replicas
    from tests import util
    r = Replicas(backend="gloo", device="cpu")
    # every rank ends up with rank 0's id and rank 0's schedule, whatever it drew or measured itself
    fake = _FakeModel()
    uid = r.attach(fake, make_id=lambda: bytes([17 + rank]) * 128)
    choice = r.agree_on({"n_streams": 3 + rank, "flags": 8 * (rank + 1)})
    # the recipe: a replica normalises by the GLOBAL row count, so its losses and gradients are shares that add up
    spec = synth.mlp_spec(6, 10, 2, 8, "gelu", "f32")
    flat = synth.init_params(spec, 2)
    params = util.structure(spec, flat)
    batch = synth.make_batch(spec, 2)
    rows = r.shard(spec["batch"])
    mine = {k: v[rows] for k, v in batch.items()}
    local = dict(spec, batch=spec["batch"] // world)
    losses, grads = orc.forward_backward(local, params, mine)        # means over this rank's rows
    share = 1.0 / world                                               # equal shards: local mean -> share of the global mean
    flatg = np.concatenate([np.asarray(losses, np.float64)] +
                           [grads[b][k].ravel() for b in range(len(grads)) for k in sorted(grads[b])]) * share
    t = torch.from_numpy(flatg)
    r.dist.all_reduce(t)                                              # what the per-block exchanges compute, block by block
    want_l, want_g = orc.forward_backward(spec, params, batch)
    want = np.concatenate([np.asarray(want_l, np.float64)] +
                          [want_g[b][k].ravel() for b in range(len(want_g)) for k in sorted(want_g[b])])
    err = float(np.abs(t.numpy() - want).max() / np.abs(want).max())
    out.put((rank, fake.got, uid, choice, (rows.start, rows.stop), err))
    r.close()


def test_two_data_parallel_ranks_share_id_schedule_and_add_up_to_the_oracle():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_dp_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, uid, choice, rows, err in res:
        assert uid == bytes([17]) * 128 and got == (rank, 2, uid)      # rank 0's id, own rank, world
        assert choice == {"n_streams": 3, "flags": 8}                  # rank 0's schedule
        assert rows == (4 * rank, 4 * rank + 4)
        assert err < 1e-12


def test_shards_must_be_equal():
    from paper_2608_18469_b200.replicas import Replicas
    r = Replicas(backend="gloo")
    r.world, r.rank = 3, 1
    assert r.shard(12) == slice(4, 8)
    with pytest.raises(ValueError):
        r.shard(10)
