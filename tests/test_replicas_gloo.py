"""The N > 1 path of the benchmark on CPU: two gloo ranks, barrier + MAX over ranks, whole-job
rate = units of all ranks / slowest rank's time."""
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
