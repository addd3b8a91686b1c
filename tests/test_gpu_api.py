"""Behaviour of the C ABI on a GPU: state and argument errors, checkpoint/resume, caller-owned
arena, launch counting, the per-phase timeline and the per-operation profile."""
import ctypes as C

import numpy as np
import pytest

from paper_2608_18469_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _gu():
    from tests import gpu_util
    return gpu_util


def _small():
    return synth.lm_spec(2, 64, 1, 128, 32, 2, 96)      # bf16, 2 blocks, AdamW


def test_step_before_parameters_are_set_is_refused():
    gu = _gu()
    spec = _small()
    m = binding.Model(spec)
    db = gu.DevBatch(spec, synth.make_batch(spec, 0))
    with pytest.raises(binding.EraseError) as e:
        m.step(**db.args())
    assert e.value.status == binding.ESTATE and "never set" in str(e.value)
    flat = synth.init_params(spec, 0)
    m.set_all(flat)
    with pytest.raises(binding.EraseError) as e:
        m.step(n_streams=0, **db.args())
    assert e.value.status == binding.EINVAL
    with pytest.raises(binding.EraseError) as e:
        m.step(ids=None)
    assert e.value.status == binding.EINVAL
    with pytest.raises(binding.EraseError) as e:
        m.losses()
    assert e.value.status == binding.ESTATE              # no step has run yet
    with pytest.raises(binding.EraseError) as e:
        m.set_params(0, np.zeros(3, np.float32))         # wrong size
    assert e.value.status == binding.EINVAL
    with pytest.raises(binding.EraseError) as e:
        m.grads(0)                                       # frozen table: no gradient
    assert e.value.status == binding.EINVAL
    m.step(n_streams=99, **db.args())                    # clamped to n_blocks + 1
    assert np.isfinite(m.losses()).all()
    m.close()


def test_checkpoint_and_resume_is_bit_identical():
    gu = _gu()
    spec = _small()
    flat = synth.init_params(spec, 2)
    batches = [gu.DevBatch(spec, synth.make_batch(spec, 2, index=i)) for i in range(6)]
    straight = gu.run_steps(spec, flat, batches, n_streams=3)
    # three steps, save everything through the ABI, restore into a new model, three more
    m = gu.new_model(spec, flat)
    for db in batches[:3]:
        m.step(n_streams=3, **db.args())
    m.sync()
    n = m.num_tensors()
    saved = [m.params(i) for i in range(n)]
    tidx = [i for i in range(n) if m.tensor_info(i)[3]]
    opt = {i: m.opt_state(i) for i in tidx}
    m.close()
    m2 = binding.Model(spec)
    m2.set_all(saved)
    for i in tidx:
        m2.set_opt_state(i, *opt[i])
    for db in batches[3:]:
        m2.step(n_streams=3, **db.args())
    for i in tidx:
        assert m2.params(i).tobytes() == straight[f"p{i}"].tobytes()
        mm, vv, t = m2.opt_state(i)
        assert mm.tobytes() == straight[f"m{i}"].tobytes() and vv.tobytes() == straight[f"v{i}"].tobytes()
        assert t == 6
    m2.close()


def test_model_in_a_caller_owned_arena_matches_library_allocation():
    import torch
    gu = _gu()
    spec = _small()
    flat = synth.init_params(spec, 4)
    batches = [gu.DevBatch(spec, synth.make_batch(spec, 4, index=i)) for i in range(2)]
    ref = gu.run_steps(spec, flat, batches, n_streams=2)
    need = binding.arena_bytes(spec)
    assert need > 0
    arena = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    base = (arena.data_ptr() + 255) // 256 * 256
    torch.cuda.synchronize()
    m = binding.Model(spec, arena=base, arena_bytes=need)
    m.set_all(flat)
    for db in batches:
        m.step(n_streams=2, **db.args())
    m.sync()
    for i in range(m.num_tensors()):
        if m.tensor_info(i)[3]:
            assert m.params(i).tobytes() == ref[f"p{i}"].tobytes()
    m.close()
    with pytest.raises(binding.EraseError) as e:
        binding.Model(spec, arena=base, arena_bytes=need // 8)     # too small
    assert e.value.status == binding.ENOMEM


def test_timeline_profile_and_launch_count():
    gu = _gu()
    spec = _small()
    nb = len(spec["blocks"])
    m = gu.new_model(spec, synth.init_params(spec, 5))
    db = gu.DevBatch(spec, synth.make_batch(spec, 5))
    l0 = m.launch_count()
    m.step(n_streams=nb + 1, **db.args())
    per_step = m.launch_count() - l0
    assert per_step > 10
    tl = m.timeline()
    assert tl.shape == (2 * nb + 1, 2) and (tl[:, 1] >= tl[:, 0]).all()
    for b in range(nb):                       # B_b is released by F_b's event, the optimizer waits for every B_b
        assert tl[nb + b, 0] >= tl[b, 1] - 1e-3
        assert tl[2 * nb, 0] >= tl[nb + b, 1] - 1e-3
    m.step(n_streams=nb + 1, flags=binding.GRAPH, **db.args())
    assert m.launch_count() - l0 == 2 * per_step          # a replayed graph launches the same kernels
    with pytest.raises(binding.EraseError) as e:
        m.timeline()                                      # graph replay records no timeline
    assert e.value.status == binding.ESTATE
    # device clock stamps are part of the captured graph: the timeline of a REPLAYED step
    stamps = 2 * (2 * nb + 1) + 1
    for rep in range(2):
        l1 = m.launch_count()
        m.step(n_streams=nb + 1, flags=binding.GRAPH | binding.STAMPS | binding.EARLY_HEAD | binding.BLOCK_OPT, **db.args())
        assert m.launch_count() - l1 == per_step + stamps + (nb - 1)   # one optimizer launch per block instead of one
        tg = m.timeline()
        assert tg.shape == (2 * nb + 1, 2) and (tg[:, 1] >= tg[:, 0]).all() and tg.min() >= 0 and tg.max() < 1e3
        for b in range(nb):
            assert tg[nb + b, 0] >= tg[b, 1] - 1e-3           # B_b starts after F_b's body
            if b + 1 < nb:
                assert tg[b + 1, 0] >= tg[b, 1] - 1e-3        # F_{b+1} follows F_b on the main stream
    recs = m.profile_step(**db.args())
    assert sum(r["launches"] for r in recs) == per_step
    assert {r["name"] for r in recs} >= {"gemm_fwd", "gemm_dgrad", "gemm_wgrad", "ce_finalize", "opt_update"}
    assert all(r["ms"] >= 0 for r in recs) and sum(r["flops"] for r in recs) > 0
    m.close()


def test_full_size_lm_configs_schedules_agree_and_losses_start_near_ln_vocab():
    """C2 in the launch configuration bench.py times, and C4 at full size (where the oracle is
    too slow to run in a test): every schedule gives the same bits, and with labels independent of
    the inputs the local losses sit between ln V and 2 ln V at initialisation."""
    import math
    gu = _gu()
    for name, steps in (("C2", 2), ("C4", 1)):
        spec = synth.config(name)
        nb = len(spec["blocks"])
        flat = synth.init_params(spec, 0)
        batches = [gu.DevBatch(spec, synth.make_batch(spec, 0, index=i)) for i in range(steps)]
        serial = gu.run_steps(spec, flat, batches, n_streams=1)
        bench_cfg = gu.run_steps(spec, flat, batches, n_streams=nb + 1,
                                 flags=binding.GRAPH | binding.EARLY_HEAD | binding.BLOCK_OPT | binding.SPLIT_BWD)
        for k in serial:
            if k != "launches":
                assert serial[k].tobytes() == bench_cfg[k].tobytes(), (name, k)
        lnv = math.log(spec["vocab"])
        # a random head cannot beat the uniform predictor on independent labels, and its logit
        # spread only adds about half its variance to the loss
        assert np.all(serial["losses"] > 0.99 * lnv) and np.all(serial["losses"] < 2.0 * lnv), serial["losses"]


def test_an_expired_device_wait_returns_etimeout_and_the_model_stays_usable():
    """One thread waits, with the bounded-wait helper of the tensor-core kernels and a limit of
    about a millisecond, on a barrier that nothing signals; the wait runs out by construction.  The
    next synchronising call reports ERASE_ETIMEOUT, a step enqueued behind the expiry skips its
    tensor-core work, and after the report the same model steps to the same bits as a fresh one."""
    import time
    gu = _gu()
    spec = _small()
    flat = synth.init_params(spec, 6)
    db = gu.DevBatch(spec, synth.make_batch(spec, 6))
    ref = gu.run_steps(spec, flat, [db], n_streams=3)
    m = gu.new_model(spec, flat)
    t0 = time.perf_counter()
    m.selftest_timeout(limit_us=1000)
    with pytest.raises(binding.EraseError) as e:
        m.sync()
    assert e.value.status == binding.ETIMEOUT and "code 8" in str(e.value)
    assert time.perf_counter() - t0 < 5.0                      # it returned; nothing hung
    m.sync()                                                   # the report cleared the status word
    # an expiry in front of a whole step: every tensor-core kernel of the step finds the word set
    m.selftest_timeout(limit_us=1000)
    t0 = time.perf_counter()
    m.step(n_streams=3, **db.args())
    with pytest.raises(binding.EraseError) as e:
        m.losses()
    assert e.value.status == binding.ETIMEOUT
    assert time.perf_counter() - t0 < 5.0
    m.close()
    # and the context is intact: a fresh model reproduces the reference bits
    again = gu.run_steps(spec, flat, [db], n_streams=3)
    for k in ref:
        if k != "launches":
            assert ref[k].tobytes() == again[k].tobytes(), k
    with pytest.raises(binding.EraseError) as e:
        gu.new_model(spec, flat).selftest_timeout(limit_us=0)
    assert e.value.status == binding.EINVAL


@pytest.mark.parametrize("kind", ["tokens_input", "tokens_last_target", "ctr"])
def test_an_id_outside_its_table_is_reported_and_never_dereferenced(kind):
    """The input staging checks every id against its table: a bad id is not used as an index (row 0
    stands in), the step's results are void and the next synchronising call returns ERASE_EINVAL.
    The model then runs a clean batch to the same losses as a model that never saw the bad one."""
    import torch
    gu = _gu()
    if kind == "ctr":
        spec = synth.ctr_spec(batch=64, table_rows=50, tower=(64, 32, 16))
    else:
        spec = _small()
    flat = synth.init_params(spec, 7)
    good = synth.make_batch(spec, 7)
    bad = {k: v.copy() for k, v in good.items()}
    if kind == "ctr":
        bad["ids"][5, 3] = spec["table_rows"] + 1000000
        bad["ids"][9, 0] = -7
    elif kind == "tokens_input":
        bad["ids"][1, 4] = spec["vocab"]                        # first id past the table
    else:
        bad["ids"][0, spec["seq"]] = -1                         # the last column is a target only
    gdb, bdb = gu.DevBatch(spec, good), gu.DevBatch(spec, bad)
    ref = gu.new_model(spec, flat)
    ref.step(n_streams=2, flags=binding.NO_OPT, **gdb.args())
    want = ref.losses()
    ref.close()
    m = gu.new_model(spec, flat)
    m.step(n_streams=2, flags=binding.NO_OPT, **bdb.args())
    with pytest.raises(binding.EraseError) as e:
        m.losses()
    assert e.value.status == binding.EINVAL and "outside its table" in str(e.value)
    torch.cuda.synchronize()                                    # no fault was raised on the device
    m.step(n_streams=2, flags=binding.NO_OPT, **gdb.args())
    assert m.losses().tobytes() == want.tobytes()
    m.close()
