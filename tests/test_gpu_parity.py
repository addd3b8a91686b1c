"""Parity of the CUDA library (through the C ABI) with the CPU oracle, and bit-identity of the
ERASE schedule with the serial one.  All inputs are seeded and synthetic."""
import numpy as np
import pytest

from paper_2608_18469_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu


def _gu():
    from tests import gpu_util
    return gpu_util


@pytest.mark.parametrize("name", list(util.tiny_specs()))
def test_tiny_fp32_every_block_kind(name):
    _gu().compare_teacher_forced(util.tiny_specs()[name], steps=3, seed=1, case=name)


def _midsize():
    s = {}
    # several 64-wide tiles with ragged tails in every dimension
    s["mlp_f32_ragged"] = synth.mlp_spec(70, 150, 3, 200, "gelu", "f32",
                                         opt={"kind": "adam", "lr": 1e-3, "wd": 0.0, "beta1": 0.9,
                                              "beta2": 0.999, "eps": 1e-8})
    s["tower_f32"] = {**synth.mlp_spec(48, 96, 2, 130, "relu", "f32")}
    for blk in s["tower_f32"]["blocks"]:
        blk["kind"] = "tower"
    s["lm_f32"] = synth.lm_spec(2, 96, 3, 160, 70, 3, 301, dtype="f32")       # dh 32, T ragged
    s["lm_f32_dh64"] = synth.lm_spec(2, 128, 2, 256, 48, 2, 200, dtype="f32")
    s["ctr_f32"] = synth.ctr_spec(batch=150, n_dense=13, n_sparse=5, table_rows=50, emb_dim=8,
                                  tower=(72, 40, 24), n_cross=3, dtype="f32")
    return s


@pytest.mark.parametrize("name", list(_midsize()))
def test_midsize_fp32(name):
    _gu().compare_teacher_forced(_midsize()[name], steps=2, seed=2, case=name)


def test_config1_fp32_ten_steps_and_free_running_losses():
    from oracle import erase_oracle as orc
    gu = _gu()
    spec = synth.config("C1")
    gu.compare_teacher_forced(spec, steps=10, seed=0, case="C1")
    # free running: ten steps from seed 0, losses against the oracle's own trajectory
    flat = synth.init_params(spec, 0)
    batches = [synth.make_batch(spec, 0, index=i) for i in range(10)]
    got = gu.run_steps(spec, flat, [gu.DevBatch(spec, b) for b in batches], n_streams=3)
    params = util.structure(spec, flat)
    state = orc.new_opt_state(params)
    for i, b in enumerate(batches):
        want, _, params, state = orc.step(spec, params, state, b)
        assert np.allclose(got["losses"][i], want, rtol=1e-4, atol=0)


def _bf16_cases():
    s = {}
    s["c5_w128_b512"] = synth.config("C5", w=128, batch=512)
    s["c5_w512_b512"] = synth.config("C5", w=512, batch=512)
    s["mlp_bf16_ragged"] = synth.mlp_spec(200, 328, 2, 300, "gelu", "bf16")
    s["lm_bf16_small"] = synth.lm_spec(2, 128, 2, 512, 128, 4, 1000)
    s["lm_bf16_ragged_vocab"] = synth.lm_spec(2, 128, 2, 256, 75, 3, 1016)   # 225 rows, 1016 = 3*256 + 248 logits: ragged in every tile size
    s["lm_bf16_ragged_T"] = synth.lm_spec(2, 192, 3, 384, 100, 3, 777)     # T not a multiple of the 64-tile
    s["lm_bf16_T320"] = synth.lm_spec(1, 64, 1, 128, 320, 2, 300)            # five key tiles per head
    s["lm_bf16_dh32"] = synth.lm_spec(1, 128, 4, 256, 96, 2, 300)            # head width 32: SIMT attention
    s["ctr_bf16_small"] = synth.ctr_spec(batch=512, table_rows=1000, tower=(256, 128, 64))
    # enough rows (>= 512) for the grouped weight-gradient kernel, with ragged M / N / K tails in every problem
    s["lm_bf16_grouped_ragged"] = synth.lm_spec(2, 192, 3, 328, 100, 6, 777)
    s["mlp_bf16_grouped_ragged"] = synth.mlp_spec(200, 328, 2, 600, "relu", "bf16")
    # the goodness objective (BCE on sum_j z_j^2) as the local loss, with and without a closing activation
    s["mlp_bf16_goodness"] = synth.mlp_spec(128, 256, 3, 512, "gelu", "bf16", head="goodness")
    s["tower_bf16_goodness"] = synth.mlp_spec(128, 256, 2, 512, "relu", "bf16", head="goodness")
    for blk in s["tower_bf16_goodness"]["blocks"]:
        blk["kind"] = "tower"
    return s


# Seeds of the small bf16 cases.  On chains of MLP blocks without norms or residuals the samples'
# features drift towards a common vector, every gradient of a later block becomes that vector times
# sum_n (sigmoid(s_n) - y_n), and on some draws of the balanced labels that sum nearly cancels: the
# instance is then ill-conditioned for ANY bf16 implementation (the oracle's own bf16-storage
# sensitivity exceeds the tolerance).  These seeds give well-conditioned instances, so every tensor
# is held to the plain 2e-2 with no exception.
_SEED = {"c5_w128_b512": 4, "mlp_bf16_ragged": 4, "mlp_bf16_grouped_ragged": 8,
         "mlp_bf16_odd_width": 11, "ctr_bf16_batch3": 11}


@pytest.mark.parametrize("name", list(_bf16_cases()))
def test_bf16_small(name):
    _gu().compare_teacher_forced(_bf16_cases()[name], steps=2, seed=_SEED.get(name, 3), case=name)


@pytest.mark.parametrize("name", ["lm_bf16_small", "lm_bf16_ragged_T", "lm_bf16_grouped_ragged"])
def test_bf16_small_with_the_fused_loss_and_bias_gradient_kernel(name, monkeypatch):
    """The persistent softmax-CE kernel that also produces the head's bias gradient is chosen by
    size (gradient matrices far beyond L2); here it is forced onto small cases, including
    vocabularies whose vector count is not a multiple of the CTA width and fewer rows than CTAs."""
    monkeypatch.setenv("ERASE_CE_MODE", "0")
    monkeypatch.setenv("ERASE_CE_FUSED", "2")
    _gu().compare_teacher_forced(_bf16_cases()[name], steps=2, seed=3, case=name)


@pytest.mark.parametrize("ce_mode", ["1", "0"])
def test_large_vocabulary_head(ce_mode, monkeypatch):
    """4224 rows x 32000 logits (270 MB in bf16, 4000 16-byte vectors per row).  Mode 1: the head
    whose GEMM epilogue leaves exp(logit - reference) and partial sums, so that loss and gradient
    never read the logits back.  Mode 0: the separate softmax pass, where this size selects the
    persistent kernel that also produces the bias gradient."""
    monkeypatch.setenv("ERASE_CE_MODE", ce_mode)
    spec = synth.lm_spec(1, 64, 1, 128, 528, 8, 32000)
    _gu().compare_teacher_forced(spec, steps=1, seed=4, case="lm_vocab32000")


@pytest.mark.parametrize("in_wgrad", ["1", "0"])
def test_softmax_head_bias_gradient_inside_the_weight_gradient_gemm(in_wgrad, monkeypatch):
    """d = 256, V = 16384: wide enough for the CTA-pair kernel (64 pair tiles), so the head's weight-gradient
    GEMM takes the 16 extra columns behind r (.) z and its narrow tiles leave db_h = sum_n r_n P[n,:]; with the
    switch off the same gradient comes from the separate weighted column sum over P.  Both against the oracle,
    and the fix-up path (rows recomputed with the true maximum rewrite r_n and the extra column) with the first."""
    monkeypatch.setenv("ERASE_HEAD_XCOL", in_wgrad)
    gu = _gu()
    spec = synth.lm_spec(1, 256, 4, 512, 64, 8, 16384)
    m = gu.new_model(spec, synth.init_params(spec, 4))
    try:
        db = gu.DevBatch(spec, synth.make_batch(spec, 4))
        names = [r["name"] for r in m.profile_step(**db.args())]
        # the block's own bias gradients are batched reductions: the only plain column sum is the head's
        assert ("colsum" in names) == (in_wgrad == "0"), names
    finally:
        m.close()
    gu.compare_teacher_forced(spec, steps=2, seed=4, case="lm_head_bias_in_wgrad")
    if in_wgrad == "1":
        def lift(values):
            values[(0, "bh")][7] += 150.0
        gu.compare_teacher_forced(spec, steps=1, seed=4, case="lm_head_bias_in_wgrad_fixup", init_hook=lift)


@pytest.mark.parametrize("name", ["lm_bf16_small", "lm_bf16_ragged_vocab", "C2"])
def test_softmax_head_with_the_separate_softmax_pass(name, monkeypatch):
    """The path that heads which do not qualify for the exp epilogue take (fp32 models,
    vocabularies or widths that are not multiples of 8), forced onto cases that do qualify."""
    monkeypatch.setenv("ERASE_CE_MODE", "0")
    spec = synth.config("C2") if name == "C2" else _bf16_cases()[name]
    _gu().compare_teacher_forced(spec, steps=2, seed=0 if name == "C2" else 3, case=name)


def test_softmax_head_rows_whose_target_logit_is_far_below_the_maximum_are_recomputed():
    """The exp epilogue measures every logit against the target's own logit.  A head bias that
    lifts one vocabulary entry by 150 puts the row maximum 150 above that reference for nearly every
    row: their sums overflow, the finalize kernel lists them, and the fix-up kernel recomputes those
    rows exactly.  A second entry lifted by 60 stays inside the safe range.  Losses (about 150 nats)
    and every gradient must still match the oracle."""
    def lift(values):
        values[(0, "bh")][7] += 150.0
        values[(1, "bh")][11] += 60.0
    spec = synth.lm_spec(2, 128, 2, 256, 96, 3, 1000)
    _gu().compare_teacher_forced(spec, steps=2, seed=3, case="lm_lifted_bias", init_hook=lift)


def test_config2_small_lm_bf16_full_size():
    _gu().compare_teacher_forced(synth.config("C2"), steps=3, seed=0, case="C2")


def test_config2_in_the_benchmark_launch_configuration():
    from paper_2608_18469_b200 import binding
    spec = synth.config("C2")
    _gu().compare_teacher_forced(spec, steps=2, seed=1, n_streams=len(spec["blocks"]) + 1,
                                 flags=binding.GRAPH | binding.EARLY_HEAD | binding.BLOCK_OPT | binding.SPLIT_BWD,
                                 case="C2_bench")


def test_config5_mid_point_w1024_b4096():
    _gu().compare_teacher_forced(synth.config("C5", w=1024, batch=4096), steps=1, seed=0, case="C5_w1024_b4096")


def test_config3_ctr_bf16_full_size():
    # seed 6: of seeds 0..6, four give a well-conditioned instance (2, 3, 4, 6: worst tensor 0.5-1.7e-2, the dot
    # block's W0) and three an ill-conditioned one (0, 1, 5: 2.3-3.4e-2 on the dot block at step 1: after Adam's
    # first sign step its gradients on 3 % positives shrink 30-fold and the oracle's own sensitivity to bf16
    # storage of activations is 2.3e-2 and more)
    _gu().compare_teacher_forced(synth.config("C3"), steps=2, seed=6, case="C3")


def test_config4_reduced_two_blocks():
    spec = synth.lm_spec(2, 768, 12, 3072, 128, 8, 32768)
    _gu().compare_teacher_forced(spec, steps=1, seed=0, case="C4_reduced")


def test_config4_one_block_at_full_size():
    """One block of the larger LM proxy at its full shapes: 8192 tokens (batch 8 x T 1024: sixteen
    key tiles per head, causal imbalance), d 768, 12 heads, MLP 3072, vocabulary 32768 -- the
    sizes at which the CTA-pair GEMM with fused residual epilogues, the pair-split dgrad and
    weight gradients and the loss path chosen by size run.  The other eleven blocks repeat these
    shapes on other values."""
    spec = synth.lm_spec(1, 768, 12, 3072, 1024, 8, 32768)
    _gu().compare_teacher_forced(spec, steps=1, seed=0, case="C4_one_block")


@pytest.mark.parametrize("w", [2048, 4096])
def test_config5_upper_sweep_two_blocks(w):
    """The wide end of the saturation sweep (w 2048 and 4096, batch 512, two of the eight blocks):
    GEMMs of 512 x 4w x w with 256 x 256 pair tiles and weight gradients of 4w x w."""
    spec = synth.mlp_spec(w, 4 * w, 2, 512, "gelu", "bf16")
    _gu().compare_teacher_forced(spec, steps=1, seed=0, case=f"C5_w{w}_b512_two_blocks")


@pytest.mark.parametrize("name", ["ctr_main_f32", "ctr_main_bf16", "ctr_main_frozen_tables", "mlp_main_bf16"])
def test_main_network_and_embedding_backward(name):
    """The undetached remainder of Eq. 2: a main network over [z_0 | sg z_1 | .. | sg z_B] with L_main,
    its usual backward, and (CTR) the gradient into the embedding tables: scatter-add by id with many
    repeated ids (Zipf draws on small tables), optimizer on the touched rows only.  Losses, every
    gradient (tables included, dense) and the updated tables are compared with the oracle."""
    adam = {"kind": "adam", "lr": 1e-3, "wd": 0.0, "beta1": 0.9, "beta2": 0.999, "eps": 1e-8}
    if name == "ctr_main_f32":
        spec = synth.with_main(synth.ctr_spec(batch=150, n_dense=13, n_sparse=5, table_rows=50, emb_dim=8, tower=(72, 40, 24),
                                              n_cross=3, dtype="f32", opt=adam), tower=(64, 32))
    elif name == "ctr_main_bf16":        # 2048 samples: a table row's gradient sums few samples, its bf16 noise falls with 1/sqrt(batch)
        spec = synth.with_main(synth.ctr_spec(batch=2048, table_rows=1000, tower=(256, 128, 64)), tower=(256, 128))
    elif name == "ctr_main_frozen_tables":
        spec = synth.with_main(synth.ctr_spec(batch=256, table_rows=300, tower=(128, 64, 32)), tower=(128, 64), train_input=False)
    else:
        # Dense input, nothing but the main network and the blocks to train.  With BALANCED labels this
        # chain is ill-conditioned on almost every draw (the features of all samples are nearly the same
        # vector, so every gradient is that vector times sum_n (sigmoid(s_n) - y_n), which cancels: the
        # oracle's own bf16-storage sensitivity is 3e-2 .. 7e-2 on 9 of 11 seeds); 20 % positives keep the
        # sum away from zero and the instance well conditioned.
        spec = synth.with_main(synth.mlp_spec(128, 512, 3, 2048, "gelu", "bf16"), tower=(256, 64))
    _gu().compare_teacher_forced(spec, steps=3, seed=5, case=name, label_p=0.2 if name == "mlp_main_bf16" else None)


def test_main_network_schedules_are_bit_identical():
    from paper_2608_18469_b200 import binding
    gu = _gu()
    spec = synth.with_main(synth.ctr_spec(batch=256, table_rows=200, tower=(128, 64, 32)), tower=(128, 64))
    flat = synth.init_params(spec, 7)
    batches = [gu.DevBatch(spec, synth.make_batch(spec, 7, index=i)) for i in range(3)]
    nb = len(spec["blocks"])
    serial = gu.run_steps(spec, flat, batches, n_streams=1)
    for ns, fl in ((nb + 1, 0), (3, binding.GRAPH), (nb + 1, binding.GRAPH | binding.EARLY_HEAD | binding.BLOCK_OPT | binding.SPLIT_BWD),
                   (nb + 1, binding.PAR_FWD | binding.EARLY_HEAD)):
        _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=ns, flags=fl))


def _edge_cases():
    s = {}
    s["mlp_bf16_batch1"] = synth.mlp_spec(64, 128, 2, 1, "gelu", "bf16")                 # a single row
    s["mlp_bf16_odd_width"] = synth.mlp_spec(50, 77, 2, 33, "relu", "bf16")             # strides not multiples of 8: SIMT GEMMs
    s["lm_bf16_seq1"] = synth.lm_spec(1, 64, 1, 128, 1, 3, 40)                           # one position per sequence
    s["lm_bf16_vocab_odd"] = synth.lm_spec(1, 64, 1, 128, 20, 2, 203)                    # vocabulary not a multiple of 8
    s["lm_bf16_T65"] = synth.lm_spec(1, 64, 1, 128, 65, 2, 96)                           # one row past a 64-tile
    s["ctr_bf16_batch3"] = synth.ctr_spec(batch=3, table_rows=9, tower=(64, 32, 16))     # fewer rows than any tile
    s["mlp_f32_batch1"] = synth.mlp_spec(8, 8, 1, 1, "relu", "f32")
    return s


@pytest.mark.parametrize("name", list(_edge_cases()))
def test_edge_shapes(name):
    _gu().compare_teacher_forced(_edge_cases()[name], steps=2, seed=_SEED.get(name, 4), case=name)


# ------------------------------------------------------------------ schedules: bit identity

def _bits_equal(a, b):
    for k in a:
        if k == "launches":
            continue
        assert a[k].tobytes() == b[k].tobytes(), k


@pytest.mark.parametrize("name", ["C1", "lm", "ctr", "c5", "goodness"])
def test_erase_schedule_is_bit_identical_to_serial(name):
    gu = _gu()
    spec = {"C1": synth.config("C1"),
            "lm": synth.lm_spec(3, 128, 2, 256, 64, 4, 512),
            "ctr": synth.ctr_spec(batch=256, table_rows=500, tower=(128, 64, 32)),
            "c5": synth.config("C5", w=128, batch=512),
            "goodness": synth.mlp_spec(128, 256, 3, 512, "gelu", "bf16", head="goodness")}[name]
    flat = synth.init_params(spec, 5)
    batches = [gu.DevBatch(spec, synth.make_batch(spec, 5, index=i)) for i in range(4)]
    serial = gu.run_steps(spec, flat, batches, n_streams=1)
    nb = len(spec["blocks"])
    for ns in sorted({2, 3, nb + 1}):
        _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=ns))
    from paper_2608_18469_b200 import binding
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=1, flags=binding.GRAPH))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=nb + 1, flags=binding.GRAPH))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=nb + 1, flags=binding.EARLY_HEAD))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=2, flags=binding.GRAPH | binding.EARLY_HEAD))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=nb + 1, flags=binding.BLOCK_OPT))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=nb + 1,
                                     flags=binding.GRAPH | binding.EARLY_HEAD | binding.BLOCK_OPT))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=nb + 1, flags=binding.SPLIT_BWD))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=2,
                                     flags=binding.GRAPH | binding.EARLY_HEAD | binding.BLOCK_OPT | binding.SPLIT_BWD))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=nb + 1,
                                     flags=binding.GRAPH | binding.EARLY_HEAD | binding.BLOCK_OPT | binding.SPLIT_BWD))
    # parallel topology: every block's forward on its side stream too (ignored on chains)
    P = binding.PAR_FWD
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=nb + 1, flags=P))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=3, flags=P | binding.EARLY_HEAD | binding.SPLIT_BWD))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=nb + 1,
                                     flags=binding.GRAPH | binding.EARLY_HEAD | binding.BLOCK_OPT | P))
    assert serial["launches"] > 0
    # F_{b+1} and B_b inside one persistent kernel on a partition of the SMs: bf16 chains of MLP blocks
    if name in ("c5", "goodness"):
        _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=1, flags=binding.PERSISTENT))
        _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=nb + 1, flags=binding.PERSISTENT | binding.GRAPH))
    else:
        with pytest.raises(binding.EraseError) as e:
            gu.run_steps(spec, flat, batches[:1], n_streams=1, flags=binding.PERSISTENT)
        assert e.value.status == binding.EUNSUPPORTED


@pytest.mark.parametrize("name", ["relu_ragged", "gelu_w1024", "tower_relu", "wide_split"])
def test_persistent_co_scheduled_kernel_is_bit_identical_to_serial(name):
    """ERASE_PERSISTENT on shapes that reach every part of the dual-list kernel: ragged M / N / K tails,
    fused ReLU and ReLU-derivative epilogues, GELU passes as elementwise problems, grouped and
    stand-alone weight gradients with split-K partials, several tiles per CTA.  The losses, gradients,
    parameters and optimizer state must be the bits of the serial schedule, which launches the same
    GEMMs one by one (partly on 256 x 256 CTA-pair tiles)."""
    from paper_2608_18469_b200 import binding
    gu = _gu()
    spec = {"relu_ragged": synth.mlp_spec(200, 328, 3, 600, "relu", "bf16"),
            "gelu_w1024": synth.mlp_spec(1024, 4096, 3, 4096, "gelu", "bf16"),
            "tower_relu": synth.mlp_spec(256, 512, 3, 1024, "relu", "bf16"),
            "wide_split": synth.mlp_spec(2048, 8192, 2, 512, "gelu", "bf16")}[name]
    if name == "tower_relu":
        for blk in spec["blocks"]:
            blk["kind"] = "tower"
    flat = synth.init_params(spec, 6)
    batches = [gu.DevBatch(spec, synth.make_batch(spec, 6, index=i)) for i in range(3)]
    serial = gu.run_steps(spec, flat, batches, n_streams=1)
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=1, flags=binding.PERSISTENT))
    _bits_equal(serial, gu.run_steps(spec, flat, batches, n_streams=1, flags=binding.PERSISTENT | binding.GRAPH))
    assert np.isfinite(serial["losses"]).all()
