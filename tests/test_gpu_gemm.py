"""The GEMM entry point against a float64 matmul: SIMT and tcgen05 engines, the three operand
layouts of forward / dgrad / wgrad, ragged sizes, split-K."""
import numpy as np
import pytest

from paper_2608_18469_b200 import binding, synth

pytestmark = pytest.mark.gpu

# (M, N, K): several 128-wide tiles with ragged tails; K tails that are not multiples of 64
SHAPES = [(128, 128, 64), (256, 128, 256), (300, 200, 136), (512, 64, 1680), (1000, 416, 328),
          (130, 24, 72), (4096, 768, 256)]
LAYOUTS = {"fwd": (False, False), "dgrad": (False, True), "wgrad": (True, True), "a_mn": (True, False)}


def _run(dtype, M, N, K, a_mn, b_mn, engine, splits=1, c_f32=False, seed=0):
    import torch
    rng = np.random.default_rng(seed)
    a = rng.standard_normal((M, K)).astype(np.float32)
    b = rng.standard_normal((N, K)).astype(np.float32)
    if dtype == "bf16":
        a, b = synth.bf16_round(a), synth.bf16_round(b)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    # physical storage: K-major = [rows, K] contiguous; MN-major = [K, rows] contiguous
    ta = torch.from_numpy(a.T.copy() if a_mn else a).to(tdt).cuda()
    tb = torch.from_numpy(b.T.copy() if b_mn else b).to(tdt).cuda()
    out_f32 = c_f32 or dtype == "f32"
    tc = torch.full((M, N), float("nan"), dtype=torch.float32 if out_f32 else tdt, device="cuda")
    torch.cuda.synchronize()
    sa = (1, M) if a_mn else (K, 1)
    sb = (1, N) if b_mn else (K, 1)
    binding.gemm(dtype, M, N, K, ta.data_ptr(), sa[0], sa[1], tb.data_ptr(), sb[0], sb[1], tc.data_ptr(), N,
                 c_f32=out_f32, splits=splits, engine=engine)
    got = tc.float().cpu().numpy().astype(np.float64)
    want = a.astype(np.float64) @ b.astype(np.float64).T
    return synth.rel_l2(got, want)


@pytest.mark.parametrize("layout", list(LAYOUTS))
@pytest.mark.parametrize("shape", SHAPES)
def test_tensor_core_gemm_bf16(shape, layout):
    M, N, K = shape
    a_mn, b_mn = LAYOUTS[layout]
    if (a_mn and M % 8) or (b_mn and N % 8) or (not a_mn and K % 8) or (not b_mn and K % 8):
        pytest.skip("leading stride not a multiple of 8 elements: the SIMT kernel takes it")
    # bf16 operands are exact inputs; products accumulate in fp32, the result is rounded to bf16
    assert _run("bf16", M, N, K, a_mn, b_mn, engine=1) < 4e-3
    assert _run("bf16", M, N, K, a_mn, b_mn, engine=1, c_f32=True) < 2e-5


# Shapes that the CTA-pair kernel takes (256 x 256 tiles over two SMs, at least 56 of them): full
# tiles, ragged M / N / K tails, a single K block, a peer CTA whose rows lie wholly outside M.
PAIR_SHAPES = [(2048, 2048, 192), (3896, 1032, 200), (4096, 8192, 64), (14400 + 8, 264, 136)]


@pytest.mark.parametrize("layout", list(LAYOUTS))
@pytest.mark.parametrize("shape", PAIR_SHAPES)
def test_cta_pair_gemm_bf16(shape, layout):
    M, N, K = shape
    a_mn, b_mn = LAYOUTS[layout]
    assert _run("bf16", M, N, K, a_mn, b_mn, engine=1) < 4e-3
    assert _run("bf16", M, N, K, a_mn, b_mn, engine=1, c_f32=True) < 2e-5


@pytest.mark.parametrize("layout", list(LAYOUTS))
def test_cta_pair_split_k(layout):
    a_mn, b_mn = LAYOUTS[layout]
    assert _run("bf16", 2048, 512, 4096 + 72, a_mn, b_mn, engine=1, splits=7, c_f32=True) < 2e-5
    assert _run("bf16", 4096, 256, 200, a_mn, b_mn, engine=1, splits=4, c_f32=True) < 2e-5   # trailing empty split


@pytest.mark.parametrize("layout", list(LAYOUTS))
def test_tensor_core_split_k_matches_and_is_deterministic(layout):
    a_mn, b_mn = LAYOUTS[layout]
    assert _run("bf16", 256, 192, 4096, a_mn, b_mn, engine=1, splits=7, c_f32=True) < 2e-5
    assert _run("bf16", 128, 128, 200, a_mn, b_mn, engine=1, splits=4, c_f32=True) < 2e-5   # trailing empty split


@pytest.mark.parametrize("layout", list(LAYOUTS))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_simt_gemm(dtype, layout):
    a_mn, b_mn = LAYOUTS[layout]
    for (M, N, K) in [(70, 33, 19), (300, 200, 136), (64, 1, 257)]:
        tol = 2e-6 if dtype == "f32" else 4e-3
        assert _run(dtype, M, N, K, a_mn, b_mn, engine=0) < tol
        assert _run(dtype, M, N, K, a_mn, b_mn, engine=0, splits=3, c_f32=True) < 2e-5


def test_unsupported_shapes_are_refused_not_mangled():
    import torch
    t = torch.zeros(64 * 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.EraseError) as e:
        binding.gemm("bf16", 64, 8, 64, t.data_ptr(), 64, 1, t.data_ptr(), 64, 1, t.data_ptr(), 8, engine=1)
    assert e.value.status == binding.EUNSUPPORTED
    with pytest.raises(binding.EraseError) as e:
        binding.gemm("f32", 64, 64, 64, t.data_ptr(), 64, 1, t.data_ptr(), 64, 1, t.data_ptr(), 64, engine=1)
    assert e.value.status == binding.EUNSUPPORTED
