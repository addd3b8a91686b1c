"""erase_gemm_static, the GEMM for callers that cannot allocate device memory (a process whose
memory belongs to another pool, or a latency budget that rules out cudaMalloc).  Its split-K
workspace is a fixed array inside the library, so this checks, through the C ABI, that it gives
the same result as erase_gemm on two calls in a row (the second call sees the first call's
leftovers in the shared array) and that it refuses requests larger than the array."""
import numpy as np
import pytest

from paper_2608_18469_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _operands(M, N, K, seed):
    import torch
    rng = np.random.default_rng(seed)
    a = synth.bf16_round(rng.standard_normal((M, K)).astype(np.float32))
    b = synth.bf16_round(rng.standard_normal((N, K)).astype(np.float32))
    # wgrad layout: both operands contiguous along M/N, strided over k
    ta = torch.from_numpy(a.T.copy()).to(torch.bfloat16).cuda()
    tb = torch.from_numpy(b.T.copy()).to(torch.bfloat16).cuda()
    torch.cuda.synchronize()
    return a, b, ta, tb


@pytest.mark.parametrize("engine", [1, 0])
def test_static_scratch_gemm_matches_allocating_gemm_twice_in_a_row(engine):
    import torch
    # first a large split-K problem, then a smaller one that reuses the dirty front of the array
    for call, (M, N, K, splits) in enumerate([(256, 192, 2048, 8), (128, 64, 1000, 5)]):
        a, b, ta, tb = _operands(M, N, K, seed=call)
        ref = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        args = ("bf16", M, N, K, ta.data_ptr(), 1, M, tb.data_ptr(), 1, N)
        binding.gemm(*args, ref.data_ptr(), N, c_f32=True, splits=splits, engine=engine)
        if call == 1:
            # by now the one-time set-up has run: the call must leave the device's free memory as it is
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
        binding.gemm_static(*args, out.data_ptr(), N, c_f32=True, splits=splits, engine=engine)
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free_before
        got, want = out.cpu().numpy(), ref.cpu().numpy()
        assert np.isfinite(got).all()
        # same kernels, same fixed split and summation order: the two entry points agree bit for bit
        assert got.tobytes() == want.tobytes()
        exact = a.astype(np.float64) @ b.astype(np.float64).T
        assert synth.rel_l2(got, exact) < 2e-5


def test_static_scratch_gemm_without_split_uses_only_the_status_words():
    """splits = 1 on the tensor-core kernel: nothing of the workspace is touched, only the status
    word and the tile-scheduler words behind it."""
    import torch
    M, N, K = 384, 256, 512
    a, b, ta, tb = _operands(M, N, K, seed=5)
    ref = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    args = ("bf16", M, N, K, ta.data_ptr(), 1, M, tb.data_ptr(), 1, N)
    binding.gemm(*args, ref.data_ptr(), N, c_f32=True, splits=1, engine=1)
    for _ in range(2):
        binding.gemm_static(*args, out.data_ptr(), N, c_f32=True, splits=1, engine=1)
        assert out.cpu().numpy().tobytes() == ref.cpu().numpy().tobytes()


def test_static_scratch_gemm_refuses_oversized_workspace():
    # real, correctly sized operands: only the workspace request (2 * 2048 * 2048 floats) is too big
    M = N = 2048
    K = 256
    a, b, ta, tb = _operands(M, N, K, seed=9)
    import torch
    out = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    assert 2 * M * N > binding.STATIC_WS_FLOATS
    with pytest.raises(binding.EraseError) as e:
        binding.gemm_static("bf16", M, N, K, ta.data_ptr(), 1, M, tb.data_ptr(), 1, N, out.data_ptr(), N,
                            c_f32=True, splits=2, engine=0)
    assert e.value.status == binding.EINVAL
    assert "static maximum" in str(e.value)
    assert float(out.abs().sum()) == 0.0      # nothing was launched
