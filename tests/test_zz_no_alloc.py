"""The allocation-free contraction entry point against the ordinary one.

tsfm_gemm_bf16_static serves callers that cannot allocate device memory while they work: a
serving loop whose other streams would be stalled by the device-wide synchronisation of
cudaMalloc / cudaFree, or a process whose device memory already belongs to a pooling allocator.
Its scratch is one fixed array shared by every call on the device, so the interesting cases are
calls in a row: the second call must not see what the first one left behind.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _operands(M, N, K, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    A = torch.randn((M, K), generator=g).to(torch.bfloat16).cuda()
    W = (torch.randn((N, K), generator=g) / K ** 0.5).to(torch.bfloat16).cuda()
    return A, W


def _both(tsfm, M, N, K, seed):
    """(static-scratch result, allocating entry point's result, fp64 product of the same operands)."""
    A, W = _operands(M, N, K, seed)
    s = torch.cuda.current_stream().cuda_stream
    want = torch.full((M, N), float("nan"), device="cuda")
    tsfm.tsfm_gemm_bf16(s, A, W, want, M, N, K, tsfm.TSFM_GEMM_AUTO)
    got = torch.full((M, N), float("nan"), device="cuda")
    tsfm.tsfm_gemm_bf16_static(s, A, W, got, M, N, K)
    torch.cuda.synchronize()
    exact = (A.cpu().double() @ W.cpu().double().T).numpy()
    return got.cpu().numpy(), want.cpu().numpy(), exact


def test_static_scratch_contraction_matches_the_allocating_one_on_calls_in_a_row():
    import paper_2511_18191_b200 as tsfm
    # a large call first, then smaller ones that reuse the front of the same scratch array, then
    # the first shape again: stale partial sums from any earlier call would show up as an error
    shapes = [(160, 1536, 512), (32, 512, 2048), (7, 130, 64), (160, 1536, 512)]
    for i, (M, N, K) in enumerate(shapes):
        got, want, exact = _both(tsfm, M, N, K, seed=10 + i)
        assert np.isfinite(got).all()
        # same tolerance as the tensor-core / FMA comparison of the contraction tests: the two
        # differ only in the order in which the K-split partial sums are added
        assert np.abs(got - want).max() < 2e-5 * K ** 0.5 + 1e-5, (i, M, N, K)
        # and against the product itself, not only against another kernel
        assert np.abs(got - exact).max() < 2e-5 * K ** 0.5 + 1e-5, (i, M, N, K)


def test_outputs_beyond_the_scratch_capacity_are_rejected_with_a_message():
    import paper_2511_18191_b200 as tsfm
    M, N, K = 1025, 1024, 64                       # M * N is one row past the 2^20-element limit
    assert M * N > tsfm.TSFM_STATIC_GEMM_MAX_ELEMS
    A, W = _operands(M, N, K, 3)
    out = torch.zeros((M, N), device="cuda")
    with pytest.raises(tsfm.TsfmError) as e:
        tsfm.tsfm_gemm_bf16_static(torch.cuda.current_stream().cuda_stream, A, W, out, M, N, K)
    assert e.value.code == tsfm.TSFM_ERR_SHAPE and "capacity" in str(e.value)
    assert float(out.abs().max()) == 0.0           # nothing was written
    # and the entry point still works afterwards
    got, want, exact = _both(tsfm, 64, 256, 128, seed=4)
    assert np.abs(got - want).max() < 2e-5 * 128 ** 0.5 + 1e-5
    assert np.abs(got - exact).max() < 2e-5 * 128 ** 0.5 + 1e-5
