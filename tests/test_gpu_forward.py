"""Forward-pass numerics of the CUDA kernels against the oracle's network, and the tensor-core
contraction against the FMA kernel and an fp64 product."""
import numpy as np
import pytest
import torch

import tests.parity as parity
from oracle import tsfm_oracle as orc
from tsfm_inputs import Arch, Workload, build_models

pytestmark = pytest.mark.gpu


def small_workload(dtype, target, draft, P=32, mode="separate", patch_in=0):
    return Workload("T", 5, 8 * P, P, 4 * P, 3, 1.0, dtype, target, draft, mode, "c1", series_seed=77,
                    patch_in=patch_in)


def run_forward_case(wl, backend, n_tokens, B=5, seed=0):
    import paper_2511_18191_b200 as tsfm
    tw, dw = build_models(wl)
    dec = tsfm.SpecDecoder(tw, dw, wl.target, wl.draft, wl.patch_len, wl.dtype,
                           "layer_skip" if wl.draft_mode == "layer_skip" else "separate",
                           max_batch=B, max_ctx_tokens=n_tokens, max_horizon_patches=4, max_K=4,
                           gemm_backend=backend, patch_in=wl.patch_in)
    rng = np.random.default_rng(seed)
    z = rng.standard_normal((B, n_tokens, wl.token_len)).astype(np.float32)
    zt = torch.from_numpy(z).cuda()
    got_t = dec.model_forward(0, zt).cpu().numpy()
    got_d = dec.model_forward(1, zt).cpu().numpy()
    dec.close()
    tm, dm = parity.oracle_models(wl, tw, dw)
    want_t = np.stack([orc.forward(tm, z[b].astype(np.float64)) for b in range(B)])
    want_d = np.stack([orc.forward(dm, z[b].astype(np.float64)) for b in range(B)])
    return got_t, want_t, got_d, want_d


@pytest.mark.parametrize("target,draft,P,n", [
    (Arch(2, 128, 4, 512), Arch(1, 64, 2, 256), 96, 7),        # C0's models (head size 32)
    (Arch(2, 128, 2, 256), Arch(1, 128, 1, 128), 32, 21),      # head sizes 64 and 128, several query tiles
    (Arch(1, 128, 2, 256), Arch(1, 64, 2, 128), 32, 197),      # long rows: keys split over a cluster, ragged tail
])
def test_fp32_forward_matches_oracle(target, draft, P, n):
    wl = small_workload("f32", target, draft, P)
    gt, wt, gd, wd = run_forward_case(wl, 0, n)
    assert np.abs(gt - wt).max() < 1e-4
    assert np.abs(gd - wd).max() < 1e-4


@pytest.mark.parametrize("backend", [1, 0], ids=["simt", "tcgen05"])
@pytest.mark.parametrize("target,draft,P,n,mode", [
    (Arch(3, 256, 4, 1024), Arch(2, 128, 4, 256), 96, 9, "separate"),      # few tokens: folded norms, K split
    (Arch(4, 512, 8, 2048), Arch(2, 512, 8, 2048), 32, 37, "layer_skip"),  # 185 tokens, layer-skip draft
    (Arch(4, 512, 8, 2048), Arch(2, 512, 8, 2048), 32, 6, "layer_skip"),   # 30 tokens: one 32-token tile
    (Arch(2, 384, 6, 1536), Arch(1, 128, 2, 256), 96, 3, "separate"),      # 6 heads: 3 feature tiles
    (Arch(2, 256, 4, 1024), Arch(1, 128, 2, 256), 32, 120, "separate"),    # 120 keys: tensor-core attention tiles
    (Arch(2, 256, 4, 1024), Arch(1, 128, 2, 256), 32, 200, "separate"),    # 200 keys: several chunks of the key stream
    (Arch(2, 256, 2, 512), Arch(1, 64, 2, 128), 32, 75, "separate"),       # head sizes 128 and 32, ragged last tile
])
def test_bf16_forward_matches_oracle(backend, target, draft, P, n, mode):
    wl = small_workload("bf16", target, draft, P, mode)
    gt, wt, gd, wd = run_forward_case(wl, backend, n)
    assert parity.value_error("rel_rms", gt, wt) < 2e-2
    assert parity.value_error("rel_rms", gd, wd) < 2e-2


@pytest.mark.parametrize("dtype,P,P_in,n", [("f32", 16, 1, 70), ("f32", 32, 8, 19), ("bf16", 64, 1, 300), ("bf16", 32, 16, 40)])
def test_forward_with_input_tokens_shorter_than_the_patch(dtype, P, P_in, n):
    """Embedding of P_in-step tokens ([d, P_in] weights; 16-byte loads or element by element) under a
    P-step head: next-patch means at every token."""
    wl = small_workload(dtype, Arch(2, 128, 2, 256), Arch(1, 64, 2, 128), P, patch_in=P_in)
    gt, wt, gd, wd = run_forward_case(wl, 0, n, B=3)
    if dtype == "f32":
        assert np.abs(gt - wt).max() < 1e-4 and np.abs(gd - wd).max() < 1e-4
    else:
        assert parity.value_error("rel_rms", gt, wt) < 2e-2 and parity.value_error("rel_rms", gd, wd) < 2e-2


@pytest.mark.parametrize("M,N,K", [(1, 128, 64), (16, 128, 64), (32, 1536, 512), (160, 512, 2048), (33, 96, 128),
                                   (200, 200, 192), (40, 512, 96), (7, 130, 16), (960, 2048, 512), (300, 384, 1280), (2048, 768, 768)])
def test_tensor_core_gemm_matches_fp64_product_and_fma_kernel(M, N, K):
    import paper_2511_18191_b200 as tsfm
    g = torch.Generator(device="cpu").manual_seed(M * 7 + N)
    A = torch.randn((M, K), generator=g).to(torch.bfloat16)
    W = (torch.randn((N, K), generator=g) / K ** 0.5).to(torch.bfloat16)
    want = (A.double() @ W.double().T).numpy()
    Ad, Wd = A.cuda(), W.cuda()
    outs = {}
    for name, backend in (("simt", tsfm.TSFM_GEMM_SIMT), ("tc", tsfm.TSFM_GEMM_AUTO)):
        Cd = torch.full((M, N), float("nan"), device="cuda")
        tsfm.tsfm_gemm_bf16(torch.cuda.current_stream().cuda_stream, Ad, Wd, Cd, M, N, K, backend)
        torch.cuda.synchronize()
        outs[name] = Cd.cpu().numpy()
        assert np.isfinite(outs[name]).all(), name
        assert np.abs(outs[name] - want).max() < 2e-5 * K ** 0.5 + 1e-5, name
    assert np.abs(outs["tc"] - outs["simt"]).max() < 2e-5 * K ** 0.5 + 1e-5


@pytest.mark.parametrize("M,N,K", [(1, 128, 64), (16, 130, 64), (32, 1536, 512), (33, 96, 128), (40, 512, 192), (64, 384, 1536),
                                   (128, 1152, 384), (31, 512, 2048), (256, 66, 448), (160, 1536, 512)])
def test_small_batch_gemm_matches_fp64_product(M, N, K):
    """The kernel that keeps its weight tile in shared memory (few tokens, K up to 2048): ragged token
    and feature tiles, every k step distribution over its eight warps, and the refusal outside its domain."""
    import paper_2511_18191_b200 as tsfm
    g = torch.Generator(device="cpu").manual_seed(M * 11 + N)
    A = torch.randn((M, K), generator=g).to(torch.bfloat16)
    W = (torch.randn((N, K), generator=g) / K ** 0.5).to(torch.bfloat16)
    Ad, Wd = A.cuda(), W.cuda()
    Cd = torch.full((M, N), float("nan"), device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    if (M, N, K) == (160, 1536, 512):                     # 480 CTAs: more than one wave, not this kernel's job
        with pytest.raises(tsfm.TsfmError) as e:
            tsfm.tsfm_gemm_bf16(s, Ad, Wd, Cd, M, N, K, tsfm.TSFM_GEMM_WS)
        assert e.value.code == tsfm.TSFM_ERR_SHAPE
        return
    tsfm.tsfm_gemm_bf16(s, Ad, Wd, Cd, M, N, K, tsfm.TSFM_GEMM_WS)
    torch.cuda.synchronize()
    got = Cd.cpu().numpy()
    want = (A.double() @ W.double().T).numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() < 2e-5 * K ** 0.5 + 1e-5
