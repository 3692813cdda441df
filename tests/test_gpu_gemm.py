"""The library's matrix multiplies (tensor-core and CUDA-core paths) against a float64 product."""
import numpy as np
import pytest
import torch

from paper_2408_08146_b200 import koala_gemm_bf16
from workloads.generate import normal_tensor

pytestmark = pytest.mark.gpu

SHAPES = [  # (tokens, out features, in features)
    (1, 128, 64), (10, 4096, 4096), (16, 256, 128), (17, 200, 192), (60, 1536, 4096),
    (64, 384, 11008), (40, 640, 5120), (256, 256, 1024), (300, 256, 512), (6, 32000, 4096),
    (250, 1280, 2048)]      # 256-row weight tiles (N = 256), several of them, ragged token tile


def _inputs(M, N, K):
    x = normal_tensor(7, f"x{M}.{N}.{K}", (M, K), 1.0, 0.0, torch.bfloat16, "cuda:0")
    w = normal_tensor(8, f"w{M}.{N}.{K}", (N, K), 0.02, 0.0, torch.bfloat16, "cuda:0")
    ref = x.double().cpu().numpy() @ w.double().cpu().numpy().T
    return x, w, ref


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("split", [0, 1, 3])
def test_tensor_core_gemm(shape, split):
    M, N, K = shape
    if split > K // 64:
        pytest.skip("fewer K blocks than splits")
    x, w, ref = _inputs(M, N, K)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    y = koala_gemm_bf16(x, w, True, split, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a bounded device-side wait ran out"
    err = np.abs(y.cpu().numpy() - ref).max()
    assert err <= 2e-5 * np.sqrt(K) + 1e-6, f"max err {err}"      # fp32 accumulation of K products


@pytest.mark.parametrize("shape", SHAPES[:8])
def test_cuda_core_gemm(shape):
    M, N, K = shape
    x, w, ref = _inputs(M, N, K)
    y = koala_gemm_bf16(x, w, False)
    torch.cuda.synchronize()
    err = np.abs(y.cpu().numpy() - ref).max()
    assert err <= 2e-5 * np.sqrt(K) + 1e-6, f"max err {err}"


@pytest.mark.parametrize("shape", [(10, 4096, 4096), (60, 1536, 4096), (100, 256, 11008), (130, 384, 512),
                                   (256, 256, 1024), (128, 512, 4096), (200, 1024, 2048), (120, 768, 1024)])
@pytest.mark.parametrize("tc", [True, False], ids=["tensor_core", "cuda_core"])
def test_gemm_with_activation_pairs(shape, tc):
    """fp32 activations given as a bf16 value + bf16 rounding residual: the product must be that of
    the pair's sum (about 16 significant bits of the activations)."""
    M, N, K = shape
    xf = normal_tensor(9, f"xf{M}.{N}.{K}", (M, K), 1.0, 0.0, torch.float32, "cuda:0")
    w = normal_tensor(8, f"w{M}.{N}.{K}", (N, K), 0.02, 0.0, torch.bfloat16, "cuda:0")
    hi = xf.to(torch.bfloat16)
    lo = (xf - hi.float()).to(torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    y = koala_gemm_bf16(hi, w, tc, 0, status, x_lo=lo)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref_pair = (hi.double() + lo.double()).cpu().numpy() @ w.double().cpu().numpy().T
    ref_full = xf.double().cpu().numpy() @ w.double().cpu().numpy().T
    assert np.abs(y.cpu().numpy() - ref_pair).max() <= 2e-5 * np.sqrt(K) + 1e-6
    # and the pair is a much better stand-in for the fp32 activations than plain bf16
    err_pair = np.abs(y.cpu().numpy() - ref_full).max()
    err_bf16 = np.abs(hi.double().cpu().numpy() @ w.double().cpu().numpy().T - ref_full).max()
    assert err_pair < 0.05 * err_bf16 + 1e-5


@pytest.mark.parametrize("shape", [(113, 1536, 1024), (128, 11008, 512), (129, 1024, 4096), (200, 700 * 16, 256),
                                   (256, 5120, 5120), (256, 512, 13824)])
def test_cta_pair_form_and_one_cta_form_agree(shape):
    """113 to 256 rows as a pair of activations: the CTA-pair kernel (default) and the one-CTA kernel
    (tuning key 17 = 1) both give the product of the pair's sum; ragged last tiles, one or many
    K blocks, one or many tiles per cluster."""
    from paper_2408_08146_b200 import binding
    lib = binding.load_library()
    M, N, K = shape
    xf = normal_tensor(11, f"xf{M}.{N}.{K}", (M, K), 1.0, 0.0, torch.float32, "cuda:0")
    w = normal_tensor(12, f"w{M}.{N}.{K}", (N, K), 0.02, 0.0, torch.bfloat16, "cuda:0")
    hi = xf.to(torch.bfloat16)
    lo = (xf - hi.float()).to(torch.bfloat16)
    ref = (hi.double() + lo.double()).cpu().numpy() @ w.double().cpu().numpy().T
    outs = []
    try:
        for off in (0, 1):
            lib.koala_set_tuning(17, off)
            status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
            y = koala_gemm_bf16(hi, w, True, 0, status, x_lo=lo)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            outs.append(y.cpu().numpy())
            assert np.abs(outs[-1] - ref).max() <= 2e-5 * np.sqrt(K) + 1e-6
    finally:
        lib.koala_set_tuning(17, 0)
    assert np.abs(outs[0] - outs[1]).max() <= 4e-5 * np.sqrt(K) + 1e-6
