"""tcgen05 GEMM against the plain definition y = x W^T evaluated in float64 on the CPU."""
import numpy as np
import pytest
import torch

from oracle.model import linear
from tests.gpu_harness import need_gpu
from workload import rng
from workload.weights import round_to_bf16

SHAPES = [
    (1, 128, 64),          # one tile, one k-block
    (6, 1152, 896),        # 0.5B QKV at batch 1
    (6, 960, 576),         # ragged last weight tile (960 = 7.5 * 128)
    (7, 200, 72),          # ragged everything: N not a multiple of 128, K not a multiple of 64
    (16, 576, 1536),
    (17, 384, 256),        # token tile of 32 with 15 padded rows
    (96, 9728, 896),       # gate/up at batch 16
    (130, 256, 4864),      # long k-loop, split-K
    (448, 1536, 1536),     # two token tiles of 224
    (1024, 640, 128),      # prefill-sized row count: four token tiles
]


@pytest.mark.gpu
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_gemm_matches_float64_definition(M, N, K):
    b = need_gpu()
    x = round_to_bf16(rng.normal(1, 1, 0, M * K, 1.0)).reshape(M, K)
    w = round_to_bf16(rng.normal(1, 2, 0, N * K, 0.05)).reshape(N, K)
    y = b.tasc_gemm_bf16(torch.from_numpy(x).cuda().bfloat16(), torch.from_numpy(w).cuda().bfloat16()).cpu().numpy()
    ref = linear(x.astype(np.float64), w.astype(np.float64))
    # bf16 products are exact in float32; only the float32 accumulation order differs
    tol = 1e-5 * np.sqrt(K) * np.abs(ref).max() + 1e-6
    assert np.abs(y - ref).max() <= tol, (np.abs(y - ref).max(), tol)


@pytest.mark.gpu
def test_gemm_is_bitwise_repeatable():
    b = need_gpu()
    x = torch.from_numpy(round_to_bf16(rng.normal(2, 1, 0, 24 * 896, 1.0)).reshape(24, 896)).cuda().bfloat16()
    w = torch.from_numpy(round_to_bf16(rng.normal(2, 2, 0, 1152 * 896, 0.05)).reshape(1152, 896)).cuda().bfloat16()
    a = b.tasc_gemm_bf16(x, w)
    for _ in range(3):
        assert torch.equal(a, b.tasc_gemm_bf16(x, w))


@pytest.mark.gpu
def test_gemm_rejects_bad_arguments():
    b = need_gpu()
    x = torch.zeros((4, 60), dtype=torch.bfloat16, device="cuda")       # K not a multiple of 8
    w = torch.zeros((8, 60), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.TascError):
        b.tasc_gemm_bf16(x, w)


@pytest.mark.gpu
@pytest.mark.parametrize("M,N,K", [(6, 1152, 896), (7, 200, 72), (96, 960, 576), (130, 256, 4864), (300, 384, 256)])
def test_paired_gemm_keeps_float32_activations(M, N, K):
    """float32 X carried as (hi, lo) bf16 pairs: the error must be far below a plain bf16 rounding of X."""
    b = need_gpu()
    x = rng.normal(3, 1, 0, M * K, 1.0).reshape(M, K)                       # not bf16-representable
    w = round_to_bf16(rng.normal(3, 2, 0, N * K, 0.05)).reshape(N, K)
    y = b.tasc_gemm_bf16x2(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda().bfloat16()).cpu().numpy()
    ref = linear(x.astype(np.float64), w.astype(np.float64))
    err = np.abs(y - ref).max()
    err_if_rounded = np.abs(linear(round_to_bf16(x).astype(np.float64), w.astype(np.float64)) - ref).max()
    # hi + lo keeps 16 mantissa bits of x: error 2^-17 relative per term instead of 2^-9
    assert err <= 3e-5 * np.sqrt(K) * np.abs(w).max() * np.abs(x).max() + 1e-6, err
    assert err < err_if_rounded / 30
