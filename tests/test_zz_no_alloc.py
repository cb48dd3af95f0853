"""tasc_gemm_bf16_static: the product for callers that cannot allocate device memory (a process whose
memory pool was fixed at start-up, a host that forbids cudaMalloc after initialisation).  Its split-K
partial sums live in a fixed device array inside the library, shared by all calls and never cleared, so
the check runs two different products back to back and compares each with tasc_gemm_bf16, which uses a
caller-provided workspace.  Collected last on purpose: a failure here cannot hide another test's result."""
import numpy as np
import pytest
import torch

from oracle.model import linear
from tests.gpu_harness import need_gpu
from workload import rng
from workload.weights import round_to_bf16


def host_operands(tag, M, N, K):
    x = round_to_bf16(rng.normal(7, tag, 0, M * K, 1.0)).reshape(M, K)
    w = round_to_bf16(rng.normal(7, tag + 100, 0, N * K, 0.05)).reshape(N, K)
    return x, w


def operands(tag, M, N, K):
    x, w = host_operands(tag, M, N, K)
    return torch.from_numpy(x).cuda().bfloat16(), torch.from_numpy(w).cuda().bfloat16()


@pytest.mark.gpu
def test_static_scratch_gemm_matches_workspace_gemm_twice_in_a_row():
    b = need_gpu()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # a long-k product with many k-splits first, then a smaller one that finds the array full of the
    # first call's partial sums, then the first shape again
    for tag, (M, N, K) in enumerate([(130, 256, 4864), (6, 1152, 896), (130, 256, 4864), (300, 3072, 576)]):
        x, w = operands(tag, M, N, K)
        want = b.tasc_gemm_bf16(x, w)
        got = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        b.tasc_gemm_bf16_static(x, w, got, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # same tolerance as the GEMM tests: bf16 products are exact in float32, only the summation order
        # (number of k-splits) may differ between the two entry points
        tol = 1e-5 * np.sqrt(K) * float(want.abs().max()) + 1e-6
        assert float((got - want).abs().max()) <= tol
        # and against the plain definition y = x W^T in float64 on the CPU
        hx, hw = host_operands(tag, M, N, K)
        ref = linear(hx.astype(np.float64), hw.astype(np.float64))
        assert np.abs(got.cpu().numpy() - ref).max() <= 1e-5 * np.sqrt(K) * np.abs(ref).max() + 1e-6
    # without a caller status word
    x, w = operands(9, 17, 384, 256)
    got = torch.empty((17, 384), dtype=torch.float32, device="cuda")
    b.tasc_gemm_bf16_static(x, w, got)
    assert float((got - b.tasc_gemm_bf16(x, w)).abs().max()) <= 1e-5 * 16 * float(got.abs().max()) + 1e-6


@pytest.mark.gpu
def test_static_scratch_gemm_allocates_nothing():
    """What the entry point is for: across a call (after the first one on this device, which looks the array's
    address up) neither the driver's free-memory figure nor torch's allocator moves."""
    b = need_gpu()
    x, w = operands(21, 96, 1536, 576)
    y = torch.empty((96, 1536), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.tasc_gemm_bf16_static(x, w, y, status)            # first call on the device: address look-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        b.tasc_gemm_bf16_static(x, w, y, status)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free0 - free1 < (2 << 20)        # the driver hands out device memory in 2 MiB granules: none was taken
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    assert int(status.item()) == 0


@pytest.mark.gpu
def test_static_scratch_gemm_refuses_what_does_not_fit():
    b = need_gpu()
    M, N, K = 1024, 4096, 64                  # 16 MiB of float32 output: more than the 8 MiB array holds
    x = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((N, K), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    with pytest.raises(b.TascError) as e:
        b.tasc_gemm_bf16_static(x, w, y)
    assert e.value.code == b.ECAPACITY
    with pytest.raises(b.TascError) as e:     # K not a multiple of 8
        b.tasc_gemm_bf16_static(torch.zeros((4, 60), dtype=torch.bfloat16, device="cuda"),
                                torch.zeros((8, 60), dtype=torch.bfloat16, device="cuda"),
                                torch.zeros((4, 8), dtype=torch.float32, device="cuda"))
    assert e.value.code == b.EINVAL
