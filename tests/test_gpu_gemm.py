"""Decoder GEMM through the C ABI against a plain fp32 matrix product of the same bf16 / fp32 inputs."""
import numpy as np
import pytest

from paper_2608_18183_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx_bf16():
    w = synth.WORKLOADS["tiny_bf16"]
    c = binding.Context(w.shape, G.weights_for(w), 4, 8)
    yield c
    c.hbsjd_destroy()


@pytest.fixture(scope="module")
def ctx_fp32():
    w = synth.WORKLOADS["tiny"]
    c = binding.Context(w.shape, G.weights_for(w), 4, 8)
    yield c
    c.hbsjd_destroy()


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (128, 64, 128), (64, 32, 64), (200, 384, 128), (1000, 768, 768),
                                   (1024, 2304, 768), (333, 4096, 768), (1024, 768, 2048), (4096, 1024, 2816),
                                   (2048, 16384, 1024), (1, 128, 64), (8192, 3072, 1024), (8192, 1024, 1024),
                                   (5000, 2048, 512), (4999, 5632, 1024), (2304, 16384, 256)])
def test_bf16_gemm_matches_fp32_product(ctx_bf16, M, N, K):
    import torch
    g = torch.Generator(device="cuda").manual_seed(M * 7 + N * 3 + K)
    A = (torch.randn(M, K, generator=g, device="cuda") * 0.5).bfloat16()
    W = (torch.randn(N, K, generator=g, device="cuda") * 0.05).bfloat16()
    C = torch.full((M, N), 7.0, device="cuda", dtype=torch.float32)
    ctx_bf16.hbsjd_gemm(A, W, C)
    ref = A.float() @ W.float().T
    scale = float(ref.abs().max())
    # fp32 accumulation of exact bf16 products: differences are summation-order rounding only
    assert float((C - ref).abs().max()) <= 2e-5 * max(scale, 1.0) * (K / 64) ** 0.5 + 1e-6
    # accumulate mode adds into C
    C0 = torch.randn(M, N, generator=g, device="cuda")
    C1 = C0.clone()
    ctx_bf16.hbsjd_gemm(A, W, C1, accumulate=True)
    assert float((C1 - (C0 + ref)).abs().max()) <= 2e-5 * max(scale, 1.0) * (K / 64) ** 0.5 + 1e-5


def test_bf16_gemm_rows_do_not_depend_on_their_tile(ctx_bf16):
    """A row's result is bit-identical wherever it sits in the batch (what lets Full and Compact
    execution agree bit for bit)."""
    import torch
    g = torch.Generator(device="cuda").manual_seed(5)
    A = torch.randn(512, 768, generator=g, device="cuda").bfloat16()
    W = (torch.randn(768, 768, generator=g, device="cuda") * 0.05).bfloat16()
    C = torch.empty(512, 768, device="cuda")
    ctx_bf16.hbsjd_gemm(A, W, C)
    perm = torch.randperm(512, generator=g, device="cuda")[:77]
    A2 = A[perm].contiguous()
    C2 = torch.empty(77, 768, device="cuda")
    ctx_bf16.hbsjd_gemm(A2, W, C2)
    assert torch.equal(C2, C[perm])


@pytest.mark.parametrize("M,N,K", [(7, 192, 64), (130, 256, 192), (64, 64, 64)])
def test_fp32_gemm(ctx_fp32, M, N, K):
    import torch
    g = torch.Generator(device="cuda").manual_seed(M + N + K)
    A = torch.randn(M, K, generator=g, device="cuda")
    W = torch.randn(N, K, generator=g, device="cuda") * 0.1
    C = torch.zeros(M, N, device="cuda")
    ctx_fp32.hbsjd_gemm(A, W, C)
    ref = (A.double() @ W.double().T).float()
    assert float((C - ref).abs().max()) < 1e-5 * K ** 0.5


def test_bounded_wait_runs_out_and_the_context_recovers(ctx_bf16):
    """The failure path of the GEMM pipeline on a healthy GPU: the epilogue warps' bounded wait for their
    accumulator is shortened to 300 ns while the main loop over K = 8192 needs tens of microseconds, so the wait
    runs out.  The kernel must not hang or fault: it raises its error flag, every role leaves its loop, the copies
    and MMAs in flight are drained, TMEM is freed, and the call returns HBSJD_ETIMEOUT (-5).  The next call on the
    same context runs normally and is correct.  (One CTA per tile: the shape is too small for CTA pairs.)"""
    import torch
    g = torch.Generator(device="cuda").manual_seed(11)
    M, N, K = 256, 256, 8192
    A = (torch.randn(M, K, generator=g, device="cuda") * 0.5).bfloat16()
    W = (torch.randn(N, K, generator=g, device="cuda") * 0.05).bfloat16()
    C = torch.zeros(M, N, device="cuda")
    with pytest.raises(binding.HbsjdError) as e:
        ctx_bf16.hbsjd_debug_gemm(A, W, C, acc_wait_ns=300)
    assert e.value.code == -5
    torch.cuda.synchronize()
    C2 = torch.zeros(M, N, device="cuda")
    ctx_bf16.hbsjd_gemm(A, W, C2)
    ref = A.float() @ W.float().T
    assert float((C2 - ref).abs().max()) <= 2e-5 * max(float(ref.abs().max()), 1.0) * (K / 64) ** 0.5 + 1e-6
    # several launches back to back through the same entry point give the same result as one
    C3 = torch.zeros(M, N, device="cuda")
    ctx_bf16.hbsjd_debug_gemm(A, W, C3, reps=3)
    assert torch.equal(C3, C2)
