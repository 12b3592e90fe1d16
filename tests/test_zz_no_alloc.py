"""The allocation-free projection entry point against the ordinary one.

echo_gemm_bf16_noalloc exists for callers that have no way to obtain device memory for the
kernel's scratch (allocator hooks, plug-ins without an allocator, processes whose memory another
runtime owns): its scratch is a fixed array inside the library.  This file is collected last on
purpose, so that a run that stops at the first failure has already exercised everything else.
The checks hold whether this file runs alone in a fresh process or after the other tests.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_02192_b200 import binding
    return binding


@pytest.mark.parametrize("M,N,K", [(32, 4096, 1024), (7, 688, 256), (16, 1024, 4096)])
def test_noalloc_matches_workspace_entry_twice_in_a_row(B, M, N, K):
    g = torch.Generator(device="cuda").manual_seed(M * 7 + N + K)
    X = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
    W = (torch.randn(N, K, device="cuda", generator=g) * 0.05).to(torch.bfloat16)
    want = B.echo_gemm_bf16(X, W, impl=2)                 # same kernel, caller-provided workspace
    exact = X.double() @ W.double().T                     # the fp64 product the other projection tests use
    tol = 2e-6 * K * 0.05 * 4 + 1e-6                      # the GEMM tests' fp32-accumulation bound
    Y = torch.empty((M, N), dtype=torch.float32, device="cuda")
    for _ in range(2):                                    # the shared scratch keeps the last call's contents
        Y.fill_(float("nan"))
        B.echo_gemm_bf16_noalloc(X, W, Y)
        assert B.echo_gemm_bf16_noalloc_status() == 0     # waits for the stream; no bounded wait ran out
        assert float((Y - want).abs().max()) < tol
        assert float((Y.double() - exact).abs().max()) < tol
    # residual-add epilogue on top of a known Y
    Y0 = torch.randn(M, N, device="cuda", generator=g)
    Y = Y0.clone()
    B.echo_gemm_bf16_noalloc(X, W, Y, epilogue=1)
    B.echo_gemm_bf16_noalloc(X, W, Y, epilogue=1)
    torch.cuda.synchronize()
    assert float((Y - (Y0 + 2 * want)).abs().max()) < 2 * tol + 1e-5


def test_noalloc_swiglu_and_limits(B):
    M, F, K = 24, 640, 512
    g = torch.Generator(device="cuda").manual_seed(3)
    X = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
    W = (torch.randn(2 * F, K, device="cuda", generator=g) * 0.05).to(torch.bfloat16)
    want = B.echo_gemm_bf16(X, W, impl=2, epilogue=2).float()
    Y = torch.empty((M, F), dtype=torch.bfloat16, device="cuda")
    for _ in range(2):
        Y.zero_()
        B.echo_gemm_bf16_noalloc(X, W, Y, epilogue=2)
        torch.cuda.synchronize()
        got = Y.float()
        assert bool(((got - want).abs() <= 2.0 ** -7 * want.abs() + 1e-4 * K / 256).all())
    # more rows than the built-in scratch covers: refused, nothing written
    Xb = torch.zeros(33, K, device="cuda", dtype=torch.bfloat16)
    Yb = torch.full((33, 2 * F), 5.0, device="cuda")
    with pytest.raises(B.EchoError) as ei:
        B.echo_gemm_bf16_noalloc(Xb, W, Yb)
    assert ei.value.code == -9
    torch.cuda.synchronize()
    assert bool((Yb == 5.0).all())
    # operands that the tile copies cannot address (not 16-byte aligned) are an argument error
    Xo = torch.zeros(M * K + 8, device="cuda", dtype=torch.bfloat16)[1: 1 + M * K].view(M, K)
    with pytest.raises(B.EchoError) as ei:
        B.echo_gemm_bf16_noalloc(Xo, W, torch.empty((M, 2 * F), device="cuda"))
    assert ei.value.code == -1
