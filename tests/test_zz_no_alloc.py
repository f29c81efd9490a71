"""The no-allocation GEMM entry point, q4d_q4_gemm_noalloc.

It exists for callers that cannot allocate device memory when they need a projection (a plugin whose
host owns all device memory, code inside an allocator callback, a loop where cudaMalloc's device-wide
synchronisation is not acceptable).  Its scratch is an array built into the library, shared by all calls,
so the test calls it twice in a row with different shapes and checks each result against the ordinary
entry point q4d_q4_gemm, which runs the same kernel on caller-provided scratch: the results must be
identical.  This file sorts last so that a run stopping at the first failure has run everything else.
"""
import gc

import numpy as np
import pytest
import torch

from gpu_util import assert_bf16_close, bits
from oracle import q4d_oracle as orc
from workload import gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q4d():
    from paper_2601_19139_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def _x(n, K, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return torch.randn(n, K, generator=g, device="cuda").to(torch.bfloat16)


def test_noalloc_gemm_equals_the_scratch_taking_entry_point_twice_in_a_row(q4d):
    # outputs are allocated before the calls under test: the entry point itself must allocate nothing
    cases = [(4096, 12288, 16, 2), (1024, 8192, 5, 0)]    # K > 4096: partial sums go through the array
    prepared = []
    for i, (N, K, n, epi) in enumerate(cases):
        w = gen.random_q4(N, K, "cuda", "noalloc", i)
        x = _x(n, K, 40 + i)
        out = torch.full((n, N), float("nan"), dtype=torch.float32 if epi == 2 else torch.bfloat16, device="cuda")
        prepared.append((w, x, n, epi, out))
    # a first call loads the kernels and looks up the array's address (both may take device memory once, in the
    # driver); the calls under test come after it
    q4d.q4_gemm_noalloc(prepared[1][0], prepared[1][1], prepared[1][2], prepared[1][4], epilogue=prepared[1][3])
    torch.cuda.synchronize()
    # tensors of earlier tests that only the cycle collector can free must not be freed between the two readings
    gc.collect()
    gc.disable()
    try:
        before = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]
        for w, x, n, epi, out in prepared:                 # two calls in a row on the shared array
            q4d.q4_gemm_noalloc(w, x, n, out, epilogue=epi)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert torch.cuda.mem_get_info()[0] == free_before  # nor did anything else take device memory
    finally:
        gc.enable()
    for w, x, n, epi, out in prepared:
        want = q4d.q4_gemm(w, x, n, epilogue=epi)
        torch.cuda.synchronize()
        assert torch.equal(out, want)
        # and against the definition itself, not only the sibling entry point
        ref = orc.q4_matmul(*(orc.to_np(a) for a in w), bits(x))
        rms = np.sqrt((ref ** 2).mean())
        if epi == 2:
            assert np.abs(out.cpu().numpy().astype(np.float64) - ref).max() <= 3e-5 * rms
        else:
            assert_bf16_close(bits(out), orc.bf16_round(ref), what="no-alloc bf16 output")
    # and again in the other order: what the previous call left in the array must not matter
    for w, x, n, epi, out in reversed(prepared):
        out.fill_(float("nan"))
        q4d.q4_gemm_noalloc(w, x, n, out, epilogue=epi)
        torch.cuda.synchronize()
        assert torch.equal(out, q4d.q4_gemm(w, x, n, epilogue=epi))


def test_noalloc_gemm_residual_epilogue_and_silu_prologue(q4d):
    """The other two modes of the entry point, each against the scratch-taking one and against the oracle."""
    N, K, n = 2048, 1024, 7
    w = gen.random_q4(N, K, "cuda", "noalloc-modes")
    x = _x(n, K, 60)
    res = _x(n, N, 61)
    res2 = res.clone()
    q4d.q4_gemm_noalloc(w, x, n, res, epilogue=1)
    q4d.q4_gemm(w, x, n, epilogue=1, out=res2)
    torch.cuda.synchronize()
    assert torch.equal(res, res2)
    gu = _x(n, 2 * K, 62)
    out = torch.zeros(n, N, dtype=torch.float32, device="cuda")
    q4d.q4_gemm_noalloc(w, gu, n, out, prologue=1, epilogue=2)
    torch.cuda.synchronize()
    assert torch.equal(out, q4d.q4_gemm(w, gu, n, prologue=1, epilogue=2))
    gub = bits(gu)
    ref = orc.q4_matmul(*(orc.to_np(a) for a in w), orc.silu_mul(gub[:, :K], gub[:, K:]))
    assert np.abs(out.cpu().numpy().astype(np.float64) - ref).max() <= 2e-3 * np.sqrt((ref ** 2).mean())
    with pytest.raises(q4d.Q4dError) as ei:                 # a row stride shorter than the operand's row
        q4d.q4_gemm_noalloc(w, _x(n, K // 2, 63), n, out, epilogue=2)
    assert ei.value.code == -1


def test_noalloc_gemm_refuses_shapes_beyond_its_array(q4d):
    N, K, n = 69632, 8192, 16                              # 2 x 69632 x 16 partial sums: more than 8 MiB
    w = gen.random_q4(N, K, "cuda", "noalloc-big")
    x = _x(n, K, 50)
    out = torch.zeros(n, N, dtype=torch.float32, device="cuda")
    with pytest.raises(q4d.Q4dError) as ei:
        q4d.q4_gemm_noalloc(w, x, n, out, epilogue=2)
    assert ei.value.code == -8 and "scratch" in str(ei.value)
    assert q4d.lib().q4d_noalloc_max_scratch_bytes() == 8 << 20
