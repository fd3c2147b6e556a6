"""mxfp4_gemm_static: the product for callers that may not allocate device memory.

Such a caller (an extension living inside a runtime that owns all device memory, a step during which
the allocator is off limits) cannot hand mxfp4_gemm its split-K workspace.  The static entry point
keeps that workspace in a fixed device array inside the library.  This file checks, through the C ABI,
that it gives what mxfp4_gemm gives -- twice in a row, because the array is reused and keeps the
previous call's contents -- and that it refuses shapes that do not fit.  It is named to be collected
last, and it passes on its own in a fresh process as well as after the other tests.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


def _operand(mx, rows, kc, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    q = mx.QMat(rows, kc)
    q.data.copy_(torch.randint(0, 256, q.data.shape, dtype=torch.uint8, device="cuda", generator=g))
    q.scales.copy_(torch.randint(118, 136, q.scales.shape, dtype=torch.uint8, device="cuda", generator=g))
    return q


# (M, N, kc): two shapes that need split-K scratch (short output, long contraction) and one that needs none
@pytest.mark.parametrize("M,N,K,out_dtype", [(384, 256, 8192, 1), (640, 384, 6400, 0), (512, 512, 512, 0)])
def test_static_scratch_gemm_matches_gemm_twice(mx, M, N, K, out_dtype):
    a, b = _operand(mx, M, K, 1), _operand(mx, N, K, 2)
    st = mx.new_status()
    want = mx.gemm(a, b, out_dtype=out_dtype, dev_status=st)
    # a second product in between leaves other partial sums in the shared array
    a2, b2 = _operand(mx, N, K, 3), _operand(mx, M, K, 4)
    want2 = mx.gemm(a2, b2, out_dtype=out_dtype, dev_status=st)
    got = torch.empty_like(want)
    got2 = torch.empty_like(want2)
    for _ in range(2):
        got.fill_(float("nan"))
        got2.fill_(float("nan"))
        mx.gemm_static(a, b, got, out_dtype=out_dtype, dev_status=st)
        mx.gemm_static(a2, b2, got2, out_dtype=out_dtype, dev_status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        # Both entry points run the same kernels with the same fixed summation order, so the results
        # agree exactly; the bound the other GEMM tests use, 2^-20 * sum|a*b|, is far looser than this.
        assert torch.equal(got, want)
        assert torch.equal(got2, want2)


def test_static_scratch_gemm_adds_the_bias(mx):
    """The bias is added by the reduction over the fixed array's partial sums, exactly as mxfp4_gemm adds it."""
    M, N, K = 640, 384, 6400
    assert mx.gemm_workspace_bytes(M, N, K) > 0
    a, b = _operand(mx, M, K, 5), _operand(mx, N, K, 6)
    bias = (torch.randn(N, device="cuda") * 3).to(torch.bfloat16)
    for out_dtype in (0, 1):
        want = mx.gemm(a, b, out_dtype=out_dtype, bias=bias)
        plain = mx.gemm(a, b, out_dtype=out_dtype)
        got = torch.full_like(want, float("nan"))
        mx.gemm_static(a, b, got, out_dtype=out_dtype, bias=bias)
        torch.cuda.synchronize()
        assert torch.equal(got, want)
        assert not torch.equal(got, plain)


def test_static_scratch_gemm_refuses_what_does_not_fit(mx):
    M, N, K = 512, 512, 36864  # eighteen split-K partial sums of 512 x 512 floats exceed the fixed array
    assert mx.gemm_workspace_bytes(M, N, K) > mx.STATIC_SCRATCH_BYTES
    a, b = mx.QMat(M, K), mx.QMat(N, K)
    out = torch.empty((M, N), dtype=torch.float32, device="cuda")
    with pytest.raises(mx.MxError) as e:
        mx.gemm_static(a, b, out, out_dtype=1)
    assert e.value.status == 4  # MXFP4_WORKSPACE_TOO_SMALL
