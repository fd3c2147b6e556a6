"""The drain path of the bounded waits, exercised without any fault.

Every wait on a barrier in the GEMM kernels and in the two-axis quantizer gives up after a bounded number of polls,
raises MXFP4_DEV_TIMEOUT, and makes every role of its thread block leave; the block then frees its tensor memory and
returns.  The self-test entry points launch the real kernels with their loads withheld and the bound at a few
thousand polls, so that path runs within milliseconds: no trap, no endless loop, no bad address.  Afterwards the same
product (and quantizer) must run normally and match the oracle: the tensor memory was handed back and the context is
intact."""
import numpy as np
import pytest
import torch

import oracle as orc
from util import assert_qmat_equal, check_gemm_bound, numpy_to_qmat, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


def rand_operand(rng, rows, kc):
    c = rng.integers(0, 16, size=(rows, kc)).astype(np.uint8)
    p = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    s = rng.integers(122, 132, size=(rows, kc // 32)).astype(np.uint8)
    return p, s


# one shape per kernel of the product: one CTA per tile (128 wide), B-stationary, CTA pairs with split-K, cluster split-K,
# CTA pairs with the B block resident
@pytest.mark.parametrize("M,N,K", [(256, 128, 512), (256, 384, 512), (1024, 512, 2048), (1280, 768, 4096), (4864, 1536, 1024)])
@pytest.mark.parametrize("out_dtype", [0, 1])
def test_gemm_waits_run_out_and_the_kernel_drains(mx, M, N, K, out_dtype):
    rng = np.random.default_rng(M + N + K)
    pa, sa = rand_operand(rng, M, K)
    pb, sb = rand_operand(rng, N, K)
    a, b = numpy_to_qmat(mx, pa, sa), numpy_to_qmat(mx, pb, sb)
    st = mx.new_status()
    mx.gemm_wait_selftest(a, b, st, out_dtype=out_dtype, spin_limit=2048)
    torch.cuda.synchronize()
    assert int(st.item()) & mx.DEV_TIMEOUT, "the withheld loads must make a bounded wait run out"
    # the same kernels, now fed: tensor memory was freed and nothing is left over from the aborted launch
    st.zero_()
    for _ in range(2):
        d = mx.gemm(a, b, out_dtype=out_dtype, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    dref, tref = orc.gemm(pa, sa, pb, sb)
    check_gemm_bound(d.float().cpu().numpy(), dref, tref, bf16_out=(out_dtype == 0), what="gemm after the self-test")


def test_quantizer_waits_run_out_and_the_kernel_drains(mx):
    rng = np.random.default_rng(9)
    x = rng.standard_normal((384, 320)).astype(np.float32)
    x = torch.from_numpy(x).to(torch.bfloat16)
    xd = x.cuda()
    st = mx.new_status()
    mx.quantize_wait_selftest(xd, st, spin_limit=2048)
    torch.cuda.synchronize()
    assert int(st.item()) & mx.DEV_TIMEOUT
    st.zero_()
    q, qt = mx.quantize_2axis(xd, (0, 0, 0, 0), (0, 1, 77, 5), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    xf = x.float().numpy()
    assert_qmat_equal(q, *orc.quantize(xf)[:2], "row-wise after the self-test")
    assert_qmat_equal(qt, *orc.quantize(xf, transpose=True, rounding=1, seed=77, stream_id=5)[:2], "transposed after the self-test")


def test_selftest_argument_errors(mx):
    a, b = mx.QMat(128, 64), mx.QMat(128, 64)
    with pytest.raises(mx.MxError):
        mx.gemm_wait_selftest(a, b, mx.new_status(), spin_limit=4)          # below the allowed range
    with pytest.raises(mx.MxError):
        mx.gemm_wait_selftest(a, b, None)                                    # the status word is required
