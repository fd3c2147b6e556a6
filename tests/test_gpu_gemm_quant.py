"""GPU parity of the product with the fused quantizing epilogue (mxfp4_gemm_quant).

The bf16 tile the kernel emits is held against the FP64 oracle product within the product's bound; the codes and
scales it emits are held, bit for bit, against the oracle's quantizers applied to THAT bf16 tile (the quantization
comes after the cast, so it cannot be pinned to the FP64 product itself)."""
import math

import numpy as np
import pytest
import torch

import oracle as orc
import workloads
from util import assert_qmat_equal, check_gemm_bound, numpy_to_qmat, qmat_to_numpy, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


def rand_operand(rng, rows, kc, lo=123, hi=131):
    c = rng.integers(0, 16, size=(rows, kc)).astype(np.uint8)
    p = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    s = rng.integers(lo, hi, size=(rows, kc // 32)).astype(np.uint8)
    return p, s


def operands(mx, M, N, K, seed):
    rng = np.random.default_rng(seed)
    pa, sa = rand_operand(rng, M, K)
    pb, sb = rand_operand(rng, N, K)
    return (pa, sa, pb, sb), numpy_to_qmat(mx, pa, sa), numpy_to_qmat(mx, pb, sb)


def bf16_tensor(M, N, pad=0):
    """[M, N] bf16 view of a wider buffer filled with a sentinel, to see writes beyond N."""
    big = torch.full((M, N + pad), 7.0, dtype=torch.bfloat16, device="cuda")
    return big, big[:, :N]


# one tile, several tiles, ragged in M and N (multiples of 32 only), short and long contractions
SHAPES = [(128, 128, 64), (256, 256, 512), (384, 320, 192), (160, 96, 64), (1024, 768, 1536), (512, 1152, 384)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("mode", ["2axis_sr", "chain", "rne_rne", "row_only", "t_only"])
def test_quantizing_epilogue_identity(mx, M, N, K, mode):
    ops, a, b = operands(mx, M, N, K, M + 3 * N + K)
    st = mx.new_status()
    big, z = bf16_tensor(M, N, 64)
    seed = 0xABC0 + M
    qp_row = {"2axis_sr": (0, 1, seed, 3), "chain": (0, 0, 0, 0), "rne_rne": (0, 0, 0, 0), "row_only": (0, 1, seed, 3), "t_only": None}[mode]
    qp_t = {"2axis_sr": (0, 1, seed, 5), "chain": (0, 1, seed, 6), "rne_rne": (1, 0, 0, 0), "row_only": None, "t_only": (0, 1, seed, 5)}[mode]
    epi = mx.Epilogue(z=z, zq=mx.QMat(M, N) if qp_row else None, qp_row=qp_row or (0, 0, 0, 0),
                      zq_t=mx.QMat(N, M) if qp_t else None, qp_t=qp_t or (0, 0, 0, 0), chain=(mode == "chain"))
    mx.gemm_quant(a, b, epi, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert (big[:, N:] == 7.0).all()
    zf = z.float().cpu().numpy()
    dref, tref = orc.gemm(*ops)
    check_gemm_bound(zf, dref, tref, True, "Z")
    if qp_row:
        pr, sr, _ = orc.quantize(zf, scale_mode=qp_row[0], rounding=qp_row[1], seed=qp_row[2], stream_id=qp_row[3])
        assert_qmat_equal(epi.zq, pr, sr, "row-wise codes of Z")
    if qp_t:
        src = orc.dequantize(pr, sr) if mode == "chain" else zf
        pt, s_t, _ = orc.quantize(src, transpose=True, scale_mode=qp_t[0], rounding=qp_t[1], seed=qp_t[2], stream_id=qp_t[3])
        assert_qmat_equal(epi.zq_t, pt, s_t, "transposed codes of Z")


def test_quantizing_epilogue_gelu_with_bias_keeps_y(mx):
    M, N, K = 384, 640, 256
    ops, a, b = operands(mx, M, N, K, 5)
    rng = np.random.default_rng(6)
    bias = workloads.round_to_bf16((rng.standard_normal(N) * 2).astype(np.float32))
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    z = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    seed = 99
    epi = mx.Epilogue(hook=mx.HOOK_GELU, y=y, z=z, zq=mx.QMat(M, N), qp_row=(0, 0, 0, 0), zq_t=mx.QMat(N, M), qp_t=(0, 1, seed, 6), chain=True)
    st = mx.new_status()
    mx.gemm_quant(a, b, epi, bias=to_dev_bf16(bias.reshape(1, -1)).reshape(-1), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    dref, tref = orc.gemm(*ops)
    yf = y.float().cpu().numpy().astype(np.float64)
    want = dref + bias
    tol = tref * 2.0 ** -20 + np.abs(want) * 2.0 ** -23
    lo = np.minimum(workloads.round_to_bf16((want - tol).astype(np.float32)), want - tol)
    hi = np.maximum(workloads.round_to_bf16((want + tol).astype(np.float32)), want + tol)
    assert ((yf >= lo) & (yf <= hi)).all(), "Y = bf16(product + bias)"
    # Z = bf16(GELU(Y)): the FP32 evaluation (absolute error below 1e-6 |y|) may land on the neighbouring bf16 value
    erf = np.vectorize(math.erf)
    g = 0.5 * yf * (1.0 + erf(yf / math.sqrt(2.0)))
    zf = z.float().cpu().numpy().astype(np.float64)
    assert (np.abs(zf - g) <= np.abs(g) * 2.0 ** -8 + np.abs(yf) * 2.0 ** -20).all(), "Z = bf16(GELU(Y))"
    pr, sr, _ = orc.quantize(zf.astype(np.float32))
    assert_qmat_equal(epi.zq, pr, sr, "Q1 of the next layer")
    pt, s_t, _ = orc.quantize(orc.dequantize(pr, sr), transpose=True, rounding=1, seed=seed, stream_id=6)
    assert_qmat_equal(epi.zq_t, pt, s_t, "Q6 of the next layer")


def test_quantizing_epilogue_multiply_is_exact(mx):
    """dX times the derivative of the activation, then Q3 / Q5 of the previous layer: the product of two bf16 values is
    exact in FP32, so Z = bf16(Y * aux) is reproducible bit for bit from the Y the kernel emitted."""
    M, N, K = 512, 384, 1536
    ops, a, b = operands(mx, M, N, K, 7)
    rng = np.random.default_rng(8)
    aux = workloads.round_to_bf16(rng.uniform(-0.2, 1.1, size=(M, N)).astype(np.float32))
    auxd = to_dev_bf16(aux)
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    z = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    seed = 1234
    epi = mx.Epilogue(hook=mx.HOOK_MULTIPLY, aux=auxd, y=y, z=z, zq=mx.QMat(M, N), qp_row=(0, 1, seed, 3), zq_t=mx.QMat(N, M), qp_t=(0, 1, seed, 5))
    st = mx.new_status()
    mx.gemm_quant(a, b, epi, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    dref, tref = orc.gemm(*ops)
    yf = y.float().cpu().numpy()
    check_gemm_bound(yf, dref, tref, True, "Y")
    zref = workloads.round_to_bf16(yf * aux)          # float32 product of bf16 values: exact, then one rounding
    zf = z.float().cpu().numpy()
    assert (zf.view(np.uint32) == zref.view(np.uint32)).all(), "Z = bf16(Y * aux)"
    assert_qmat_equal(epi.zq, *orc.quantize(zf, rounding=1, seed=seed, stream_id=3)[:2], "Q3")
    assert_qmat_equal(epi.zq_t, *orc.quantize(zf, transpose=True, rounding=1, seed=seed, stream_id=5)[:2], "Q5")


def test_quantizing_epilogue_equals_the_standalone_quantizers(mx):
    """At a size the oracle would take long on: the fused results against mxfp4_quantize_chain / _2axis on the same Z."""
    M, N, K = 4096, 1536, 384
    g = torch.Generator(device="cuda").manual_seed(3)
    a, b = mx.QMat(M, K), mx.QMat(N, K)
    for q in (a, b):
        q.data.copy_(torch.randint(0, 256, q.data.shape, dtype=torch.uint8, device="cuda", generator=g))
        q.scales.copy_(torch.randint(124, 130, q.scales.shape, dtype=torch.uint8, device="cuda", generator=g))
    seed = 4242
    for chain, qp_row, qp_t in ((True, (0, 0, 0, 0), (0, 1, seed, 6)), (False, (0, 1, seed, 3), (0, 1, seed, 5))):
        z = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        epi = mx.Epilogue(z=z, zq=mx.QMat(M, N), qp_row=qp_row, zq_t=mx.QMat(N, M), qp_t=qp_t, chain=chain)
        mx.gemm_quant(a, b, epi)
        assert torch.equal(z, mx.gemm(a, b)), "the bf16 tile equals the plain product's"
        if chain:
            q, qt = mx.quantize_chain(z, seed=seed)
        else:
            q, qt = mx.quantize_2axis(z, qp_row, qp_t)
        assert torch.equal(epi.zq.data, q.data) and torch.equal(epi.zq.scales, q.scales)
        assert torch.equal(epi.zq_t.data, qt.data) and torch.equal(epi.zq_t.scales, qt.scales)


def test_gemm_quant_argument_errors(mx):
    a, b = mx.QMat(128, 64), mx.QMat(128, 64)
    with pytest.raises(mx.MxError) as e:
        mx.gemm_quant(a, b, mx.Epilogue())                       # nothing asked for
    assert e.value.status == 1
    with pytest.raises(mx.MxError) as e:
        mx.gemm_quant(a, b, mx.Epilogue(zq=mx.QMat(128, 128), chain=True))   # a chain needs both results
    assert e.value.status == 1
    with pytest.raises(mx.MxError) as e:
        mx.gemm_quant(a, mx.QMat(72, 64), mx.Epilogue(zq=mx.QMat(128, 72)))  # N must be a multiple of 32
    assert e.value.status == 2
