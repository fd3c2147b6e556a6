"""GPU parity of the block-scaled MXFP4 GEMM: |err| <= 2^-20 * sum|a*b| against the FP64 oracle product."""
import numpy as np
import pytest
import torch

import oracle as orc
import workloads
from util import check_gemm_bound, numpy_to_qmat, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


def rand_operand(rng, rows, kc, lo=118, hi=136):
    c = rng.integers(0, 16, size=(rows, kc)).astype(np.uint8)
    p = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    s = rng.integers(lo, hi, size=(rows, kc // 32)).astype(np.uint8)
    return p, s


def run_gemm(mx, pa, sa, pb, sb, out_dtype, bias=None):
    a, b = numpy_to_qmat(mx, pa, sa), numpy_to_qmat(mx, pb, sb)
    st = mx.new_status()
    d = mx.gemm(a, b, out_dtype=out_dtype, bias=bias, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return d.float().cpu().numpy()


# single tile, several tiles, ragged M/N/K tails, K = 192 (6 scale blocks padded to 8), wide tiles, split-K,
SHAPES = [(128, 128, 64), (128, 128, 256), (256, 256, 512), (1024, 768, 192), (1024, 192, 768), (768, 192, 1024),
          (384, 1536, 192), (160, 200, 320), (96, 8, 32), (512, 512, 4096), (640, 384, 8192), (256, 128, 6400),
          # CTA pairs adding their halves of the contraction through distributed shared memory: ragged in M, N and K
          (1280, 768, 4096), (1200, 760, 4352),
          # CTA pairs walking down columns of 256 x 192 tiles with the B block resident (3 or 4 K tiles, at least 2048 rows
          # and at least as many pair tiles as SMs): about one tile per pair; an odd number of row tiles with ragged N (a last
          # column of 8) and K; several tiles per pair; K = 3 tiles + 32 with many short columns; one tall column
          (4864, 1536, 1024), (4224, 1736, 960), (8320, 1536, 768), (2080, 3600, 800), (38400, 192, 1024),
          # the same contraction lengths with too few tiles for that kernel
          (2304, 768, 1024), (2080, 200, 800)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("out_dtype", [0, 1])
def test_gemm_random_codes_and_scales(mx, M, N, K, out_dtype):
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    pa, sa = rand_operand(rng, M, K)
    pb, sb = rand_operand(rng, N, K)
    d = run_gemm(mx, pa, sa, pb, sb, out_dtype)
    dref, tref = orc.gemm(pa, sa, pb, sb)
    check_gemm_bound(d, dref, tref, bf16_out=(out_dtype == 0), what="gemm %dx%dx%d" % (M, N, K))


def test_gemm_small_integers_exact(mx):
    rng = np.random.default_rng(1)
    M, N, K = 256, 384, 512
    ca = (rng.integers(0, 3, size=(M, K)) * 2).astype(np.uint8) | (rng.integers(0, 2, size=(M, K)) * 8).astype(np.uint8)
    cb = (rng.integers(0, 3, size=(N, K)) * 2).astype(np.uint8)
    pa = (ca[:, 0::2] | (ca[:, 1::2] << 4)).astype(np.uint8)
    pb = (cb[:, 0::2] | (cb[:, 1::2] << 4)).astype(np.uint8)
    sa = np.full((M, K // 32), 127, np.uint8)
    sb = np.full((N, K // 32), 127, np.uint8)
    d = run_gemm(mx, pa, sa, pb, sb, 1)
    ia = (ca & 7).astype(np.int64) // 2 * np.where(ca & 8, -1, 1)
    ib = (cb & 7).astype(np.int64) // 2
    assert (d == (ia @ ib.T)).all()


def test_gemm_one_hot_pins_scale_layout_and_nibble_order(mx):
    """A single non-zero element per operand, moved over rows / K positions: reads back exactly one
    (code, scale) pair of each operand, so any mismatch in the scale tiling or nibble order shows."""
    M, N, K = 256, 256, 512
    rng = np.random.default_rng(2)
    sa = rng.integers(100, 150, size=(M, K // 32)).astype(np.uint8)
    sb = rng.integers(100, 150, size=(N, K // 32)).astype(np.uint8)
    for (i, j, k) in [(0, 0, 0), (1, 2, 33), (37, 130, 71), (129, 255, 300), (255, 31, 511), (64, 65, 255)]:
        pa = np.zeros((M, K // 2), np.uint8)
        pb = np.zeros((N, K // 2), np.uint8)
        pa[i, k // 2] = 5 << (4 * (k & 1))  # 3.0
        pb[j, k // 2] = 0xB << (4 * (k & 1))  # -1.5
        d = run_gemm(mx, pa, sa, pb, sb, 1)
        want = 3.0 * 2.0 ** (int(sa[i, k // 32]) - 127) * -1.5 * 2.0 ** (int(sb[j, k // 32]) - 127)
        assert d[i, j] == np.float32(want)
        d[i, j] = 0
        assert (d == 0).all()


# Contractions that stay in ONE accumulator for more than 16 MMAs (no split-K, no second accumulator): the pair kernel
# with 64- and 32-MMA chains, the 192-wide kernel with 24, a 128-MMA chain, and the cluster kernel's two 64-MMA chains.
LONG_CHAINS = [(2048, 2048, 4096), (2048, 2048, 2048), (2048, 384, 1536), (4096, 1024, 8192), (1024, 1024, 16384)]


@pytest.mark.parametrize("M,N,K", LONG_CHAINS)
@pytest.mark.parametrize("out_dtype", [0, 1])
def test_gemm_long_accumulation_chains(mx, M, N, K, out_dtype):
    """The tensor core adds every MMA's 64-term sum into its FP32 accumulator with truncation: up to one ulp of the
    running sum is lost per MMA, so the bound grows with the chain: |err| <= max(1, chain / 8) * 2^-20 * sum|a*b|
    (the header's statement).  Operands with 18-binade-wide random scales and little cancellation make the drift show
    (measured 2.4 x 2^-20 at chains of 64 and 128); sampled rows keep the FP64 product affordable."""
    chain = mx.gemm_chain_mmas(M, N, K)
    assert chain > 16
    rng = np.random.default_rng(M + N + K)
    pa, sa = rand_operand(rng, M, K)
    pb, sb = rand_operand(rng, N, K)
    d = run_gemm(mx, pa, sa, pb, sb, out_dtype)
    rows = np.sort(rng.choice(M, size=192, replace=False))
    rows[0], rows[-1] = 0, M - 1
    dref, tref = orc.gemm(pa[rows], sa[rows], pb, sb)
    check_gemm_bound(d[rows], dref, tref, bf16_out=(out_dtype == 0), what="gemm %dx%dx%d chain %d" % (M, N, K, chain),
                     factor=max(1.0, chain / 8.0))


def test_gemm_chain_query(mx):
    assert mx.gemm_chain_mmas(128, 128, 64) == 1 and mx.gemm_chain_mmas(128, 128, 96) == 2
    assert mx.gemm_chain_mmas(25216, 1536, 384) == 6
    assert mx.gemm_chain_mmas(50432, 1024, 4096) == 64            # one accumulator per tile, no split
    assert mx.gemm_chain_mmas(512, 512, 4096) == 16               # four splits of four K tiles
    assert mx.gemm_chain_mmas(0, 128, 64) == 0


def _bias_case(mx, M, N, K, out_dtype, static=False):
    rng = np.random.default_rng(M + 3 * N + K + out_dtype)
    pa, sa = rand_operand(rng, M, K, 125, 130)
    pb, sb = rand_operand(rng, N, K, 125, 130)
    bias = workloads.round_to_bf16(rng.standard_normal(N).astype(np.float32) * 4.0)
    a, b = numpy_to_qmat(mx, pa, sa), numpy_to_qmat(mx, pb, sb)
    dt = torch.float32 if out_dtype == 1 else torch.bfloat16
    big = torch.full((M, N + 64), 7.0, dtype=dt, device="cuda")
    out = big[:, :N]
    bias_dev = to_dev_bf16(bias.reshape(1, -1)).reshape(-1)
    st = mx.new_status()
    if static:
        mx.gemm_static(a, b, out, out_dtype=out_dtype, bias=bias_dev, dev_status=st)
    else:
        mx.gemm(a, b, out_dtype=out_dtype, bias=bias_dev, out=out, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    dref, tref = orc.gemm(pa, sa, pb, sb)
    want = dref + bias
    tol = tref * 2.0 ** -20 + np.abs(want) * 2.0 ** -23 + np.abs(bias) * 2.0 ** -23    # the product's bound + the FP32 add of the bias
    d = out.float().cpu().numpy().astype(np.float64)
    if out_dtype == 1:
        assert (np.abs(d - want) <= tol).all()
    else:
        lo = np.minimum(workloads.round_to_bf16((want - tol).astype(np.float32)).astype(np.float64), want - tol)
        hi = np.maximum(workloads.round_to_bf16((want + tol).astype(np.float32)).astype(np.float64), want + tol)
        assert ((d >= lo) & (d <= hi)).all()
    assert (big[:, N:] == 7.0).all()  # nothing written beyond N


# every path that adds the bias: the single-kernel epilogue (fp32 boxes; bf16 through the 64-column boxes), the 192-wide
# B-stationary kernel, the pair kernel, the split-K reduction, the cluster split-K epilogue
BIAS_SHAPES = [(256, 192, 256), (512, 512, 512), (1024, 384, 384), (4096, 1536, 2048), (640, 384, 8192), (1280, 768, 4096),
               (4224, 1736, 960)]


@pytest.mark.parametrize("M,N,K", BIAS_SHAPES)
@pytest.mark.parametrize("out_dtype", [0, 1])
def test_gemm_bias_and_strided_output(mx, M, N, K, out_dtype):
    _bias_case(mx, M, N, K, out_dtype)


def test_gemm_argument_errors(mx):
    a, b = mx.QMat(128, 64), mx.QMat(128, 96)
    with pytest.raises(mx.MxError) as e:
        mx.gemm(a, b)
    assert e.value.status == 2
    a, b = mx.QMat(128, 6400), mx.QMat(128, 6400)
    out = torch.empty((128, 128), dtype=torch.float32, device="cuda")
    assert mx.gemm_workspace_bytes(128, 128, 6400) > 0
    with pytest.raises(mx.MxError) as e:
        mx.gemm(a, b, out_dtype=1, out=out, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4  # WORKSPACE_TOO_SMALL


@pytest.mark.parametrize("config,layer,rows", [(1, 0, None), (2, 0, 1024), (4, 1, 512)])
def test_config_products(mx, config, layer, rows):
    """Eq. 3-5 on the config's tensors: operands from the GPU quantizers (checked bit-exact elsewhere),
    products against the FP64 oracle of those same operands."""
    L, x, w, dy = workloads.make_layer(config, layer, rows=rows)
    seed = workloads.sr_seed(config, layer)
    f = orc.linear_fwd(x, w)
    b = orc.linear_bwd(dy, f["xq"], f["wq"], seed)
    xq, wq = numpy_to_qmat(mx, *f["xq"]), numpy_to_qmat(mx, *f["wq"])
    y = mx.gemm(xq, wq, out_dtype=0).float().cpu().numpy()
    check_gemm_bound(y, f["y"], f["t"], True, "Y")
    dx = mx.gemm(numpy_to_qmat(mx, *b["dyq"]), numpy_to_qmat(mx, *b["wq_t"]), out_dtype=0).float().cpu().numpy()
    check_gemm_bound(dx, b["dx"], b["tdx"], True, "dX")
    dw = mx.gemm(numpy_to_qmat(mx, *b["dyq_t"]), numpy_to_qmat(mx, *b["xq_t"]), out_dtype=1).cpu().numpy()
    check_gemm_bound(dw, b["dw"], b["tdw"], False, "dW")


def test_mma_issue_ceiling_loop_runs(mx):
    """The measurement aid: an MMA-only loop on every SM.  It must finish with a clean status and a rate that is at
    least what the GEMM kernels reach (they cannot be faster than the pipe they run on)."""
    for bn in (128, 192, 256):
        rate = mx.mma_issue_ceiling(bn=bn, iters=500, reps=2)
        assert rate > 2000.0, (bn, rate)
    with pytest.raises(mx.MxError):
        mx.mma_issue_ceiling(bn=64)
