"""GPU parity of the MX quantizers against the CPU oracle: packed nibbles and scale bytes bit-exact."""
import numpy as np
import pytest
import torch

import oracle as orc
import workloads
from util import assert_qmat_equal, numpy_to_qmat, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


def rand_bf16(rng, shape, spread=2.0):
    x = rng.standard_normal(shape).astype(np.float32)
    x *= np.exp(rng.standard_normal((shape[0], 1)) * spread).astype(np.float32)
    return workloads.round_to_bf16(x)


SPECIALS = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, -0.25, -0.75, -1.25, -1.75, -2.5, -3.5, -5.0, -6.0]


@pytest.mark.parametrize("scale_mode", [0, 1])
@pytest.mark.parametrize("shape", [(300, 192), (1, 32), (129, 160), (1024, 192)])
def test_rowwise_rne(mx, scale_mode, shape):
    rng = np.random.default_rng(hash(shape) % 1000)
    x = rand_bf16(rng, shape)
    if shape[1] >= 32:
        x[0, :16] = SPECIALS  # all seven ties, both signs, with group max 6 -> scale 1
        if shape[0] > 3:
            x[1, :4] = [31, -31, 15.5, 8]
            x[2, :] = 0
            x[3, :3] = [-0.099609375, 6, -0.0]  # negative value that rounds to zero keeps its sign
    q = mx.quantize(to_dev_bf16(x), scale_mode=scale_mode)
    p, s, _ = orc.quantize(x, scale_mode=scale_mode)
    assert_qmat_equal(q, p, s, "rowwise rne")


@pytest.mark.parametrize("scale_mode", [0, 1])
def test_rowwise_sr(mx, scale_mode):
    rng = np.random.default_rng(2)
    x = rand_bf16(rng, (260, 256))
    x[0, :16] = SPECIALS
    seed = 0x123456789ABCDEF
    q = mx.quantize(to_dev_bf16(x), scale_mode=scale_mode, rounding=1, seed=seed, stream_id=3)
    p, s, _ = orc.quantize(x, scale_mode=scale_mode, rounding=1, seed=seed, stream_id=3)
    assert_qmat_equal(q, p, s, "rowwise sr")
    # another stream gives other codes, same scales
    q2 = mx.quantize(to_dev_bf16(x), scale_mode=scale_mode, rounding=1, seed=seed, stream_id=4)
    assert not torch.equal(q2.data, q.data)


def test_rowwise_strided_source(mx):
    rng = np.random.default_rng(3)
    x = rand_bf16(rng, (64, 256))
    xd = to_dev_bf16(x)[:, 64:192]  # ld = 256, cols = 128
    q = mx.quantize(xd, rounding=1, seed=4, stream_id=3)
    p, s, _ = orc.quantize(np.ascontiguousarray(x[:, 64:192]), rounding=1, seed=4, stream_id=3)
    assert_qmat_equal(q, p, s, "strided")


@pytest.mark.parametrize("rounding", [0, 1])
@pytest.mark.parametrize("shape", [(288, 160), (32, 32), (128, 64), (1024, 768)])
def test_transposed(mx, rounding, shape):
    rng = np.random.default_rng(5)
    x = rand_bf16(rng, shape)
    for sm in (0, 1):
        q = mx.quantize_t(to_dev_bf16(x), scale_mode=sm, rounding=rounding, seed=77, stream_id=5)
        p, s, _ = orc.quantize(x, transpose=True, scale_mode=sm, rounding=rounding, seed=77, stream_id=5)
        assert q.rows == shape[1] and q.cols == shape[0]
        assert_qmat_equal(q, p, s, "transposed")


def test_two_axis_equals_separate_quantizers(mx):
    rng = np.random.default_rng(6)
    x = rand_bf16(rng, (288, 192))
    q, qt = mx.quantize_2axis(to_dev_bf16(x), (0, 1, 9, 3), (0, 1, 9, 5))
    p, s, _ = orc.quantize(x, rounding=1, seed=9, stream_id=3)
    assert_qmat_equal(q, p, s, "2axis row")
    p, s, _ = orc.quantize(x, transpose=True, rounding=1, seed=9, stream_id=5)
    assert_qmat_equal(qt, p, s, "2axis transposed")
    q1 = mx.quantize(to_dev_bf16(x), rounding=1, seed=9, stream_id=3)
    assert torch.equal(q1.data, q.data) and torch.equal(q1.scales_linear(), q.scales_linear())


@pytest.mark.parametrize("rounding", [0, 1])
def test_chain_equals_quantize_then_double_quantization(mx, rounding):
    rng = np.random.default_rng(16)
    x = rand_bf16(rng, (288, 224))
    x[5, 3] = np.inf  # a non-finite group of the first quantizer must poison the column groups it touches
    for sm in (0, 1):
        q, qt = mx.quantize_chain(to_dev_bf16(x), seed=21, scale_mode=sm, rounding=rounding, stream_id=1)
        p1, s1, _ = orc.quantize(x, scale_mode=sm, rounding=rounding, seed=21, stream_id=1)
        assert_qmat_equal(q, p1, s1, "chain: first quantizer")
        p2, s2, _ = orc.quantize(orc.dequantize(p1, s1), transpose=True, scale_mode=sm, rounding=1, seed=21, stream_id=6)
        assert_qmat_equal(qt, p2, s2, "chain: double quantization")


def test_double_quantization_and_dequantize(mx):
    rng = np.random.default_rng(7)
    x = rand_bf16(rng, (160, 224))
    q1 = mx.quantize(to_dev_bf16(x))
    p1, s1, _ = orc.quantize(x)
    assert_qmat_equal(q1, p1, s1, "first quantizer")
    d = mx.dequantize(q1).cpu().numpy().astype(np.float64)
    assert (d == orc.dequantize(p1, s1)).all()
    for sm in (0, 1):
        q2 = mx.quantize_t(q1, scale_mode=sm, rounding=1, seed=5, stream_id=6)
        p2, s2, _ = orc.quantize(orc.dequantize(p1, s1), transpose=True, scale_mode=sm, rounding=1, seed=5, stream_id=6)
        assert_qmat_equal(q2, p2, s2, "double quantization")


@pytest.mark.parametrize("scale_mode", [0, 1])
def test_qema_with_fp32_ema_state(mx, scale_mode):
    rng = np.random.default_rng(8)
    w = workloads.round_to_bf16((rng.standard_normal((96, 192)) * 0.02).astype(np.float32))
    ema = (w + rng.standard_normal(w.shape).astype(np.float32) * 0.004).astype(np.float32)
    e_ref = ema.copy()
    e_gpu = torch.from_numpy(ema.copy()).cuda()
    for step in range(3):
        w = workloads.round_to_bf16(w + rng.standard_normal(w.shape).astype(np.float32) * 2e-5)
        q = mx.qema_quantize(to_dev_bf16(w), e_gpu, beta=0.998, update_ema=True, scale_mode=scale_mode)
        p, s = orc.qema_quantize(w, e_ref, beta=0.998, update_ema=True, scale_mode=scale_mode)
        assert_qmat_equal(q, p, s, "qema step %d" % step)
        assert (e_gpu.cpu().numpy().view(np.uint32) == e_ref.view(np.uint32)).all()
    # update_ema = 0 leaves the state alone and gives the same codes
    before = e_gpu.clone()
    q2 = mx.qema_quantize(to_dev_bf16(w), e_gpu, update_ema=False, scale_mode=scale_mode)
    assert torch.equal(before, e_gpu) and torch.equal(q2.data, q.data)


def test_qema_equals_plain_when_ema_is_w(mx):
    rng = np.random.default_rng(9)
    w = workloads.round_to_bf16((rng.standard_normal((128, 128)) * 0.02).astype(np.float32))
    w[0, :16] = np.array(SPECIALS, dtype=np.float32)
    wd = to_dev_bf16(w)
    q = mx.qema_quantize(wd, wd.float().contiguous(), update_ema=False)
    q0 = mx.quantize(wd)
    assert torch.equal(q.data, q0.data) and torch.equal(q.scales_linear(), q0.scales_linear())


def test_qema_oscillation_counters(mx):
    rng = np.random.default_rng(10)
    w0 = workloads.round_to_bf16((rng.standard_normal((64, 128)) * 0.02).astype(np.float32))
    ema_ref = w0.copy()
    ema_gpu = torch.from_numpy(w0.copy()).cuda()
    p, s, _ = orc.quantize(w0)
    wp, pp, sp = w0.copy(), p.copy(), s.copy()
    dw = np.zeros_like(w0)
    dq = np.zeros_like(w0)
    st = mx.OscState(to_dev_bf16(w0).clone(), numpy_to_qmat(mx, p, s), torch.zeros(w0.shape, device="cuda"),
                     torch.zeros(w0.shape, device="cuda"))
    w = w0
    for step in range(4):
        w = workloads.round_to_bf16(w + rng.standard_normal(w.shape).astype(np.float32) * 0.002)
        q = mx.qema_quantize(to_dev_bf16(w), ema_gpu, osc=st)
        p, s = orc.qema_quantize(w, ema_ref)
        orc.osc_update(w, p, s, wp, pp, sp, dw, dq)
        assert_qmat_equal(q, p, s, "qema under counters")
        assert_qmat_equal(st.wq_prev, pp, sp, "rolled previous codes")
        assert (st.dist_w.cpu().numpy().view(np.uint32) == dw.view(np.uint32)).all()
        assert (st.dist_q.cpu().numpy().view(np.uint32) == dq.view(np.uint32)).all()
        assert (st.w_prev.float().cpu().numpy() == wp).all()
    assert dq.max() > 0


def test_nonfinite_groups_flagged(mx):
    x = np.ones((128, 64), dtype=np.float32)
    x[5, 40] = np.inf
    x[7, 3] = np.nan
    st = mx.new_status()
    q = mx.quantize(to_dev_bf16(x), dev_status=st)
    p, s, nbad = orc.quantize(x)
    assert nbad == 2
    assert_qmat_equal(q, p, s, "nonfinite")
    assert int(st.item()) == mx.DEV_NONFINITE
    st = mx.new_status()
    qt = mx.quantize_t(to_dev_bf16(x), dev_status=st)
    p, s, _ = orc.quantize(x, transpose=True)
    assert_qmat_equal(qt, p, s, "nonfinite transposed")
    assert int(st.item()) == mx.DEV_NONFINITE


def test_extreme_exponents(mx):
    x = np.zeros((32, 32), dtype=np.float32)
    x[0, :3] = [float.fromhex("0x1.fep127"), 2.0 ** 127, 1]
    x[1, :2] = [2.0 ** -133, 2.0 ** -130]
    x[2, :3] = [2.0 ** -126, 2.0 ** -127, -(2.0 ** -120)]
    for sm in (0, 1):
        for rnd in (0, 1):
            q = mx.quantize(to_dev_bf16(x), scale_mode=sm, rounding=rnd, seed=1)
            p, s, _ = orc.quantize(x, scale_mode=sm, rounding=rnd, seed=1)
            assert_qmat_equal(q, p, s, "extreme exponents")
            qt = mx.quantize_t(to_dev_bf16(x), scale_mode=sm, rounding=rnd, seed=1)
            p, s, _ = orc.quantize(x, transpose=True, scale_mode=sm, rounding=rnd, seed=1)
            assert_qmat_equal(qt, p, s, "extreme exponents transposed")


def test_scale_padding_is_one(mx):
    x = to_dev_bf16(np.ones((32, 192), dtype=np.float32))
    q = mx.QMat(32, 192)
    q.scales.fill_(0xFF)
    mx.quantize(x, out=q)
    lin = q.scales_linear()
    used = torch.zeros_like(q.scales, dtype=torch.bool)
    for r in range(32):
        for b in range(6):
            used[mx.scale_offset(r, b, 192)] = True
    assert (q.scales[~used] == 0x7F).all() and (lin != 0xFF).all()


def test_argument_errors(mx):
    x = torch.zeros((32, 48), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mx.MxError) as e:
        mx.quantize(x, out=mx.QMat(32, 64))
    assert e.value.status == 2  # BAD_SHAPE: 48 is not a multiple of 32
    x = torch.zeros((48, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mx.MxError):
        mx.quantize_t(x)  # 48 rows cannot be grouped by 32
    x = torch.zeros((32, 72), dtype=torch.bfloat16, device="cuda")[:, 1:65]
    with pytest.raises(mx.MxError) as e:
        mx.quantize(x)
    assert e.value.status == 3  # MISALIGNED
    # empty input is fine
    mx.quantize(torch.zeros((0, 64), dtype=torch.bfloat16, device="cuda"))


@pytest.mark.parametrize("config,layer", [(1, 0), (2, 1)])
def test_config_tensors_all_quantizers(mx, config, layer):
    """The config's own X, W, dY (a 2048-row slab for config 2) through all six quantizers."""
    L, x, w, dy = workloads.make_layer(config, layer, rows=None if config == 1 else 2048)
    seed = workloads.sr_seed(config, layer)
    xq = mx.quantize(to_dev_bf16(x))
    wq = mx.quantize(to_dev_bf16(w))
    fx = orc.quantize(x)
    fw = orc.quantize(w)
    assert_qmat_equal(xq, fx[0], fx[1], "Q1")
    assert_qmat_equal(wq, fw[0], fw[1], "Q2")
    ops = orc.linear_bwd_operands(dy, fx[:2], fw[:2], seed)
    dyq, dyq_t = mx.quantize_2axis(to_dev_bf16(dy), (0, 1, seed, 3), (0, 1, seed, 5))
    assert_qmat_equal(dyq, *ops["dyq"], "Q3")
    assert_qmat_equal(dyq_t, *ops["dyq_t"], "Q5")
    assert_qmat_equal(mx.quantize_t(wq, rounding=1, seed=seed, stream_id=4), *ops["wq_t"], "Q4")
    assert_qmat_equal(mx.quantize_t(xq, rounding=1, seed=seed, stream_id=6), *ops["xq_t"], "Q6")
