"""GPU parity of the whole quantized linear layer (Eq. 3-5) through mxfp4_linear_fwd / mxfp4_linear_bwd."""
import numpy as np
import pytest
import torch

import oracle as orc
import workloads
from util import assert_qmat_equal, check_gemm_bound, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


@pytest.mark.parametrize("config,layer,rows", [(1, 0, None), (2, 0, 2048), (2, 1, 2048), (3, 1, 1024), (5, 0, 1024),
                                               (6, 0, 1568), (6, 1, 1568), (6, 2, 1568), (6, 3, 800), (6, 4, 288)])
@pytest.mark.parametrize("scale_mode", [0, 1])
def test_linear_fwd_bwd(mx, config, layer, rows, scale_mode):
    if scale_mode == 1 and config != 1:
        pytest.skip("floor scaling is covered on config 1")
    L, x, w, dy = workloads.make_layer(config, layer, rows=rows)
    seed = workloads.sr_seed(config, layer)
    st = mx.new_status()
    y, ctx = mx.linear_fwd(to_dev_bf16(x), to_dev_bf16(w), scale_mode=scale_mode, dev_status=st)
    dx, dw = mx.linear_bwd(to_dev_bf16(dy), ctx, seed, scale_mode=scale_mode, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    f = orc.linear_fwd(x, w, scale_mode=scale_mode)
    b = orc.linear_bwd(dy, f["xq"], f["wq"], seed, scale_mode=scale_mode)
    assert_qmat_equal(ctx.xq, *f["xq"], "Q1(X)")
    assert_qmat_equal(ctx.wq, *f["wq"], "Q2(W)")
    check_gemm_bound(y.float().cpu().numpy(), f["y"], f["t"], True, "Y")
    check_gemm_bound(dx.float().cpu().numpy(), b["dx"], b["tdx"], True, "dX")
    check_gemm_bound(dw.cpu().numpy(), b["dw"], b["tdw"], False, "dW")


@pytest.mark.parametrize("config,layer,rows", [(1, 0, None), (2, 1, 1024), (5, 3, 512)])
def test_linear_fwd_makes_q6_for_the_backward_pass(mx, config, layer, rows):
    """With the backward seed known at forward time, one kernel emits Q1(X) and Q6 = Q(deq(Q1(X))^T); the backward pass
    then skips its own double-quantization pass over Q1(X).  Every operand and result is the same as without it."""
    L, x, w, dy = workloads.make_layer(config, layer, rows=rows)
    seed = workloads.sr_seed(config, layer)
    st = mx.new_status()
    y, ctx = mx.linear_fwd(to_dev_bf16(x), to_dev_bf16(w), dev_status=st, bwd_seed=seed)
    dx, dw = mx.linear_bwd(to_dev_bf16(dy), ctx, seed, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    f = orc.linear_fwd(x, w)
    b = orc.linear_bwd(dy, f["xq"], f["wq"], seed)
    assert_qmat_equal(ctx.xq, *f["xq"], "Q1(X)")
    assert_qmat_equal(ctx.xq_t, *b["xq_t"], "Q6 made by the forward pass")
    check_gemm_bound(y.float().cpu().numpy(), f["y"], f["t"], True, "Y")
    check_gemm_bound(dx.float().cpu().numpy(), b["dx"], b["tdx"], True, "dX")
    check_gemm_bound(dw.cpu().numpy(), b["dw"], b["tdw"], False, "dW")
    # another seed at backward time: the stored Q6 is not used, the pass is redone
    dx2, dw2 = mx.linear_bwd(to_dev_bf16(dy), ctx, seed + 1)
    b2 = orc.linear_bwd(dy, f["xq"], f["wq"], seed + 1)
    check_gemm_bound(dw2.cpu().numpy(), b2["dw"], b2["tdw"], False, "dW, other seed")


@pytest.mark.parametrize("config,layer,rows", [(1, 0, None), (2, 0, 1024), (6, 0, 800)])
def test_linear_bwd_takes_q4_made_ahead(mx, config, layer, rows):
    """Q4 = Q(deq(Q2(W))^T) depends on the weight and the seed only, so a caller may make it ahead (on another stream,
    once per optimizer step) and hand it over in the context: operands and results equal the oracle's all the same."""
    L, x, w, dy = workloads.make_layer(config, layer, rows=rows)
    seed = workloads.sr_seed(config, layer)
    st = mx.new_status()
    y, ctx = mx.linear_fwd(to_dev_bf16(x), to_dev_bf16(w), dev_status=st, bwd_seed=seed)
    ctx.wq_t = mx.quantize_t(ctx.wq, rounding=1, seed=seed, stream_id=4, dev_status=st)
    dx, dw = mx.linear_bwd(to_dev_bf16(dy), ctx, seed, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    f = orc.linear_fwd(x, w)
    b = orc.linear_bwd(dy, f["xq"], f["wq"], seed)
    assert_qmat_equal(ctx.wq_t, *b["wq_t"], "Q4")
    check_gemm_bound(dx.float().cpu().numpy(), b["dx"], b["tdx"], True, "dX")
    check_gemm_bound(dw.cpu().numpy(), b["dw"], b["tdw"], False, "dW")
    # a context made for another seed is not used: the backward pass makes its own Q4
    dx2, dw2 = mx.linear_bwd(to_dev_bf16(dy), ctx, seed + 1, dev_status=st)
    b2 = orc.linear_bwd(dy, f["xq"], f["wq"], seed + 1)
    check_gemm_bound(dx2.float().cpu().numpy(), b2["dx"], b2["tdx"], True, "dX, other seed")


@pytest.mark.parametrize("config,layer,rows", [(1, 0, None), (2, 1, 640)])
def test_linear_fwd_makes_q4_with_q2_when_given_the_weight(mx, config, layer, rows):
    """With the weight itself and a buffer for Q4 in the context, the forward pass makes Q2 and Q4 in one pass over W
    (as it makes Q1 and Q6 in one pass over X); the backward pass with the same seed then uses both."""
    L, x, w, dy = workloads.make_layer(config, layer, rows=rows)
    seed = workloads.sr_seed(config, layer)
    st = mx.new_status()
    ctx = mx.LinearCtx(mx.QMat(L.M if rows is None else rows, L.K), mx.QMat(L.N, L.K), xq_t=mx.QMat(L.K, L.M if rows is None else rows),
                       seed=seed, wq_t=mx.QMat(L.K, L.N))
    ctx.wq_t.data.fill_(0x5A)       # whatever was there is overwritten
    y, ctx = mx.linear_fwd(to_dev_bf16(x), to_dev_bf16(w), ctx=ctx, dev_status=st, bwd_seed=seed)
    dx, dw = mx.linear_bwd(to_dev_bf16(dy), ctx, seed, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    f = orc.linear_fwd(x, w)
    b = orc.linear_bwd(dy, f["xq"], f["wq"], seed)
    assert_qmat_equal(ctx.wq, *f["wq"], "Q2(W)")
    assert_qmat_equal(ctx.wq_t, *b["wq_t"], "Q4 made by the forward pass")
    check_gemm_bound(y.float().cpu().numpy(), f["y"], f["t"], True, "Y")
    check_gemm_bound(dx.float().cpu().numpy(), b["dx"], b["tdx"], True, "dX")
    check_gemm_bound(dw.cpu().numpy(), b["dw"], b["tdw"], False, "dW")


def test_linear_with_qema_weight_and_bias(mx):
    L, x, w, dy = workloads.make_layer(2, 0, rows=512)
    hist, ema0 = workloads.make_ema(L, w, workloads.tensor_seed(2, 0, "W"))
    ema_ref = ema0.copy()
    ema_gpu = torch.from_numpy(ema0.copy()).cuda()
    for wt in hist:
        wq = mx.qema_quantize(to_dev_bf16(wt), ema_gpu, beta=0.998)
        f = orc.linear_fwd(x, wt, ema=ema_ref, beta=0.998)
    assert_qmat_equal(wq, *f["wq"], "Q-EMA weight")
    assert (ema_gpu.cpu().numpy().view(np.uint32) == ema_ref.view(np.uint32)).all()
    rng = np.random.default_rng(0)
    bias = workloads.round_to_bf16(rng.standard_normal(L.N).astype(np.float32) * 0.1)
    y, ctx = mx.linear_fwd(to_dev_bf16(x), wq=wq, bias=to_dev_bf16(bias.reshape(1, -1)).reshape(-1))
    yref = f["y"] + bias
    tol = f["t"] * 2.0 ** -20
    lo = workloads.round_to_bf16((yref - tol - np.abs(yref) * 2.0 ** -22).astype(np.float32))
    hi = workloads.round_to_bf16((yref + tol + np.abs(yref) * 2.0 ** -22).astype(np.float32))
    yg = y.float().cpu().numpy()
    assert ((yg >= np.minimum(lo, yref - tol)) & (yg <= np.maximum(hi, yref + tol))).all()
    # backward uses the forward operand that was actually used (the Q-EMA weight)
    seed = 11
    dx, dw = mx.linear_bwd(to_dev_bf16(dy), ctx, seed)
    b = orc.linear_bwd(dy, f["xq"], f["wq"], seed)
    check_gemm_bound(dx.float().cpu().numpy(), b["dx"], b["tdx"], True, "dX")
    check_gemm_bound(dw.cpu().numpy(), b["dw"], b["tdw"], False, "dW")


def test_linear_bwd_workspace_check(mx):
    x = torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    y, ctx = mx.linear_fwd(x, w)
    with pytest.raises(mx.MxError) as e:
        mx.linear_bwd(torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda"), ctx, 0,
                      workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4


@pytest.mark.parametrize("M,K,N", [(512, 4096, 1024), (256, 8192, 384)])
def test_linear_fwd_small_batch_long_contraction(mx, M, K, N):
    """Few output tiles and a long contraction: mxfp4_gemm would split K through a workspace here; the forward pass has
    none and must run the product unsplit (and say so before anything is enqueued, not after its quantizers)."""
    assert mx.gemm_workspace_bytes(M, N, K) > 0
    rng = np.random.default_rng(M + K + N)
    x = workloads.round_to_bf16(rng.standard_normal((M, K)).astype(np.float32))
    w = workloads.round_to_bf16((rng.standard_normal((N, K)) * 0.02).astype(np.float32))
    st = mx.new_status()
    y, ctx = mx.linear_fwd(to_dev_bf16(x), to_dev_bf16(w), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    f = orc.linear_fwd(x, w)
    assert_qmat_equal(ctx.xq, *f["xq"], "Q1(X)")
    assert_qmat_equal(ctx.wq, *f["wq"], "Q2(W)")
    check_gemm_bound(y.float().cpu().numpy(), f["y"], f["t"], True, "Y")


def test_linear_errors_leave_the_stream_untouched(mx):
    """An argument error is reported before the first launch: the context's buffers keep their contents."""
    x = torch.ones((128, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.ones((64, 64), dtype=torch.bfloat16, device="cuda")
    ctx = mx.LinearCtx(mx.QMat(128, 64), mx.QMat(64, 64))
    ctx.xq.data.fill_(0xAB)
    y = torch.empty((128, 72), dtype=torch.bfloat16, device="cuda")[:, 4:68]   # 8-byte aligned rows: misaligned output
    with pytest.raises(mx.MxError) as e:
        mx.linear_fwd(x, w, ctx=ctx, out=y)
    assert e.value.status == 3
    torch.cuda.synchronize()
    assert (ctx.xq.data == 0xAB).all()


def test_mlp_pair_with_the_quantizations_fused_into_the_products(mx):
    """fc1 -> GELU -> fc2 forward and backward with every quantization at the layer boundary done by the neighbouring
    product's epilogue: fc1's forward product emits Q1 / Q6 of fc2's input, fc2's input-gradient product multiplies by
    the activation's derivative and emits Q3 / Q5 of fc1's output gradient.  Operands are held against the oracle's
    quantizers applied to the bf16 tensors the kernels emitted, products against the FP64 oracle of those operands."""
    rows = 1024
    L1, x, w1, _ = workloads.make_layer(2, 0, rows=rows)
    L2, _, w2, dy2 = workloads.make_layer(2, 1, rows=rows)
    s1, s2 = workloads.sr_seed(2, 0), workloads.sr_seed(2, 1)
    M, K1, N1, N2 = rows, L1.K, L1.N, L2.N
    rng = np.random.default_rng(3)
    gprime = workloads.round_to_bf16(rng.uniform(-0.15, 1.1, size=(M, N1)).astype(np.float32))   # stands in for GELU'(Y1)
    st = mx.new_status()
    # ---- forward ----
    ctx2 = mx.LinearCtx(mx.QMat(M, N1), mx.QMat(N2, N1), xq_t=mx.QMat(N1, M), seed=s2)
    y1 = torch.empty((M, N1), dtype=torch.bfloat16, device="cuda")
    z1 = torch.empty((M, N1), dtype=torch.bfloat16, device="cuda")
    epi = mx.Epilogue(hook=mx.HOOK_GELU, y=y1, z=z1, zq=ctx2.xq, qp_row=(0, 0, 0, 0), zq_t=ctx2.xq_t, qp_t=(0, 1, s2, 6), chain=True)
    _, ctx1 = mx.linear_fwd(to_dev_bf16(x), to_dev_bf16(w1), dev_status=st, bwd_seed=s1, epi=epi)
    y2, _ = mx.linear_fwd(None, to_dev_bf16(w2), ctx=ctx2, dev_status=st)
    # ---- backward ----
    ws1 = torch.empty(mx.linear_workspace_bytes(M, K1, N1), dtype=torch.uint8, device="cuda")
    dyq1, dyq1_t = mx.QMat(M, N1), mx.QMat(N1, M)
    dy1 = torch.empty((M, N1), dtype=torch.bfloat16, device="cuda")
    epi_dx = mx.Epilogue(hook=mx.HOOK_MULTIPLY, aux=to_dev_bf16(gprime), z=dy1, zq=dyq1, qp_row=(0, 1, s1, 3), zq_t=dyq1_t, qp_t=(0, 1, s1, 5))
    _, dw2 = mx.linear_bwd(to_dev_bf16(dy2), ctx2, s2, dev_status=st, epi_dx=epi_dx)
    dx1, dw1 = mx.linear_bwd(None, ctx1, s1, dev_status=st, workspace=ws1, dyq=dyq1, dyq_t=dyq1_t)
    torch.cuda.synchronize()
    assert int(st.item()) == 0

    f1 = orc.linear_fwd(x, w1)
    assert_qmat_equal(ctx1.xq, *f1["xq"], "Q1(X)")
    check_gemm_bound(y1.float().cpu().numpy(), f1["y"], f1["t"], True, "Y1")
    z1f = z1.float().cpu().numpy()
    xq2 = orc.quantize(z1f)[:2]
    assert_qmat_equal(ctx2.xq, *xq2, "Q1 of fc2's input, made by fc1's epilogue")
    wq2 = orc.quantize(w2)[:2]
    y2ref, t2 = orc.gemm(*xq2, *wq2)
    check_gemm_bound(y2.float().cpu().numpy(), y2ref, t2, True, "Y2")
    b2 = orc.linear_bwd(dy2, xq2, wq2, s2)
    assert_qmat_equal(ctx2.xq_t, *b2["xq_t"], "Q6 of fc2's input, made by fc1's epilogue")
    check_gemm_bound(dw2.cpu().numpy(), b2["dw"], b2["tdw"], False, "dW2")
    dy1f = dy1.float().cpu().numpy()
    # dY1 = bf16(bf16(dZ) * GELU'): bf16(dZ) is not stored; dZ * g within the product's bound and two roundings
    want = b2["dx"] * gprime
    tol = b2["tdx"] * 2.0 ** -20 * np.abs(gprime) + np.abs(want) * 2.0 ** -7
    assert (np.abs(dy1f - want) <= tol).all(), "dY1 = dZ * GELU'(Y1)"
    b1 = orc.linear_bwd(dy1f, f1["xq"], f1["wq"], s1)
    assert_qmat_equal(dyq1, *b1["dyq"], "Q3 of fc1's output gradient, made by fc2's epilogue")
    assert_qmat_equal(dyq1_t, *b1["dyq_t"], "Q5 of fc1's output gradient, made by fc2's epilogue")
    check_gemm_bound(dx1.float().cpu().numpy(), b1["dx"], b1["tdx"], True, "dX1")
    check_gemm_bound(dw1.cpu().numpy(), b1["dw"], b1["tdw"], False, "dW1")
