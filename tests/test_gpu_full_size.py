"""Parity at the configurations' FULL sizes, in the launch configuration the benchmark times, on sampled outputs.

The oracle cannot redo 50432-token layers in seconds, so every check here is one it can compute by itself:
row-wise operands on sampled source rows, transposed operands on sampled 32-row groups x 32-column blocks (each slab
told where it sits, because stochastic rounding draws by position), products on sampled output rows x columns from the
operands the GPU itself produced (which the operand samples vouch for).  Bit-exact for codes and scales,
|err| <= 2^-20 * sum|a*b| for products.
"""
import numpy as np
import pytest
import torch

import oracle as orc
import workloads
from util import check_gemm_bound, numpy_to_qmat, qmat_to_numpy, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


def sample_rows(rng, n, k, align=1):
    """k distinct multiples of `align` below n, always with the first and the last."""
    cand = np.arange(0, n, align)
    pick = set(rng.choice(cand, size=min(k, len(cand)), replace=False).tolist()) | {0, int(cand[-1])}
    return np.array(sorted(pick))


def check_rowwise(q, src, rows, what, **kw):
    """Operand q = Q(src) with groups along columns, checked on the given source rows."""
    p, s = qmat_to_numpy(q)
    ncols = src.shape[1]
    for r in rows:
        pr, sr, _ = orc.quantize(np.ascontiguousarray(src[r:r + 1]), out_row0=int(r), out_ld=ncols, **kw)
        assert (s[r] == sr[0]).all(), "%s: scales of row %d differ" % (what, r)
        assert (p[r] == pr[0]).all(), "%s: codes of row %d differ" % (what, r)


def check_transposed(qt, src, rgroups, cblocks, what, **kw):
    """Operand qt = Q(src^T) (groups of 32 source rows), checked on 32-row groups x 32-column blocks of the source."""
    p, s = qmat_to_numpy(qt)
    nrows = src.shape[0]
    for r0 in rgroups:
        for c0 in cblocks:
            sub = np.ascontiguousarray(src[r0:r0 + 32, c0:c0 + 32])
            ps, ss, _ = orc.quantize(sub, transpose=True, out_row0=int(c0), out_col0=int(r0), out_ld=nrows, **kw)
            assert (s[c0:c0 + 32, r0 // 32] == ss[:, 0]).all(), "%s: scales at rows %d, cols %d differ" % (what, r0, c0)
            assert (p[c0:c0 + 32, r0 // 2:r0 // 2 + 16] == ps).all(), "%s: codes at rows %d, cols %d differ" % (what, r0, c0)


def check_product(d_gpu, a, b, rows, cols, bf16_out, what):
    """d_gpu[rows x cols] against the FP64 product of those rows of the (GPU-made) operands a [M, Kc], b [N, Kc]."""
    pa, sa = qmat_to_numpy(a)
    pb, sb = qmat_to_numpy(b)
    dref, tref = orc.gemm(pa[rows], sa[rows], pb[cols], sb[cols])
    got = d_gpu[torch.as_tensor(rows, device=d_gpu.device)][:, torch.as_tensor(cols, device=d_gpu.device)].float().cpu().numpy()
    check_gemm_bound(got, dref, tref, bf16_out, what)


def check_product_sampled(rng, d_gpu, a, b, bf16_out, what, full):
    """The whole product when the oracle can afford it (`full`: the DeiT-Small layers, about 30 GFLOP each); otherwise
    256 random rows x all columns, 64 random columns x all rows, and the first and the last 128 x 128 tile."""
    m, n = a.rows, b.rows
    all_r, all_c = np.arange(m), np.arange(n)
    if full:
        check_product(d_gpu, a, b, all_r, all_c, bf16_out, what + " (all)")
        return
    check_product(d_gpu, a, b, sample_rows(rng, m, 256), all_c, bf16_out, what + " (256 rows x all columns)")
    check_product(d_gpu, a, b, all_r, sample_rows(rng, n, 64), bf16_out, what + " (all rows x 64 columns)")
    check_product(d_gpu, a, b, all_r[:128], all_c[:128], bf16_out, what + " (first tile)")
    check_product(d_gpu, a, b, all_r[-128:], all_c[-128:], bf16_out, what + " (last tile)")


LAYERS = [(2, 0), (2, 1), (3, 0), (3, 1), (4, 0), (4, 1), (5, 0), (5, 1), (5, 2), (5, 3), (6, 0), (6, 2), (6, 3), (6, 4)]


@pytest.mark.parametrize("config,layer", LAYERS)
def test_full_size_layer(mx, config, layer):
    L, x, w, dy = workloads.make_layer(config, layer)
    M, K, N = L.M, L.K, L.N
    seed = workloads.sr_seed(config, layer)
    rng = np.random.default_rng(100 * config + layer)
    st = mx.new_status()
    xd, wd, dyd = to_dev_bf16(x), to_dev_bf16(w), to_dev_bf16(dy)

    # ---- the step as the benchmark runs it: weight quantizer, forward (Q1 + Q6 in one pass), backward ----
    if L.qema:
        hist, ema0 = workloads.make_ema(L, w, workloads.tensor_seed(config, layer, "W"), steps=2)
        ema_ref, ema_gpu = ema0.copy(), torch.from_numpy(ema0.copy()).cuda()
        p0, s0, _ = orc.quantize(w)
        prev = dict(w=w.copy(), p=p0.copy(), s=s0.copy(), dw=np.zeros_like(w), dq=np.zeros_like(w))
        osc = mx.OscState(wd.clone(), numpy_to_qmat(mx, p0, s0), torch.zeros(w.shape, device="cuda"), torch.zeros(w.shape, device="cuda"))
        for wt in hist:
            wq = mx.qema_quantize(to_dev_bf16(wt), ema_gpu, beta=0.998, osc=osc, dev_status=st)
            pw, sw = orc.qema_quantize(wt, ema_ref, beta=0.998)
            orc.osc_update(wt, pw, sw, prev["w"], prev["p"], prev["s"], prev["dw"], prev["dq"])
        gp, gs = qmat_to_numpy(wq)
        assert (gp == pw).all() and (gs == sw).all(), "Q-EMA weight"
        assert (ema_gpu.cpu().numpy().view(np.uint32) == ema_ref.view(np.uint32)).all(), "EMA state"
        assert (osc.dist_w.cpu().numpy().view(np.uint32) == prev["dw"].view(np.uint32)).all(), "dist_W"
        assert (osc.dist_q.cpu().numpy().view(np.uint32) == prev["dq"].view(np.uint32)).all(), "dist_Q"
        y, ctx = mx.linear_fwd(xd, wq=wq, dev_status=st, bwd_seed=seed)
    else:
        y, ctx = mx.linear_fwd(xd, wd, dev_status=st, bwd_seed=seed)
        pw, sw, _ = orc.quantize(w)
        gp, gs = qmat_to_numpy(ctx.wq)
        assert (gp == pw).all() and (gs == sw).all(), "Q2(W)"
    dx, dw = mx.linear_bwd(dyd, ctx, seed, dev_status=st)
    # the backward operands once more through the quantizer entry points (the backward pass keeps its own in scratch)
    dyq, dyq_t = mx.quantize_2axis(dyd, (0, 1, seed, 3), (0, 1, seed, 5), dev_status=st)
    wq_t = mx.quantize_t(ctx.wq, rounding=1, seed=seed, stream_id=4, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0

    # ---- operands on samples ----
    rows = sample_rows(rng, M, 24)
    rgroups = sample_rows(rng, M, 6, align=32)
    check_rowwise(ctx.xq, x, rows, "Q1(X)")
    check_rowwise(dyq, dy, rows, "Q3(dY)", rounding=1, seed=seed, stream_id=3)
    check_transposed(dyq_t, dy, rgroups, sample_rows(rng, N, 4, align=32), "Q5(dY^T)", rounding=1, seed=seed, stream_id=5)
    # Q6 re-quantizes the dequantized Q1(X): dequantize the GPU's Q1 rows of the sampled groups with the oracle
    xp, xs = qmat_to_numpy(ctx.xq)
    for r0 in rgroups:
        xdeq = orc.dequantize(xp[r0:r0 + 32], xs[r0:r0 + 32])
        pt, s_t = qmat_to_numpy(ctx.xq_t)
        for c0 in sample_rows(rng, K, 3, align=32):
            sub = np.ascontiguousarray(xdeq[:, c0:c0 + 32])
            ps, ss, _ = orc.quantize(sub, transpose=True, rounding=1, seed=seed, stream_id=6, out_row0=int(c0), out_col0=int(r0), out_ld=M)
            assert (s_t[c0:c0 + 32, r0 // 32] == ss[:, 0]).all() and (pt[c0:c0 + 32, r0 // 2:r0 // 2 + 16] == ps).all(), "Q6"
    p4, s4, _ = orc.quantize(orc.dequantize(pw, sw), transpose=True, rounding=1, seed=seed, stream_id=4)
    g4p, g4s = qmat_to_numpy(wq_t)
    assert (g4p == p4).all() and (g4s == s4).all(), "Q4"

    # ---- products: everything for the DeiT-Small layers, large samples (with the first and the last tile) for the rest ----
    full = config in (2, 5)
    check_product_sampled(rng, y, ctx.xq, ctx.wq, True, "Y", full)
    check_product_sampled(rng, dx, dyq, wq_t, True, "dX", full)
    check_product_sampled(rng, dw, dyq_t, ctx.xq_t, False, "dW", full)


def test_full_size_fused_epilogues_config4(mx):
    """The quantizing epilogue at the largest workload: fc1's forward product with GELU and the Q1 / Q6 chain of fc2's
    input behind it, and fc2's input-gradient product with the multiplication and Q3 / Q5 of fc1's output gradient.
    Sampled rows and groups against the oracle (on the bf16 tensors the kernel emitted), everything against the
    stand-alone quantizers on the GPU, which the other tests hold against the oracle."""
    import math
    L1, x, w1, _ = workloads.make_layer(4, 0)
    L2, _, w2, dy2 = workloads.make_layer(4, 1)
    M, N1 = L1.M, L1.N
    s1, s2 = workloads.sr_seed(4, 0), workloads.sr_seed(4, 1)
    rng = np.random.default_rng(44)
    st = mx.new_status()
    xq, wq1 = mx.quantize(to_dev_bf16(x), dev_status=st), mx.quantize(to_dev_bf16(w1), dev_status=st)
    y1 = torch.empty((M, N1), dtype=torch.bfloat16, device="cuda")
    z1 = torch.empty((M, N1), dtype=torch.bfloat16, device="cuda")
    epi = mx.Epilogue(hook=mx.HOOK_GELU, y=y1, z=z1, zq=mx.QMat(M, N1), qp_row=(0, 0, 0, 0), zq_t=mx.QMat(N1, M), qp_t=(0, 1, s2, 6), chain=True)
    mx.gemm_quant(xq, wq1, epi, dev_status=st)
    q, qt = mx.quantize_chain(z1, seed=s2, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert torch.equal(epi.zq.data, q.data) and torch.equal(epi.zq.scales, q.scales), "Q1 of fc2's input"
    assert torch.equal(epi.zq_t.data, qt.data) and torch.equal(epi.zq_t.scales, qt.scales), "Q6 of fc2's input"
    rows = sample_rows(rng, M, 48)
    check_product(y1, xq, wq1, rows, np.arange(N1), True, "Y1 (48 rows x all columns)")
    yf = y1[torch.as_tensor(rows, device="cuda")].float().cpu().numpy().astype(np.float64)
    zf = z1[torch.as_tensor(rows, device="cuda")].float().cpu().numpy().astype(np.float64)
    g = 0.5 * yf * (1.0 + np.vectorize(math.erf)(yf / math.sqrt(2.0)))
    assert (np.abs(zf - g) <= np.abs(g) * 2.0 ** -8 + np.abs(yf) * 2.0 ** -20).all(), "Z1 = bf16(GELU(Y1))"
    z1h = z1.float().cpu().numpy()
    check_rowwise(epi.zq, z1h, rows[:24], "Q1(Z1)")
    zp, zs = qmat_to_numpy(epi.zq)
    pt, s_t = qmat_to_numpy(epi.zq_t)
    for r0 in sample_rows(rng, M, 5, align=32):
        zdeq = orc.dequantize(zp[r0:r0 + 32], zs[r0:r0 + 32])
        for c0 in sample_rows(rng, N1, 3, align=32):
            ps, ss, _ = orc.quantize(np.ascontiguousarray(zdeq[:, c0:c0 + 32]), transpose=True, rounding=1, seed=s2, stream_id=6,
                                     out_row0=int(c0), out_col0=int(r0), out_ld=M)
            assert (s_t[c0:c0 + 32, r0 // 32] == ss[:, 0]).all() and (pt[c0:c0 + 32, r0 // 2:r0 // 2 + 16] == ps).all(), "Q6(Z1)"
    del y1, z1, epi, q, qt, z1h, zp, zs, pt, s_t

    # ---- backward: dZ = Q3(dY2) Q4(W2), dY1 = dZ * g', Q3 / Q5 of dY1 from the epilogue ----
    wq2 = mx.quantize(to_dev_bf16(w2), dev_status=st)
    dyq2 = mx.quantize(to_dev_bf16(dy2), rounding=1, seed=s2, stream_id=3, dev_status=st)
    wq2_t = mx.quantize_t(wq2, rounding=1, seed=s2, stream_id=4, dev_status=st)
    gprime = workloads.round_to_bf16(rng.uniform(-0.15, 1.1, size=(M, N1)).astype(np.float32))
    dz = torch.empty((M, N1), dtype=torch.bfloat16, device="cuda")
    dy1 = torch.empty((M, N1), dtype=torch.bfloat16, device="cuda")
    epi = mx.Epilogue(hook=mx.HOOK_MULTIPLY, aux=to_dev_bf16(gprime), y=dz, z=dy1, zq=mx.QMat(M, N1), qp_row=(0, 1, s1, 3),
                      zq_t=mx.QMat(N1, M), qp_t=(0, 1, s1, 5))
    mx.gemm_quant(dyq2, wq2_t, epi, dev_status=st)
    q, qt = mx.quantize_2axis(dy1, (0, 1, s1, 3), (0, 1, s1, 5), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert torch.equal(epi.zq.data, q.data) and torch.equal(epi.zq.scales, q.scales), "Q3 of fc1's output gradient"
    assert torch.equal(epi.zq_t.data, qt.data) and torch.equal(epi.zq_t.scales, qt.scales), "Q5 of fc1's output gradient"
    check_product(dz, dyq2, wq2_t, rows, np.arange(N1), True, "dZ (48 rows x all columns)")
    dzf = dz.float().cpu().numpy()
    want = workloads.round_to_bf16(dzf * gprime)
    assert (dy1.float().cpu().numpy().view(np.uint32) == want.view(np.uint32)).all(), "dY1 = bf16(dZ * g')"
    check_rowwise(epi.zq, want, rows[:24], "Q3(dY1)", rounding=1, seed=s1, stream_id=3)
    check_transposed(epi.zq_t, want, sample_rows(rng, M, 5, align=32), sample_rows(rng, N1, 3, align=32), "Q5(dY1^T)", rounding=1, seed=s1, stream_id=5)
