"""The fifth workload: one DeiT-Small block training step around the library's linear layers (attention, LayerNorm,
GELU and residuals in PyTorch bf16), with the Q-EMA weight quantizer and the oscillation counters on all four linear
layers.  Every linear layer's captured (X, W, dY) is replayed through the CPU oracle: operands bit-exact, EMA and
counters bit-exact, products within the bound."""
import numpy as np
import pytest
import torch

import oracle as orc
from util import check_gemm_bound, qmat_to_numpy

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


def f32(t):
    return t.detach().float().cpu().numpy()


def replay_layer(layer, before, full):
    """One linear layer of the step against the oracle.  `before`: host copies of the layer's state before the step."""
    rec = layer.record
    w = f32(layer.w)
    # ---- weight side: Q-EMA with its EMA update, counters ----
    ema = before["ema"].copy()
    pw, sw = orc.qema_quantize(w, ema, beta=layer.beta)
    gp, gs = qmat_to_numpy(layer.wq)
    assert (gp == pw).all() and (gs == sw).all(), layer.name + ": Q-EMA weight"
    assert (layer.ema.cpu().numpy().view(np.uint32) == ema.view(np.uint32)).all(), layer.name + ": EMA state"
    prev = {k: v.copy() for k, v in before.items() if k != "ema"}
    orc.osc_update(w, pw, sw, prev["w_prev"], prev["p_prev"], prev["s_prev"], prev["dist_w"], prev["dist_q"])
    assert (layer.osc.dist_w.cpu().numpy().view(np.uint32) == prev["dist_w"].view(np.uint32)).all(), layer.name + ": dist_W"
    assert (layer.osc.dist_q.cpu().numpy().view(np.uint32) == prev["dist_q"].view(np.uint32)).all(), layer.name + ": dist_Q"
    # ---- activations: on all rows, or on a sample of 32-row groups at full size ----
    x, dy = f32(rec["x"]), f32(rec["dy"])
    M = x.shape[0]
    rng = np.random.default_rng(M + layer.N)
    groups = np.arange(M // 32) if full else np.sort(rng.choice(M // 32, size=24, replace=False))
    rows = (groups[:, None] * 32 + np.arange(32)[None, :]).reshape(-1)
    xp, xs = qmat_to_numpy(rec["ctx"].xq)
    for r0 in groups[:: max(1, len(groups) // 8)] * 32:
        pr, sr, _ = orc.quantize(np.ascontiguousarray(x[r0:r0 + 32]))
        assert (xp[r0:r0 + 32] == pr).all() and (xs[r0:r0 + 32] == sr).all(), layer.name + ": Q1(X)"
    # products from the oracle's own operands of the sampled rows
    xq = orc.quantize(np.ascontiguousarray(x[rows]))[:2]
    yref, ty = orc.gemm(*xq, pw, sw)
    check_gemm_bound(f32(rec["y"])[rows], yref, ty, True, layer.name + ": Y")
    # dX rows depend on the same rows of dY only (Q3 groups run along N): slab quantization at the rows' positions
    N = layer.N
    dyq_p = np.zeros((len(rows), N // 2), np.uint8)
    dyq_s = np.zeros((len(rows), N // 32), np.uint8)
    for i, g in enumerate(groups):
        p, s, _ = orc.quantize(np.ascontiguousarray(dy[g * 32:g * 32 + 32]), rounding=1, seed=layer.seed, stream_id=3, out_row0=int(g) * 32, out_ld=N)
        dyq_p[i * 32:(i + 1) * 32], dyq_s[i * 32:(i + 1) * 32] = p, s
    wq_t = orc.quantize(orc.dequantize(pw, sw), transpose=True, rounding=1, seed=layer.seed, stream_id=4)[:2]
    dxref, tdx = orc.gemm(dyq_p, dyq_s, *wq_t)
    check_gemm_bound(f32(rec["dx"])[rows], dxref, tdx, True, layer.name + ": dX")
    if full:
        b = orc.linear_bwd(dy, orc.quantize(x)[:2], (pw, sw), layer.seed)
        check_gemm_bound(rec["dw"].cpu().numpy(), b["dw"], b["tdw"], False, layer.name + ": dW")


@pytest.mark.parametrize("batch,full", [(32, True), (128, False)])
def test_block_step_replayed_through_the_oracle(mx, batch, full):
    from workloads import block_harness as bh
    blk = bh.Block(mx)
    x, dout = bh.make_block_inputs(batch)
    blk.weight_step()                 # a first step fills the "previous" buffers of the counters
    blk.perturb_weights(seed=77)      # the weights move, the EMA lags behind
    before = {}
    for name, layer in blk.layers.items():
        p_prev, s_prev = qmat_to_numpy(layer.osc.wq_prev)
        before[name] = dict(ema=layer.ema.cpu().numpy().copy(), w_prev=f32(layer.osc.w_prev), p_prev=p_prev.copy(), s_prev=s_prev.copy(),
                            dist_w=layer.osc.dist_w.cpu().numpy().copy(), dist_q=layer.osc.dist_q.cpu().numpy().copy())
    out, dx = blk.step(x, dout)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all() and torch.isfinite(dx.float()).all()
    for name, layer in blk.layers.items():
        assert int(layer.status.item()) == 0, name
        replay_layer(layer, before[name], full)
    if not full:
        # the weight gradient of one layer in full at full size as well (its contraction runs over all 25216 tokens)
        layer = blk.layers["proj"]
        rec = layer.record
        pw, sw = qmat_to_numpy(layer.wq)
        b = orc.linear_bwd(f32(rec["dy"]), orc.quantize(f32(rec["x"]))[:2], (pw, sw), layer.seed)
        check_gemm_bound(rec["dw"].cpu().numpy(), b["dw"], b["tdw"], False, "proj: dW at full size")
