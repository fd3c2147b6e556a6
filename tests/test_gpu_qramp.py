"""GPU parity of the Q-Ramping entry points (Sec. 6, Algorithm 2) against the CPU oracle.

The ramp factor is an integer decided by two FP32 quotients that both sides take in FP32: bit-exact.  The optimizer
step is FP32 arithmetic with every operation rounded once; the oracle takes the same step in FP64 from the GPU's own
FP32 state, so one step's difference is a few FP32 roundings: the update n lr (m^/(sqrt(v^) + eps) + wd w) goes through
about ten of them and the bias corrections are rounded to FP32 once more (|w' - w'_ref| <= ulp + 16 * 2^-24 |w' - w|
plus what the moments' own differences contribute to first order: m can cancel almost completely), the moments are within
8 * 2^-24 relative to the larger of their two summands."""
import numpy as np
import pytest
import torch

import oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    import paper_2502_20853_b200 as m
    m.lib()
    assert torch.cuda.is_available()
    return m


def make_trajectories(rng, n):
    """Trajectory lengths with the structure of Sec. 6.1: most elements move alike (ratio near 1), some oscillate
    (quantized value flips by a grid step while the master weight barely moves), some never moved."""
    dist_w = rng.gamma(2.0, 1e-3, n).astype(np.float32)
    ratio = np.where(rng.random(n) < 0.08, rng.uniform(10.0, 400.0, n), rng.uniform(0.0, 3.0, n))
    dist_q = (dist_w * ratio).astype(np.float32)
    still = rng.random(n) < 0.01
    dist_w[still] = 0.0
    dist_q[still & (rng.random(n) < 0.5)] = 0.0
    return dist_w, dist_q


@pytest.mark.parametrize("n,k1,k2,n_max", [(4096 * 1024, 16.0, 5, 255), (1000003, 16.0, 5, 20), (1000003, 12.0, 4, 255),
                                           (7, 0.75, 3, 255), (0, 16.0, 5, 255)])
def test_detect_matches_oracle(mx, n, k1, k2, n_max):
    rng = np.random.default_rng(n % 9973 + k2)
    dist_w, dist_q = make_trajectories(rng, n)
    ref, osc_ref = orc.qramp_detect(dist_w, dist_q, k1, k2, n_max)
    n_w, osc = mx.qramp_detect(torch.from_numpy(dist_w).cuda(), torch.from_numpy(dist_q).cuda(), k1, k2, n_max)
    torch.cuda.synchronize()
    assert (n_w.cpu().numpy() == ref).all()
    assert int(osc.item()) == osc_ref


def test_detect_edge_values(mx):
    dist_w = np.array([1.0, 1.0, 1.0, 0.5, 0.0, 0.0, np.nan, 1.0, np.inf, 1.0], dtype=np.float32)
    dist_q = np.array([15.99, 16.0, 1e9, 16.0, 1.0, 0.0, 1.0, np.inf, 1.0, np.nan], dtype=np.float32)
    ref, osc_ref = orc.qramp_detect(dist_w, dist_q, 16.0, 5, 100)
    n_w, osc = mx.qramp_detect(torch.from_numpy(dist_w).cuda(), torch.from_numpy(dist_q).cuda(), 16.0, 5, 100)
    assert n_w.cpu().numpy().tolist() == ref.tolist()
    assert int(osc.item()) == osc_ref


def test_detect_argument_errors(mx):
    d = torch.zeros(64, device="cuda")
    for kw in (dict(k1=0.0), dict(k2=0), dict(n_max=0), dict(n_max=256)):
        with pytest.raises(mx.MxError):
            mx.qramp_detect(d, d, **kw)
    with pytest.raises(mx.MxError):
        mx.qramp_detect(d[1:], d[1:])      # not 16-byte aligned


def ulp32(x):
    return np.spacing(np.abs(x).astype(np.float32)).astype(np.float64)


@pytest.mark.parametrize("n,ramped", [(768 * 192 + 3, True), (4096 * 1024, True), (5, False)])
def test_adamw_steps_match_oracle(mx, n, ramped):
    rng = np.random.default_rng(n % 1009)
    # hyper-parameters that FP32 holds exactly, so that both sides compute with the same numbers
    hp = {k: float(np.float32(v)) for k, v in dict(lr=2e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.05).items()}
    w = rng.normal(0, 0.02, n).astype(np.float32)
    if ramped:
        n_w = rng.choice(np.array([1, 1, 1, 1, 2, 6, 11], dtype=np.uint8), size=n)
    else:
        n_w = None
    dev = lambda a: torch.from_numpy(a.copy()).cuda()  # noqa: E731
    W, M, V, A = dev(w), dev(np.zeros(n, np.float32)), dev(np.zeros(n, np.float32)), dev(np.zeros(n, np.float32))
    Cn = torch.zeros(n, dtype=torch.uint8, device="cuda")
    Wb = dev(w).to(torch.bfloat16)
    NW = None if n_w is None else torch.from_numpy(n_w).cuda()
    moved_total = 0
    for step in range(1, 13):
        g = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
        # the oracle starts every step from the GPU's own FP32 state
        w64, m64, v64, a64 = (t.cpu().numpy().astype(np.float64) for t in (W, M, V, A))
        c8 = Cn.cpu().numpy().copy()
        w_before, wb_before = w64.copy(), Wb.float().cpu().numpy()
        m_before, v_before = m64.copy(), v64.copy()
        upd = orc.qramp_adamw(w64, g.astype(np.float64), m64, v64, a64, c8, n_w, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                              hp["weight_decay"], step=step)
        mx.qramp_adamw(W, dev(g), M, V, A, Cn, NW, step=step, w_bf16=Wb, **hp)
        torch.cuda.synchronize()
        gw, gm, gv, ga = (t.cpu().numpy().astype(np.float64) for t in (W, M, V, A))
        assert (Cn.cpu().numpy() == c8).all(), "accumulation counters"
        moved = w64 != w_before
        assert int(moved.sum()) <= upd
        moved_total += upd
        assert (np.abs(ga - a64) <= ulp32(a64)).all(), "accumulator"
        gbar = np.where(c8 == 0, 1.0, 0.0)    # elements whose window closed this step
        tol_m = 8 * 2.0 ** -24 * np.maximum(np.abs(hp["beta1"] * m_before), np.abs(m64 - hp["beta1"] * m_before)) + 1e-45
        tol_v = 8 * 2.0 ** -24 * np.maximum(np.abs(hp["beta2"] * v_before), np.abs(v64 - hp["beta2"] * v_before)) + 1e-45
        assert (np.abs(gm - m64) <= tol_m).all(), "first moment"
        assert (np.abs(gv - v64) <= tol_v).all(), "second moment"
        # the weight: its own rounding, the roundings of the update, and the moments' differences carried through
        # d(update)/dm = 1 / (c1 (sqrt(v^) + eps)),  d(update)/dv = -m^ / (2 c2 sqrt(v^) (sqrt(v^) + eps)^2)
        c1, c2 = 1.0 - hp["beta1"] ** step, 1.0 - hp["beta2"] ** step
        root = np.sqrt(v64 / c2)
        carried = tol_m / c1 / (root + hp["eps"]) + np.abs(m64 / c1) * (tol_v / c2) / (2 * np.maximum(root, 1e-30) * (root + hp["eps"]) ** 2)
        ramp = 1.0 if n_w is None else n_w.astype(np.float64)
        tol_w = (ulp32(np.maximum(np.abs(w_before), np.abs(w64))) + 16 * 2.0 ** -24 * np.abs(w64 - w_before)
                 + np.where(c8 == 0, ramp * hp["lr"] * carried, 0.0))
        assert (np.abs(gw - w64) <= tol_w).all(), "weight"
        # the bf16 copy is the rounding of the GPU's own FP32 weight where it changed and untouched elsewhere
        wb = Wb.float().cpu().numpy()
        closed = gbar == 1.0
        assert (wb[closed] == W.to(torch.bfloat16).float().cpu().numpy()[closed]).all()
        assert (wb[~closed] == wb_before[~closed]).all()
    assert moved_total > 0
