"""Pins of the Q-Ramping oracle (Sec. 6, Algorithm 2) against things other than itself: values worked by hand from the
algorithm's two assignments, and torch.optim.AdamW (a library routine) for the update rule."""
import numpy as np
import pytest
import torch

import oracle as orc


def test_detect_hand_worked_values():
    # Algorithm 2 with the paper's defaults k1 = 16, k2 = 5:  n_w = min(5 * floor(R_w / 16) + 1, N_max), R_w = dist_Q / dist_W
    dist_w = np.array([1.0, 1.0, 1.0, 1.0, 0.5, 2.0, 1.0, 0.25], dtype=np.float32)
    dist_q = np.array([0.0, 15.99, 16.0, 31.9, 16.0, 16.0, 160.0, 100.0], dtype=np.float32)
    #  R_w             0     15.99  16     31.9  32    8     160     400
    #  floor(R/16)     0     0      1      1     2     0     10      25
    n_w, osc = orc.qramp_detect(dist_w, dist_q, k1=16.0, k2=5, n_max=255)
    assert n_w.tolist() == [1, 1, 6, 6, 11, 1, 51, 126]
    # "oscillating weights": R_w > 16 (Sec. 7.2) -> 31.9, 32, 160, 400
    assert osc == 4


def test_detect_clamp_and_degenerate_trajectories():
    dist_w = np.array([1.0, 0.0, 0.0, 1e-30, np.nan], dtype=np.float32)
    dist_q = np.array([1e6, 1.0, 0.0, 1.0, 1.0], dtype=np.float32)
    n_w, osc = orc.qramp_detect(dist_w, dist_q, k1=16.0, k2=5, n_max=20)
    # huge ratio: clamped at N_max; a weight that never moved while its quantized value did: N_max; nothing moved: 1;
    # a NaN ratio leaves the element alone
    assert n_w.tolist() == [20, 20, 1, 20, 1]
    assert osc == 3


def test_detect_is_monotone_in_the_ratio():
    rng = np.random.default_rng(5)
    dw = rng.uniform(0.1, 2.0, 4096).astype(np.float32)
    dq = (dw * rng.uniform(0.0, 200.0, 4096)).astype(np.float32)
    n_w, _ = orc.qramp_detect(dw, dq, 16.0, 5, 255)
    order = np.argsort(dq / dw, kind="stable")
    assert (np.diff(n_w[order].astype(int)) >= 0).all()
    assert set(np.unique((n_w.astype(int) - 1) % 5)) == {0}      # n_w - 1 is a multiple of k2


def _torch_adamw(w0, grads, lr, b1, b2, eps, wd):
    p = torch.nn.Parameter(torch.tensor(w0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    traj = []
    for g in grads:
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        traj.append(p.detach().numpy().copy())
    return traj


def test_adamw_with_unit_ramp_is_adamw():
    """n_w = 1 for every element: the customized AdamW is torch.optim.AdamW, step by step."""
    rng = np.random.default_rng(11)
    n, steps = 257, 6
    w = rng.normal(0, 0.02, n)
    grads = [rng.standard_t(3, n) * 1e-3 for _ in range(steps)]
    hp = dict(lr=3e-3, b1=0.9, b2=0.95, eps=1e-8, wd=0.05)
    ref = _torch_adamw(w, grads, **hp)
    m, v, acc, cnt = np.zeros(n), np.zeros(n), np.zeros(n), np.zeros(n, dtype=np.uint8)
    wq = w.copy()
    for t, g in enumerate(grads, start=1):
        upd = orc.qramp_adamw(wq, g.copy(), m, v, acc, cnt, None, hp["lr"], hp["b1"], hp["b2"], hp["eps"], hp["wd"], step=t)
        assert upd == n
        np.testing.assert_allclose(wq, ref[t - 1], rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("ramp", [2, 5])
def test_adamw_ramped_element_takes_mean_gradient_and_scaled_learning_rate(ramp):
    """An element with factor n accumulates n gradients and then takes ONE AdamW step with their mean and n times the
    learning rate (LR_w = n LR, BS_w = n BS in Algorithm 2); in between it does not move."""
    rng = np.random.default_rng(13 + ramp)
    n = 64
    w = rng.normal(0, 0.02, n)
    grads = [rng.normal(0, 1e-3, n) for _ in range(ramp)]
    hp = dict(lr=1e-3, b1=0.9, b2=0.999, eps=1e-8, wd=0.1)
    ref = _torch_adamw(w, [np.mean(grads, axis=0)], lr=hp["lr"] * ramp, b1=hp["b1"], b2=hp["b2"], eps=hp["eps"], wd=hp["wd"])[0]
    m, v, acc, cnt = np.zeros(n), np.zeros(n), np.zeros(n), np.zeros(n, dtype=np.uint8)
    wq, n_w = w.copy(), np.full(n, ramp, dtype=np.uint8)
    for t, g in enumerate(grads, start=1):
        # torch's single step uses the bias correction of ITS first step: hand the oracle the same one
        upd = orc.qramp_adamw(wq, g.copy(), m, v, acc, cnt, n_w, hp["lr"], hp["b1"], hp["b2"], hp["eps"], hp["wd"], step=1)
        if t < ramp:
            assert upd == 0 and (wq == w).all() and (cnt == t).all()
    assert upd == n and (cnt == 0).all() and (acc == 0).all()
    np.testing.assert_allclose(wq, ref, rtol=1e-12, atol=1e-15)


def test_adamw_mixed_ramps_update_on_their_own_schedule():
    n_w = np.array([1, 2, 3, 4], dtype=np.uint8)
    w, m, v, acc, cnt = np.ones(4), np.zeros(4), np.zeros(4), np.zeros(4), np.zeros(4, dtype=np.uint8)
    updates = []
    for t in range(1, 13):
        before = w.copy()
        orc.qramp_adamw(w, np.full(4, 1e-2), m, v, acc, cnt, n_w, 1e-3, step=t)
        updates.append((w != before).astype(int))
    assert np.sum(updates, axis=0).tolist() == [12, 6, 4, 3]
