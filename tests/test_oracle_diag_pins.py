"""Pins of the diagnostics oracle (quantization confidence, Sec. 4.2 / App. A.2; rate of change, App. A.3)."""
from fractions import Fraction

import numpy as np

import oracle as orc

GRID = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3), Fraction(4), Fraction(6)]


def conf_by_definition(a: Fraction) -> Fraction:
    """The definition taken literally, in exact rationals and by search: thresholds of the signed grid, the set of
    latents that round to the same value as `a`, and the largest threshold distance inside that set."""
    signed = sorted(set([-g for g in GRID] + GRID))
    thr = [(x + y) / 2 for x, y in zip(signed[:-1], signed[1:])]
    dist = lambda v: min(abs(v - t) for t in thr)  # noqa: E731
    nearest = min(signed, key=lambda g: (abs(a - g), g))          # the value `a` rounds to (ties do not matter: distance 0)
    lo = max([t for t in thr if t <= a] or [Fraction(-6)])
    hi = min([t for t in thr if t >= a] or [Fraction(6)])
    if a in thr:
        return Fraction(0)
    assert lo <= nearest <= hi
    # largest distance to a threshold within the cell [lo, hi] (clipped to the representable range +-6), on a fine lattice
    pts = [lo + (hi - lo) * Fraction(i, 64) for i in range(65)]
    return dist(a) / max(dist(p) for p in pts)


def test_confidence_hand_values():
    # on a grid value whose cell is symmetric the confidence is 1; 2 and 4 sit off-centre in their cells
    assert orc.quant_conf(0.0) == 1.0 and orc.quant_conf(0.5) == 1.0 and orc.quant_conf(3.0) == 1.0 and orc.quant_conf(6.0) == 1.0
    assert orc.quant_conf(2.0) == np.float32(np.float32(0.25) / np.float32(0.375))
    assert orc.quant_conf(4.0) == np.float32(np.float32(0.5) / np.float32(0.75))
    for t in (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0):
        assert orc.quant_conf(t) == 0.0
    assert orc.quant_conf(7.5) == 1.0          # beyond the grid (floor scaling): saturated, counted as confident


def test_confidence_against_the_definition_on_all_bf16_latents():
    # every latent magnitude a bf16 value can produce in [2^-6, 6]: 8 significant bits
    vals = set()
    for e in range(-6, 3):
        for m in range(128, 256):
            v = Fraction(m, 128) * Fraction(2) ** e
            if v <= 6:
                vals.add(v)
    vals.add(Fraction(0))
    for a in sorted(vals):
        want = conf_by_definition(a)
        got = orc.quant_conf(float(a))
        assert 0.0 <= got <= 1.0
        assert abs(Fraction(got) - want) <= Fraction(1, 2 ** 23), (a, got, float(want))


def test_histogram_counts_every_element_once_and_matches_elementwise():
    rng = np.random.default_rng(3)
    w = (rng.normal(0, 0.02, (64, 96))).astype(np.float32)
    import workloads
    w = workloads.round_to_bf16(w)
    h = orc.quant_conf_hist(w, bins=16)
    assert int(h.sum()) == w.size
    # element by element with the scale the quantizer uses
    p, s, _ = orc.quantize(w)
    ref = np.zeros(16, dtype=np.uint64)
    for r in range(w.shape[0]):
        for c in range(w.shape[1]):
            a = np.float32(abs(w[r, c])) / np.float32(2.0) ** (int(s[r, c // 32]) - 127)
            b = min(int(np.floor(np.float32(orc.quant_conf(float(a))) * np.float32(16))), 15)
            ref[b] += 1
    assert (h == ref).all()


def test_change_sums_closed_form():
    prev = np.arange(1, 101, dtype=np.float64)
    cur = prev + 0.5
    d2, p2 = orc.change_sums(cur, prev)
    assert d2 == 100 * 0.25 and p2 == 100 * 101 * 201 / 6
    # r(X) for a uniformly scaled tensor: ||(1+c)X - X|| / ||X|| = c
    x = np.random.default_rng(1).normal(size=1000)
    d2, p2 = orc.change_sums(1.25 * x, x)
    assert abs(np.sqrt(d2 / p2) - 0.25) < 1e-12
