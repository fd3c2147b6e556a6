"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test compares the oracle with something that is not the oracle: values the paper prints,
closed forms, exact rational arithmetic, brute force, published known-answer vectors, numpy.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
GRID = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


# ------------------------------------------------------------------ format (Sec. 3.1)
def test_e2m1_table_and_range():
    vals = [orc.e2m1_decode(c) for c in range(16)]
    assert vals[:8] == GRID
    assert vals[8:] == [-v for v in GRID]
    assert max(vals) == 6.0 and min(vals) == -6.0  # Qp, Qn
    # E_max = 2: the largest binade starts at 2^2
    assert orc.e2m1_decode(6) == 2.0 ** 2


# ------------------------------------------------------------------ scale (Sec. 3.2, Eq. 2)
def test_scale_paper_worked_example_m31():
    # truncation-free: S = 2^3, 31/8 = 3.875 inside [-6, 6]
    assert orc.scale_exponent(31.0, orc.SCALE_TRUNCATION_FREE) == 3
    # Microscaling: S = 2^(4-2) = 4, 31/4 = 7.75 > 6 -> truncated to 6
    assert orc.scale_exponent(31.0, orc.SCALE_FLOOR) == 2
    assert orc.round_nearest(31.0 / 4.0) == 7
    assert orc.round_nearest(31.0 / 8.0) == 6  # 3.875 -> 4


def test_scale_boundaries():
    tf = lambda m: orc.scale_exponent(m, orc.SCALE_TRUNCATION_FREE)
    fl = lambda m: orc.scale_exponent(m, orc.SCALE_FLOOR)
    assert tf(6.0) == 0 and tf(3.0) == -1 and tf(6.03125) == 1 and tf(3.0000002) == 0
    assert fl(4.0) == 0 and fl(7.999) == 0 and fl(8.0) == 1 and fl(3.999) == -1
    # M = 0 -> M~ = 1e-8: ceil(log2(1e-8/6)) = -29 and floor(log2 1e-8) - 2 = -29
    assert tf(0.0) == -29 and fl(0.0) == -29
    assert math.ceil(math.log2(1e-8 / 6)) == -29 and math.floor(math.log2(1e-8)) - 2 == -29


def _all_positive_bf16():
    bits = np.arange(1, 0x7F80, dtype=np.uint32) << 16
    return bits.view(np.float32).astype(np.float64)


def test_scale_brute_force_all_bf16():
    """Every positive finite bf16 value as group maximum, against exact rational arithmetic."""
    for m in _all_positive_bf16():
        fm = Fraction(float(m))
        mant, e = math.frexp(float(m))  # m = mant * 2^e, mant in [0.5, 1)
        e_floor = e - 1  # floor(log2 m)
        s_tf = orc.scale_exponent(m, orc.SCALE_TRUNCATION_FREE)
        s_fl = orc.scale_exponent(m, orc.SCALE_FLOOR)
        # closed form of the ceiling: floor(log2 m) - 2 + [mantissa > 1.5]
        closed = e_floor - 2 + (1 if mant * 2 > 1.5 else 0)
        if -127 <= closed <= 127:
            assert s_tf == closed
            # definition: smallest s with 6 * 2^s >= m  <=>  3 < m / 2^s <= 6
            ratio = fm / (Fraction(2) ** s_tf)
            assert Fraction(3) < ratio <= Fraction(6)
        else:
            assert s_tf == max(-127, min(127, closed))
        want_fl = max(-127, min(127, e_floor - 2))
        assert s_fl == want_fl
        if -127 <= e_floor - 2 <= 127:
            ratio = fm / (Fraction(2) ** s_fl)
            assert Fraction(4) <= ratio < Fraction(8)  # [2^Emax, 2^(Emax+1))


# ------------------------------------------------------------------ round_D (Sec. 3.2)
def test_rne_midpoints_and_threshold():
    mids = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    want = [0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0]
    for m, w in zip(mids, want):
        assert orc.e2m1_decode(orc.round_nearest(m)) == w
        assert orc.e2m1_decode(orc.round_nearest(-m)) == -w
    # Sec. 4.1: threshold -0.75 between q1 = -1 and q2 = -0.5
    assert orc.e2m1_decode(orc.round_nearest(-0.7500001)) == -1.0
    assert orc.e2m1_decode(orc.round_nearest(-0.7499999)) == -0.5


def test_paper_tie_rule_goes_up():
    for m in [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]:
        lo = max(g for g in GRID if g < m)
        hi = min(g for g in GRID if g > m)
        assert orc.e2m1_decode(orc.round_nearest(m, orc.TIE_PAPER_Q2)) == hi
        assert orc.e2m1_decode(orc.round_nearest(-m, orc.TIE_PAPER_Q2)) == -lo


def test_rne_is_nearest_monotone_idempotent_saturating():
    xs = np.linspace(-7.5, 7.5, 6001)
    prev = -10.0
    for x in xs:
        q = orc.e2m1_decode(orc.round_nearest(float(np.float32(x))))
        xc = min(6.0, max(-6.0, float(np.float32(x))))
        best = min(abs(xc - g) for g in GRID + [-g for g in GRID])
        assert abs(xc - q) == best  # a nearest grid point
        assert q >= prev  # monotone
        prev = q
        assert orc.e2m1_decode(orc.round_nearest(q)) == q  # idempotent
    assert orc.round_nearest(100.0) == 7 and orc.round_nearest(-100.0) == 15
    assert orc.round_nearest(-0.0) == 8 and orc.round_nearest(-0.1) == 8  # sign of the source kept


def _read_groups():
    rows = []
    with open(os.path.join(GOLDEN, "hand_worked_groups.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, mode, vals, byte, codes = [p.strip() for p in line.split(";")]
            v = [float.fromhex(t) if "x" in t else float(t) for t in vals.split()]
            rows.append((name, mode, v, int(byte), [int(c, 16) for c in codes.split()]))
    return rows


@pytest.mark.parametrize("name,mode,vals,byte,codes", _read_groups())
def test_hand_worked_groups(name, mode, vals, byte, codes):
    x = np.zeros((1, 32), dtype=np.float32)
    x[0, :len(vals)] = vals
    sm = orc.SCALE_TRUNCATION_FREE if mode == "TF" else orc.SCALE_FLOOR
    packed, scales, nbad = orc.quantize(x, scale_mode=sm)
    assert nbad == 0
    assert scales[0, 0] == byte
    got = []
    for b in packed[0]:
        got += [b & 15, b >> 4]
    assert got[:len(codes)] == codes
    assert all(c == 0 for c in got[len(codes):])
    # the same group quantized along rows (transposed quantizer) gives the same bytes
    pt, st, _ = orc.quantize(x.T.copy(), transpose=True, scale_mode=sm)
    assert (pt == packed).all() and (st == scales).all()


def test_nibble_order_and_packing():
    x = np.zeros((1, 32), dtype=np.float32)
    x[0, 0], x[0, 1], x[0, 31] = 6.0, -3.0, 1.0
    packed, scales, _ = orc.quantize(x)
    assert scales[0, 0] == 127
    assert packed[0, 0] == (7 | (0xD << 4))  # even element in the low nibble
    assert packed[0, 15] == (2 << 4)


def test_truncation_free_never_saturates_and_floor_does():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal((64, 128)) * np.exp(rng.standard_normal((64, 1)) * 4)).astype(np.float32)
    p, s, _ = orc.quantize(x)
    d = orc.dequantize(p, s)
    S = 2.0 ** (s.astype(np.float64) - 127)
    amax = np.abs(x.reshape(64, 4, 32)).max(axis=2)
    assert (amax / S <= 6).all() and (amax / S > 3).all()
    # the group maximum is never clipped: |deq| of the max element >= 0.8 * amax (nearest grid point)
    assert (np.abs(d.reshape(64, 4, 32)).max(axis=2) >= amax * 0.8).all()
    pf, sf, _ = orc.quantize(x, scale_mode=orc.SCALE_FLOOR)
    Sf = 2.0 ** (sf.astype(np.float64) - 127)
    assert (amax / Sf >= 4).all() and (amax / Sf < 8).all()
    assert (amax / Sf > 6).any()  # some groups do get truncated under Eq. 2


def test_nonfinite_group():
    x = np.ones((2, 64), dtype=np.float32)
    x[0, 40] = np.inf
    x[1, 3] = np.nan
    p, s, nbad = orc.quantize(x)
    assert nbad == 2
    assert s[0, 1] == 0xFF and s[1, 0] == 0xFF and s[0, 0] != 0xFF
    assert (p[0, 16:] == 0).all() and (p[1, :16] == 0).all()


# ------------------------------------------------------------------ Philox + round_S
def test_philox_known_answers():
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        lines = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(lines) == 3
    for w in lines:
        v = [int(t, 16) for t in w if t != "->"]
        assert orc.philox4x32_10(v[0:4], v[4:6]) == v[6:10]


def test_sr_u16_indexing():
    seed = 0x0123456789ABCDEF

    def rev16(x):
        return int("{:016b}".format(x)[::-1], 2)

    for i in [0, 1, 2, 3, 4, 7, 8, 13, 15, 16, 17, 1000003, (1 << 35) + 5, (1 << 40) + 2]:
        q, m = i >> 4, i >> 1
        w = orc.philox4x32_10([q & 0xFFFFFFFF, q >> 32, 5, 0], [seed & 0xFFFFFFFF, seed >> 32])[(m & 7) >> 1]
        field = (w >> 16) if (m & 1) else (w & 0xFFFF)
        assert orc.sr_u16(seed, 5, i) == (rev16(field) if (i & 1) else field)
    assert [orc.sr_u16(seed, 5, i) for i in range(16, 32)] != [orc.sr_u16(seed, 6, i) for i in range(16, 32)]
    assert [orc.sr_u16(seed, 5, i) for i in range(16, 32)] != [orc.sr_u16(seed + 1, 5, i) for i in range(16, 32)]
    # the two elements of a pair read one field in opposite bit orders; a reversed draw is as uniform as a plain one
    assert all(orc.sr_u16(seed, 3, 2 * m + 1) == rev16(orc.sr_u16(seed, 3, 2 * m)) for m in range(64))
    assert sorted(rev16(x) for x in range(1 << 16)) == list(range(1 << 16))
    odd = np.array([orc.sr_u16(seed, 3, 2 * m + 1) for m in range(1 << 15)])
    even = np.array([orc.sr_u16(seed, 3, 2 * m) for m in range(1 << 15)])
    for draws in (odd, even):
        top = np.bincount(draws >> 12, minlength=16)       # 16 bins, mean 2048, sigma ~44
        assert top.min() > 1800 and top.max() < 2300
    # the coarse decisions of the two elements of a pair (their top bits) are uncorrelated
    both = np.mean((odd >> 15) & (even >> 15))
    assert abs(both - 0.25) < 0.02


def test_sr_threshold_counts_exact():
    """P(up) = f exactly: up iff f + u >= 1, u = u16 / 2^16.  The decision flips between
    u16 = 2^16 (1 - f) - 1 and 2^16 (1 - f) and is monotone in u16, hence exactly f * 2^16 of the
    2^16 values of u16 round up.  Checked exhaustively for one case, at the boundary for the rest."""
    for lo, hi in [(0.0, 0.5), (0.5, 1.0), (1.0, 1.5), (2.0, 3.0), (4.0, 6.0)]:
        for j in range(1, 8):
            f = j / 8.0
            v = lo + f * (hi - lo)
            first_up = int((1 - f) * (1 << 16))
            for sign in (1.0, -1.0):
                up = lambda u: abs(orc.e2m1_decode(orc.round_stochastic(sign * v, u))) == hi
                assert not up(first_up - 1) and up(first_up)
                assert not up(0) and up(0xFFFF)
                res = orc.e2m1_decode(orc.round_stochastic(sign * v, 0))
                assert math.copysign(1.0, res) == sign
    ups = sum(orc.e2m1_decode(orc.round_stochastic(2.375, u)) == 3.0 for u in range(1 << 16))
    assert ups == int(0.375 * (1 << 16))
    # a fraction finer than 2^-16 rounds the probability down: floor(f * 2^16) / 2^16
    tiny = 2.0 ** -20  # f = 2^-19
    assert all(orc.e2m1_decode(orc.round_stochastic(tiny, u)) == 0.0 for u in (0, 1, 0x8000, 0xFFFF))
    v = 0.5 - 2.0 ** -20  # f = 1 - 2^-19: every u16 >= 1 rounds up, u16 = 0 does not
    assert orc.e2m1_decode(orc.round_stochastic(v, 0)) == 0.0
    assert orc.e2m1_decode(orc.round_stochastic(v, 1)) == 0.5


def _rev16_table():
    f = np.arange(1 << 16, dtype=np.uint32)
    r = np.zeros_like(f)
    for b in range(16):
        r |= ((f >> b) & 1) << (15 - b)
    return f, r


def test_sr_pair_joint_law_is_close_to_independent():
    """Sec. 3.2 rounds "each value independently".  Elements 2m and 2m+1 of a quantizer's output share one 16-bit field
    F: the even one rounds up iff F >= 2^16 (1 - f_e), the odd one iff rev16(F) >= 2^16 (1 - f_o).  Over the 2^16 equally
    likely fields each marginal is exact (pinned above); this pins the JOINT law: for fractions with at most 8 bits
    the two decisions read disjoint halves of the field, so P(both up) = f_e f_o exactly, and for every other pair of
    16-bit fractions |P(both up) - f_e f_o| <= 2^-13 (the largest deviation over all 2^32 pairs of thresholds, found by
    an exhaustive scan, is 8.31e-5 = 2^-13.56 at f_e = f_o = 21845 / 65536).  The counts below come from the oracle's
    own rounding rule applied to every field."""
    F, R = _rev16_table()

    def ups(v, draws):
        # which of the 2^16 draws round the latent v (between 2 and 3, so f = v - 2) up, by the oracle's rule
        lo_first = int(round((1.0 - (v - 2.0)) * 65536))
        for u in (lo_first - 1, lo_first):
            if 0 <= u <= 0xFFFF:
                assert (orc.e2m1_decode(orc.round_stochastic(v, u)) == 3.0) == (u >= lo_first)
        return draws >= lo_first

    def latent(k16):
        return 2.0 + k16 / 65536.0          # exact in float32: 2 + a 16-bit fraction

    eight_bit = [1 * 256, 37 * 256, 128 * 256, 200 * 256, 255 * 256]
    # bf16 latents below 0.25 have fractions 2|v| with up to 16 bits (8 significant bits at exponents down to 2^-9)
    bf16_small = [int(m * 2.0 ** e * 2 * 65536) for m, e in ((1.0078125, -3), (1.4921875, -5), (1.9921875, -9), (1.5078125, -7))]
    fine = [1, 2, 255, 257, 21845, 21846, 32767, 32768, 32769, 43690, 43691, 65535] + bf16_small
    rng = np.random.default_rng(11)
    fine += [int(x) for x in rng.integers(1, 65536, size=40)]
    worst = 0.0
    for ke in eight_bit + fine:
        up_e = ups(latent(ke), F)
        assert int(up_e.sum()) == ke
        for ko in eight_bit + fine:
            up_o = ups(latent(ko), R)
            assert int(up_o.sum()) == ko
            both = int((up_e & up_o).sum())
            dev = both / 65536.0 - (ke / 65536.0) * (ko / 65536.0)
            if ke % 256 == 0 and ko % 256 == 0:
                assert both * 65536 == ke * ko, (ke, ko)      # exactly independent
            assert abs(dev) <= 2.0 ** -13, (ke, ko, dev)
            worst = max(worst, abs(dev))
    assert worst >= 8.3e-5      # the grid holds the worst pair of the exhaustive scan


def test_sr_dot_product_variance_matches_independent_draws():
    """What the independence of Sec. 3.2 is needed for: the variance of a sum of stochastically rounded values.  A
    32-term dot product sum_i b_i round_S(v_i) over 2^15 rows (each row its own counters, so rows are independent
    draws) must have the variance sum_i b_i^2 f_i (1 - f_i) D_i^2 of independent roundings, within 5 sigma of the
    sample variance's own spread, and the mean of exact unbiased rounding."""
    rng = np.random.default_rng(5)
    grid = np.array(GRID)
    v = np.empty(32)
    for i in range(32):
        j = rng.integers(0, 7)
        frac = rng.integers(1, 65536) / 65536.0 if i % 3 else rng.integers(1, 256) / 256.0
        v[i] = grid[j] + frac * (grid[j + 1] - grid[j])
    v[0] = 5.96875                                  # keeps the group's scale exponent at 0
    v *= rng.choice([-1.0, 1.0], size=32)
    v = v.astype(np.float32).astype(np.float64)
    b = rng.standard_normal(32)
    lo = np.array([grid[grid <= a].max() for a in np.abs(v)])
    hi = np.array([grid[grid > a].min() if (grid > a).any() else 6.0 for a in np.abs(v)])
    f = (np.abs(v) - lo) / (hi - lo)
    assert (np.abs(f * 65536 - np.round(f * 65536)) < 1e-9).all()     # P(up) = f exactly for these latents
    var_ind = float(np.sum(b ** 2 * f * (1 - f) * (hi - lo) ** 2))
    rows = 1 << 15
    x = np.tile(v.astype(np.float32), (rows, 1))
    p, s, _ = orc.quantize(x, rounding=orc.ROUND_STOCHASTIC, seed=0xC0FFEE, stream_id=3)
    assert (s == 127).all()
    d = orc.dequantize(p, s) @ b
    mean_err = abs(d.mean() - float(v @ b))
    assert mean_err <= 5 * np.sqrt(var_ind / rows)
    m2 = d.var(ddof=1)
    m4 = np.mean((d - d.mean()) ** 4)
    se = np.sqrt((m4 - m2 ** 2) / rows)                          # standard error of the sample variance
    assert abs(m2 - var_ind) <= 5 * se, (m2, var_ind, se)
    # the pair covariance the shared field can add is at most 2^-13 D_e D_o |b_e b_o| per pair: far inside that band
    pair_cov = sum(2.0 ** -13 * (hi[2 * m] - lo[2 * m]) * (hi[2 * m + 1] - lo[2 * m + 1]) * abs(b[2 * m] * b[2 * m + 1]) for m in range(16))
    assert 2 * pair_cov < 0.01 * var_ind


def test_sr_on_grid_never_moves_and_saturates():
    for g in GRID:
        for u in (0, 0xFFFF, 0x8000, 12345):
            assert orc.e2m1_decode(orc.round_stochastic(g, u)) == g
            assert orc.e2m1_decode(orc.round_stochastic(-g, u)) == -g
    assert orc.round_stochastic(7.5, 0xFFFF) == 7 and orc.round_stochastic(-9.0, 0) == 15


def test_sr_unbiased_monte_carlo():
    """E[round_S(x/S)] = x/S (Sec. 3.2): average over seeds on one group."""
    rng = np.random.default_rng(7)
    x = (rng.standard_normal((1, 32)) * 2).astype(np.float32)
    x[0, 0] = 5.9  # scale exponent 0
    n = 4096
    acc = np.zeros(32)
    acc2 = np.zeros(32)
    for seed in range(n):
        p, s, _ = orc.quantize(x, rounding=orc.ROUND_STOCHASTIC, seed=seed, stream_id=3)
        assert s[0, 0] == 127
        d = orc.dequantize(p, s)[0]
        acc += d
        acc2 += d * d
    mean = acc / n
    var = np.maximum(acc2 / n - mean ** 2, 0)
    tol = 5 * np.sqrt(var / n) + 1e-12
    assert (np.abs(mean - x[0].astype(np.float64)) <= tol).all()
    assert (np.abs(orc.dequantize(p, s)) <= 6).all()


# ------------------------------------------------------------------ transposed / double quantization
def test_transposed_equals_rowwise_on_transpose():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((96, 40)).astype(np.float32)
    for sm in (orc.SCALE_TRUNCATION_FREE, orc.SCALE_FLOOR):
        pt, st, _ = orc.quantize(x, transpose=True, scale_mode=sm)
        pr, sr, _ = orc.quantize(np.ascontiguousarray(x.T), transpose=False, scale_mode=sm)
        assert pt.shape == (40, 48) and st.shape == (40, 3)
        assert (pt == pr).all() and (st == sr).all()


def test_transposed_sr_equals_rowwise_sr_on_transpose():
    rng = np.random.default_rng(14)
    x = rng.standard_normal((96, 48)).astype(np.float32)
    pt, st, _ = orc.quantize(x, transpose=True, rounding=orc.ROUND_STOCHASTIC, seed=5, stream_id=5)
    pr, sr, _ = orc.quantize(np.ascontiguousarray(x.T), transpose=False, rounding=orc.ROUND_STOCHASTIC, seed=5, stream_id=5)
    assert (pt == pr).all() and (st == sr).all()


def test_slab_quantization_equals_the_slice_of_the_whole():
    """A slab quantized on its own, told where it sits, gives exactly the corresponding part of the full result."""
    rng = np.random.default_rng(15)
    x = rng.standard_normal((96, 128)).astype(np.float32)
    kw = dict(rounding=orc.ROUND_STOCHASTIC, seed=3, stream_id=5)
    p, s, _ = orc.quantize(x, **kw)
    ps, ss, _ = orc.quantize(np.ascontiguousarray(x[32:64]), out_row0=32, **kw)
    assert (ps == p[32:64]).all() and (ss == s[32:64]).all()
    pt, st, _ = orc.quantize(x, transpose=True, **kw)
    # source rows 32..63, source columns 64..95 -> output rows 64..95, output positions 32..63
    sub = np.ascontiguousarray(x[32:64, 64:96])
    ps, ss, _ = orc.quantize(sub, transpose=True, out_row0=64, out_col0=32, out_ld=96, **kw)
    assert (ps == pt[64:96, 16:32]).all() and (ss == st[64:96, 1:2]).all()


def test_transposed_sr_uses_output_index():
    rng = np.random.default_rng(4)
    rows, cols = 64, 8
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    seed, stream = 99, 5
    pt, st, _ = orc.quantize(x, transpose=True, rounding=orc.ROUND_STOCHASTIC, seed=seed, stream_id=stream)
    for c in range(cols):
        for g in range(rows // 32):
            s = int(st[c, g]) - 127
            for i in range(32):
                r = g * 32 + i
                v = np.float32(x[r, c]) / np.float32(2.0 ** s)
                want = orc.round_stochastic(float(v), orc.sr_u16(seed, stream, c * rows + r))
                b = pt[c, (g * 32 + i) // 2]
                got = (b >> 4) if (i & 1) else (b & 15)
                assert got == want


def test_double_quantization_keeps_group_max_and_is_exact_on_grid():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((64, 64)).astype(np.float32)
    p1, s1, _ = orc.quantize(x)
    d1 = orc.dequantize(p1, s1)
    # re-quantizing along the other axis: every value is P*2^s; the column-group maximum is
    # m*2^e with m in {1,1.5} -> under the truncation-free scale it lands on 4 or 6 exactly.
    for seed in range(3):
        p2, s2, _ = orc.quantize(d1, transpose=True, rounding=orc.ROUND_STOCHASTIC, seed=seed, stream_id=6)
        d2 = orc.dequantize(p2, s2).T
        amax_in = np.abs(d1.reshape(2, 32, 64)).max(axis=1)
        amax_out = np.abs(d2.reshape(2, 32, 64)).max(axis=1)
        assert (amax_in == amax_out).all()
    # same axis again reproduces the same values (the scale may drop when the maximum rounded down)
    p3, s3, _ = orc.quantize(d1)
    assert (orc.dequantize(p3, s3) == d1).all()


# ------------------------------------------------------------------ Q-EMA (Sec. 5, Algorithm 1)
def test_qema_reduces_to_plain_when_ema_equals_w():
    rng = np.random.default_rng(6)
    w = (rng.standard_normal((48, 96)) * 0.02).astype(np.float32)
    for sm in (orc.SCALE_TRUNCATION_FREE, orc.SCALE_FLOOR):
        ema = w.copy()
        p, s = orc.qema_quantize(w, ema, update_ema=False, scale_mode=sm)
        pr, sr, _ = orc.quantize(w, scale_mode=sm)
        assert (p == pr).all() and (s == sr).all()
        # updating with ema == w leaves ema (numerically almost) at w and the codes unchanged
        ema = w.copy()
        p, s = orc.qema_quantize(w, ema, beta=0.5, update_ema=True, scale_mode=sm)
        assert (p == pr).all()


def test_qema_worked_pairs():
    w = np.zeros((1, 32), dtype=np.float32)
    ema = np.zeros((1, 32), dtype=np.float32)
    w[0, 0] = ema[0, 0] = 6.0  # S = 1
    w[0, 1], ema[0, 1] = 0.7421875, 0.7578125  # plain: 0.5; EMA is past the 0.75 threshold -> 1.0
    w[0, 2], ema[0, 2] = 0.7578125, 0.2  # plain: 1.0; EMA says 0.5
    w[0, 3], ema[0, 3] = -0.76, -0.70  # plain: -1.0; EMA says -0.5  (Sec. 4.1 threshold -0.75)
    w[0, 4], ema[0, 4] = 1.5, 5.0  # on the grid: kept
    w[0, 5], ema[0, 5] = 2.2, -6.0  # EMA far on the other side: nearer endpoint of [2, 3] is 2
    w[0, 6], ema[0, 6] = 2.2, 100.0  # EMA beyond the range: nearer endpoint is 3
    p, s = orc.qema_quantize(w, ema, update_ema=False)
    d = orc.dequantize(p, s)[0]
    assert s[0, 0] == 127
    assert list(d[:7]) == [6.0, 1.0, 0.5, -0.5, 1.5, 2.0, 3.0]
    plain = orc.dequantize(*orc.quantize(w)[:2])[0]
    assert list(plain[:4]) == [6.0, 0.5, 1.0, -1.0]


def test_qema_output_is_one_of_the_two_neighbours():
    rng = np.random.default_rng(8)
    w = (rng.standard_normal((16, 64))).astype(np.float32)
    ema = (w + rng.standard_normal((16, 64)) * 0.7).astype(np.float32)
    p, s = orc.qema_quantize(w, ema, update_ema=False)
    d = orc.dequantize(p, s)
    S = np.repeat(2.0 ** (s.astype(np.float64) - 127), 32, axis=1)
    lat = w.astype(np.float64) / S
    for v, q in zip(lat.ravel(), (d / S).ravel()):
        a = abs(v)
        lo = max(g for g in GRID if g <= a)
        hi = min(g for g in GRID if g >= a)
        assert abs(q) in (lo, hi) and (q == 0 or math.copysign(1, q) == math.copysign(1, v))


def test_ema_closed_form():
    """Eq. 10 with a constant weight: ema_n = w + beta^n (ema_0 - w)."""
    w = np.full((1, 32), 0.3125, dtype=np.float32)
    ema0 = np.linspace(-1, 1, 32, dtype=np.float32).reshape(1, 32)
    ema = ema0.copy()
    beta = 0.998
    n = 500
    for _ in range(n):
        orc.qema_quantize(w, ema, beta=beta, update_ema=True)
    want = 0.3125 + (np.float32(beta).astype(np.float64) ** n) * (ema0.astype(np.float64) - 0.3125)
    assert np.allclose(ema, want, rtol=0, atol=n * 2.0 ** -23)
    # update_ema = False leaves the state alone
    before = ema.copy()
    orc.qema_quantize(w, ema, beta=beta, update_ema=False)
    assert (ema == before).all()


def test_ema_update_is_fp32_fma_order():
    # one step, checked against exact rational arithmetic rounded to float32
    w = np.array([[0.02001953125] + [0.0] * 31], dtype=np.float32)
    ema = np.array([[0.0137] + [0.0] * 31], dtype=np.float32)
    beta = np.float32(0.998)
    omb = np.float32(1.0) - beta
    e0 = Fraction(float(ema[0, 0]))
    t = np.float32(omb * w[0, 0])
    exact = Fraction(float(beta)) * e0 + Fraction(float(t))
    orc.qema_quantize(w, ema, beta=0.998, update_ema=True)
    got = Fraction(float(ema[0, 0]))
    # correctly rounded: no other float32 is closer to the exact value
    up = Fraction(float(np.nextafter(ema[0, 0], np.float32(np.inf))))
    dn = Fraction(float(np.nextafter(ema[0, 0], np.float32(-np.inf))))
    assert abs(got - exact) <= abs(up - exact) and abs(got - exact) <= abs(dn - exact)


# ------------------------------------------------------------------ oscillation counters (Sec. 6.1)
def test_oscillation_counters_scripted_trajectory():
    k = 32
    S = 1.0  # group max 6 keeps the scale at 1
    traj = [0.74, 0.76, 0.74, 0.76, 0.74, 0.76, 0.74]  # crosses 0.75 six times
    w0 = np.zeros((1, k), dtype=np.float32)
    w0[0, 0] = 6.0
    w0[0, 1] = traj[0]
    w0[0, 2] = 1.1
    p, s, _ = orc.quantize(w0)
    w_prev, p_prev, s_prev = w0.copy(), p.copy(), s.copy()
    dist_w = np.zeros((1, k), dtype=np.float32)
    dist_q = np.zeros((1, k), dtype=np.float32)
    for t in traj[1:]:
        w = w0.copy()
        w[0, 1] = t
        p, s, _ = orc.quantize(w)
        orc.osc_update(w, p, s, w_prev, p_prev, s_prev, dist_w, dist_q)
    # each flip between 0.5 and 1.0 adds |q1 - q2| * S = 0.5
    assert dist_q[0, 1] == pytest.approx(6 * 0.5 * S)
    assert dist_w[0, 1] == pytest.approx(6 * 0.02, rel=1e-4)
    assert dist_q[0, 1] / dist_w[0, 1] > 16  # oscillating by the paper's k1 = 16 criterion
    assert dist_q[0, 2] == 0 and dist_w[0, 2] == 0 and dist_q[0, 0] == 0
    assert (w_prev == w).all() and (p_prev == p).all()


# ------------------------------------------------------------------ products (Eq. 3-5)
def _unpack(p):
    out = np.zeros((p.shape[0], p.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = p & 15
    out[:, 1::2] = p >> 4
    return out


def test_gemm_small_integer_exact():
    rng = np.random.default_rng(9)
    m, n, k = 24, 40, 96
    ca = rng.integers(0, 3, size=(m, k)).astype(np.uint8) * 2  # codes 0,2,4 = 0,1,2
    cb = rng.integers(0, 3, size=(n, k)).astype(np.uint8) * 2
    sgn_a = rng.integers(0, 2, size=(m, k)).astype(np.uint8) * 8
    ca |= sgn_a
    pa = (ca[:, 0::2] | (ca[:, 1::2] << 4)).astype(np.uint8)
    pb = (cb[:, 0::2] | (cb[:, 1::2] << 4)).astype(np.uint8)
    sa = np.full((m, k // 32), 127, dtype=np.uint8)
    sb = np.full((n, k // 32), 127, dtype=np.uint8)
    ia = (ca & 7).astype(np.int64) // 2 * np.where(ca & 8, -1, 1)
    ib = (cb & 7).astype(np.int64) // 2
    d, t = orc.gemm(pa, sa, pb, sb)
    assert (d == (ia @ ib.T)).all()
    assert (t == (np.abs(ia) @ ib.T)).all()


def test_gemm_one_hot_reads_scales_and_nibbles():
    m, n, k = 4, 6, 128
    pa = np.zeros((m, k // 2), dtype=np.uint8)
    pb = np.zeros((n, k // 2), dtype=np.uint8)
    sa = np.arange(m * 4, dtype=np.uint8).reshape(m, 4) + 120
    sb = np.arange(n * 4, dtype=np.uint8).reshape(n, 4) + 110
    # A[2, 71] = 3.0 (code 5, odd element -> high nibble), B[4, 71] = -1.5 (code 0xB)
    pa[2, 35] = 5 << 4
    pb[4, 35] = 0xB << 4
    d, t = orc.gemm(pa, sa, pb, sb)
    want = 3.0 * 2.0 ** (int(sa[2, 2]) - 127) * -1.5 * 2.0 ** (int(sb[4, 2]) - 127)
    assert d[2, 4] == want and t[2, 4] == abs(want)
    d[2, 4] = 0
    assert (d == 0).all()


def test_gemm_matches_numpy_on_dequantized_and_transposition():
    rng = np.random.default_rng(10)
    x = rng.standard_normal((40, 128)).astype(np.float32)
    w = (rng.standard_normal((24, 128)) * 0.02).astype(np.float32)
    xp, xs, _ = orc.quantize(x)
    wp, ws, _ = orc.quantize(w)
    d, t = orc.gemm(xp, xs, wp, ws)
    ref = orc.dequantize(xp, xs) @ orc.dequantize(wp, ws).T
    assert np.allclose(d, ref, rtol=1e-12, atol=1e-300)
    assert (t >= np.abs(d) - 1e-300).all()
    d2, _ = orc.gemm(wp, ws, xp, xs)
    assert (d2 == d.T).all()  # a transposed operand order fails here


def test_linear_composition_matches_eq_3_to_5():
    rng = np.random.default_rng(11)
    M, K, N = 64, 96, 32
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    dy = (rng.standard_normal((M, N)) * 1e-3).astype(np.float32)
    f = orc.linear_fwd(x, w)
    xd, wd = orc.dequantize(*f["xq"]), orc.dequantize(*f["wq"])
    assert np.allclose(f["y"], xd @ wd.T, rtol=1e-12, atol=0)
    b = orc.linear_bwd(dy, f["xq"], f["wq"], seed=5)
    assert b["dx"].shape == (M, K) and b["dw"].shape == (N, K)
    dyq = orc.dequantize(*b["dyq"])  # [M, N]
    wq_t = orc.dequantize(*b["wq_t"])  # [K, N]
    dyq_t = orc.dequantize(*b["dyq_t"])  # [N, M]
    xq_t = orc.dequantize(*b["xq_t"])  # [K, M]
    assert np.allclose(b["dx"], dyq @ wq_t.T, rtol=1e-12, atol=0)
    assert np.allclose(b["dw"], dyq_t @ xq_t.T, rtol=1e-12, atol=0)
    # the four stochastic quantizers draw from different streams
    assert not (orc.dequantize(*b["dyq"]).T == orc.dequantize(*b["dyq_t"])).all()


def test_gradient_unbiased_tiny_layer():
    """E[Q3(dY) Q4(.)] = dY Q2(W^T)^T and E[Q5(dY^T) Q6(.)] = dY^T Q1(X) (Sec. 3.4)."""
    rng = np.random.default_rng(12)
    M, K, N = 32, 32, 32
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = rng.standard_normal((N, K)).astype(np.float32)
    dy = rng.standard_normal((M, N)).astype(np.float32)
    f = orc.linear_fwd(x, w)
    xd, wd = orc.dequantize(*f["xq"]), orc.dequantize(*f["wq"])
    want_dx = dy.astype(np.float64) @ wd
    want_dw = dy.astype(np.float64).T @ xd
    n = 1500
    sx = np.zeros_like(want_dx); sx2 = np.zeros_like(want_dx)
    sw = np.zeros_like(want_dw); sw2 = np.zeros_like(want_dw)
    for seed in range(n):
        b = orc.linear_bwd(dy, f["xq"], f["wq"], seed=seed, want_bound=False)
        sx += b["dx"]; sx2 += b["dx"] ** 2
        sw += b["dw"]; sw2 += b["dw"] ** 2
    for s1, s2, want in ((sx, sx2, want_dx), (sw, sw2, want_dw)):
        mean = s1 / n
        sd = np.sqrt(np.maximum(s2 / n - mean ** 2, 0) / n)
        z = np.abs(mean - want) / (sd + 1e-12)
        assert z.max() < 5.5, z.max()
        assert np.mean(z) < 1.2
