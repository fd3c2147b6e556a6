"""Python face of the CPU oracle (TEST INFRASTRUCTURE — never imported by the product).

Thin ctypes marshalling around ``mxfp4_oracle.c`` plus the composition of the quantized linear
layer (Eq. 3-5 of the paper) out of the oracle's own primitives.  Arrays are numpy; sources are
float32 arrays holding values that are exactly the bf16 (or dequantized MXFP4) inputs.
"""
import ctypes as C

import numpy as np

from .build import build as _build

SCALE_TRUNCATION_FREE, SCALE_FLOOR = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
TIE_EVEN, TIE_PAPER_Q2 = 0, 1

# Random stream of each stochastic quantizer of the backward pass (Q3..Q6 of Eq. 4-5).
STREAM_Q3, STREAM_Q4, STREAM_Q5, STREAM_Q6 = 3, 4, 5, 6

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build())
        u8p, f32p, f64p = C.POINTER(C.c_uint8), C.POINTER(C.c_float), C.POINTER(C.c_double)
        u32p = C.POINTER(C.c_uint32)
        L.orc_e2m1_decode.restype = C.c_double
        L.orc_e2m1_decode.argtypes = [C.c_int]
        L.orc_scale_exponent.restype = C.c_int
        L.orc_scale_exponent.argtypes = [C.c_double, C.c_int]
        L.orc_round_nearest.restype = C.c_int
        L.orc_round_nearest.argtypes = [C.c_float, C.c_int]
        L.orc_round_stochastic.restype = C.c_int
        L.orc_round_stochastic.argtypes = [C.c_float, C.c_uint32]
        L.orc_philox4x32_10.restype = None
        L.orc_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.orc_sr_u16.restype = C.c_uint32
        L.orc_sr_u16.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
        L.orc_quantize.restype = C.c_int64
        L.orc_quantize.argtypes = [f32p, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int,
                                   C.c_int, C.c_uint64, C.c_uint32, u8p, u8p]
        L.orc_quantize_slab.restype = C.c_int64
        L.orc_quantize_slab.argtypes = [f32p, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int,
                                        C.c_int, C.c_uint64, C.c_uint32, C.c_int64, C.c_int64, C.c_int64, u8p, u8p]
        L.orc_dequantize.restype = None
        L.orc_dequantize.argtypes = [u8p, u8p, C.c_int64, C.c_int64, f64p]
        L.orc_qema_quantize.restype = C.c_int64
        L.orc_qema_quantize.argtypes = [f32p, f32p, C.c_float, C.c_int, C.c_int64, C.c_int64, C.c_int,
                                        C.c_int, u8p, u8p]
        L.orc_osc_update.restype = None
        L.orc_osc_update.argtypes = [f32p, u8p, u8p, C.c_int64, C.c_int64, f32p, u8p, u8p, f32p, f32p]
        L.orc_gemm.restype = C.c_int
        L.orc_gemm.argtypes = [u8p, u8p, u8p, u8p, C.c_int64, C.c_int64, C.c_int64, f64p, f64p]
        L.orc_quant_conf.argtypes = [C.c_float]
        L.orc_quant_conf.restype = C.c_float
        L.orc_quant_conf_hist.argtypes = [f32p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.POINTER(C.c_uint64)]
        L.orc_change_sums.argtypes = [f64p, f64p, C.c_int64, f64p]
        L.orc_qramp_detect.argtypes = [f32p, f32p, C.c_int64, C.c_float, C.c_int, C.c_int, u8p]
        L.orc_qramp_detect.restype = C.c_int64
        L.orc_qramp_adamw.argtypes = [f64p, f64p, f64p, f64p, f64p, u8p, u8p, C.c_int64] + [C.c_double] * 7
        L.orc_qramp_adamw.restype = C.c_int64
        _lib = L
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def e2m1_decode(code):
    return lib().orc_e2m1_decode(int(code))


def scale_exponent(amax, scale_mode=SCALE_TRUNCATION_FREE):
    return lib().orc_scale_exponent(float(amax), scale_mode)


def round_nearest(v, tie_mode=TIE_EVEN):
    return lib().orc_round_nearest(C.c_float(v), tie_mode)


def round_stochastic(v, u16):
    return lib().orc_round_stochastic(C.c_float(v), C.c_uint32(int(u16) & 0xFFFF))


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def sr_u16(seed, stream_id, i):
    return int(lib().orc_sr_u16(C.c_uint64(seed), C.c_uint32(stream_id), C.c_uint64(i)))


def quantize(src, transpose=False, scale_mode=SCALE_TRUNCATION_FREE, rounding=ROUND_NEAREST,
             tie_mode=TIE_EVEN, seed=0, stream_id=0, out_row0=0, out_col0=0, out_ld=0):
    """MXFP4-quantize src[rows, cols].  Returns (packed, scales, n_nonfinite_groups).

    transpose=False: packed [rows, cols/2], scales [rows, cols/32] (groups along columns).
    transpose=True : packed [cols, rows/2], scales [cols, rows/32] (groups of 32 source rows).
    out_row0 / out_col0 / out_ld: src is a slab whose output sits at that row and group-axis position of a full
    output with a group axis out_ld long (stochastic rounding draws by position in the full output).
    """
    src = _f32(src)
    rows, cols = src.shape
    glen, outer = (rows, cols) if transpose else (cols, rows)
    if glen % 32:
        raise ValueError("grouped axis must be a multiple of 32")
    packed = np.zeros((outer, glen // 2), dtype=np.uint8)
    scales = np.zeros((outer, glen // 32), dtype=np.uint8)
    nbad = lib().orc_quantize_slab(_p(src, C.c_float), rows, cols, cols, int(bool(transpose)), scale_mode,
                                   rounding, tie_mode, C.c_uint64(seed), C.c_uint32(stream_id), out_row0, out_col0, out_ld,
                                   _p(packed, C.c_uint8), _p(scales, C.c_uint8))
    if nbad < 0:
        raise ValueError("bad shape")
    return packed, scales, int(nbad)


def dequantize(packed, scales):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    rows, half = packed.shape
    out = np.zeros((rows, half * 2), dtype=np.float64)
    lib().orc_dequantize(_p(packed, C.c_uint8), _p(scales, C.c_uint8), rows, half * 2, _p(out, C.c_double))
    return out


def qema_quantize(w, ema, beta=0.998, update_ema=True, scale_mode=SCALE_TRUNCATION_FREE,
                  tie_mode=TIE_EVEN):
    """Q-EMA (Algorithm 1).  ``ema`` is a float32 array updated IN PLACE.  Returns (packed, scales)."""
    w = _f32(w)
    assert ema.dtype == np.float32 and ema.flags.c_contiguous and ema.shape == w.shape
    n, k = w.shape
    packed = np.zeros((n, k // 2), dtype=np.uint8)
    scales = np.zeros((n, k // 32), dtype=np.uint8)
    r = lib().orc_qema_quantize(_p(w, C.c_float), _p(ema, C.c_float), C.c_float(beta), int(bool(update_ema)),
                                n, k, scale_mode, tie_mode, _p(packed, C.c_uint8), _p(scales, C.c_uint8))
    if r < 0:
        raise ValueError("bad shape")
    return packed, scales


def osc_update(w, packed, scales, w_prev, packed_prev, scales_prev, dist_w, dist_q):
    """Oscillation counters (Sec. 6.1); the *_prev and dist_* arrays are updated IN PLACE."""
    w = _f32(w)
    n, k = w.shape
    for a, dt in ((w_prev, np.float32), (packed_prev, np.uint8), (scales_prev, np.uint8),
                  (dist_w, np.float32), (dist_q, np.float32)):
        assert a.dtype == dt and a.flags.c_contiguous
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    lib().orc_osc_update(_p(w, C.c_float), _p(packed, C.c_uint8), _p(scales, C.c_uint8), n, k,
                         _p(w_prev, C.c_float), _p(packed_prev, C.c_uint8), _p(scales_prev, C.c_uint8),
                         _p(dist_w, C.c_float), _p(dist_q, C.c_float))


def gemm(pa, sa, pb, sb, want_bound=True):
    """D = deq(A) @ deq(B)^T in float64 and T = sum_k |a*b|.  A: [m, kc], B: [n, kc] (packed + scales)."""
    pa = np.ascontiguousarray(pa, dtype=np.uint8)
    pb = np.ascontiguousarray(pb, dtype=np.uint8)
    sa = np.ascontiguousarray(sa, dtype=np.uint8)
    sb = np.ascontiguousarray(sb, dtype=np.uint8)
    m, half = pa.shape
    n, half_b = pb.shape
    assert half == half_b
    d = np.zeros((m, n), dtype=np.float64)
    t = np.zeros((m, n), dtype=np.float64) if want_bound else None
    r = lib().orc_gemm(_p(pa, C.c_uint8), _p(sa, C.c_uint8), _p(pb, C.c_uint8), _p(sb, C.c_uint8),
                       m, n, half * 2, _p(d, C.c_double), _p(t, C.c_double) if want_bound else None)
    if r != 0:
        raise ValueError("orc_gemm failed: %d" % r)
    return d, t


# ------------------------------------------------------------------------------------------------
# The quantized linear layer, composed exactly as Eq. 3-5: six quantizers, three products.
# ------------------------------------------------------------------------------------------------
def linear_fwd(x, w, scale_mode=SCALE_TRUNCATION_FREE, ema=None, beta=0.998, update_ema=True,
               tie_mode=TIE_EVEN, want_bound=True):
    """Y = Q1(X) Q2(W)^T (Eq. 3).  With ``ema`` given, Q2 is Q-EMA (Algorithm 1).

    Returns dict(y, t, xq=(packed, scales), wq=(packed, scales)).
    """
    xp, xs, _ = quantize(x, False, scale_mode, ROUND_NEAREST, tie_mode)
    if ema is None:
        wp, ws, _ = quantize(w, False, scale_mode, ROUND_NEAREST, tie_mode)
    else:
        wp, ws = qema_quantize(w, ema, beta, update_ema, scale_mode, tie_mode)
    y, t = gemm(xp, xs, wp, ws, want_bound)
    return dict(y=y, t=t, xq=(xp, xs), wq=(wp, ws))


def linear_bwd_operands(dy, xq, wq, seed, scale_mode=SCALE_TRUNCATION_FREE):
    """The four stochastic quantizers of the backward pass (Eq. 4-5, double quantization)."""
    dyq = quantize(dy, False, scale_mode, ROUND_STOCHASTIC, seed=seed, stream_id=STREAM_Q3)[:2]
    wq_t = quantize(dequantize(*wq), True, scale_mode, ROUND_STOCHASTIC, seed=seed, stream_id=STREAM_Q4)[:2]
    dyq_t = quantize(dy, True, scale_mode, ROUND_STOCHASTIC, seed=seed, stream_id=STREAM_Q5)[:2]
    xq_t = quantize(dequantize(*xq), True, scale_mode, ROUND_STOCHASTIC, seed=seed, stream_id=STREAM_Q6)[:2]
    return dict(dyq=dyq, wq_t=wq_t, dyq_t=dyq_t, xq_t=xq_t)


def linear_bwd(dy, xq, wq, seed, scale_mode=SCALE_TRUNCATION_FREE, want_bound=True):
    """dX = Q3(dY) Q4(Q2(W^T)^T) (Eq. 4) and dW = Q5(dY^T) Q6(Q1(X)) (Eq. 5)."""
    ops = linear_bwd_operands(dy, xq, wq, seed, scale_mode)
    dx, tdx = gemm(*ops["dyq"], *ops["wq_t"], want_bound)
    dw, tdw = gemm(*ops["dyq_t"], *ops["xq_t"], want_bound)
    return dict(dx=dx, tdx=tdx, dw=dw, tdw=tdw, **ops)


def qramp_detect(dist_w, dist_q, k1=16.0, k2=5, n_max=255):
    """Algorithm 2, OscillationDetection: per-element ramp factor n_w and the count of elements with R_w > k1."""
    dw, dq = _f32(dist_w).ravel(), _f32(dist_q).ravel()
    n_w = np.empty(dw.size, dtype=np.uint8)
    osc = lib().orc_qramp_detect(_p(dw, C.c_float), _p(dq, C.c_float), dw.size, k1, k2, n_max, _p(n_w, C.c_uint8))
    return n_w.reshape(np.shape(dist_w)), int(osc)


def qramp_adamw(w, g, m, v, acc, cnt, n_w, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.05, step=1):
    """One step of the customized AdamW of Algorithm 2 (in place on the float64 arrays w, m, v, acc and the uint8 cnt).
    ``step`` is the global step count used for the bias corrections.  Returns the number of updated elements."""
    for a in (w, g, m, v, acc):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    assert cnt.dtype == np.uint8 and cnt.flags.c_contiguous
    nw = None if n_w is None else np.ascontiguousarray(n_w, dtype=np.uint8)
    f64 = C.POINTER(C.c_double)
    return int(lib().orc_qramp_adamw(_p(w, C.c_double), _p(g, C.c_double), _p(m, C.c_double), _p(v, C.c_double),
                                     _p(acc, C.c_double), _p(cnt, C.c_uint8), None if nw is None else _p(nw, C.c_uint8),
                                     w.size, lr, beta1, beta2, eps, weight_decay, 1.0 - beta1 ** step, 1.0 - beta2 ** step))


def quant_conf(a):
    """Quantization confidence (Sec. 4.2) of a latent magnitude a = |w| / 2^s."""
    return float(lib().orc_quant_conf(float(a)))


def quant_conf_hist(w, bins=20, scale_mode=SCALE_TRUNCATION_FREE):
    """Histogram (uint64[bins]) of the quantization confidence of the weight matrix w [n, k]."""
    w = _f32(w)
    n, k = w.shape
    hist = np.zeros(bins, dtype=np.uint64)
    lib().orc_quant_conf_hist(_p(w, C.c_float), n, k, scale_mode, bins, _p(hist, C.c_uint64))
    return hist


def change_sums(cur, prev):
    """(sum (cur - prev)^2, sum prev^2): the two sums of one term of the rate of change r(X) of App. A.3."""
    c = np.ascontiguousarray(cur, dtype=np.float64).ravel()
    p = np.ascontiguousarray(prev, dtype=np.float64).ravel()
    out = np.zeros(2, dtype=np.float64)
    lib().orc_change_sums(_p(c, C.c_double), _p(p, C.c_double), c.size, _p(out, C.c_double))
    return float(out[0]), float(out[1])
