"""ctypes binding of libmxfp4.so: argument marshalling only — every step runs in the CUDA kernels.

torch is used for device memory and streams.  The library must be present (built in-tree by
``paper_2502_20853_b200.build``); there is no fallback path of any kind.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmxfp4.so")

SCALE_TRUNCATION_FREE, SCALE_FLOOR = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
OUT_BF16, OUT_FP32 = 0, 1
DEV_NONFINITE, DEV_TIMEOUT, DEV_SMEM_LAYOUT = 1, 2, 4
HOOK_IDENTITY, HOOK_GELU, HOOK_MULTIPLY = 0, 1, 2

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "BAD_SHAPE", 3: "MISALIGNED", 4: "WORKSPACE_TOO_SMALL",
                5: "UNSUPPORTED_DEVICE", 6: "CUDA_ERROR"}

EXPORTS = ["mxfp4_launch_count", "mxfp4_scale_bytes", "mxfp4_scale_offset", "mxfp4_gemm_workspace_bytes", "mxfp4_gemm_chain_mmas",
           "mxfp4_linear_workspace_bytes", "mxfp4_quantize", "mxfp4_quantize_t", "mxfp4_quantize_2axis", "mxfp4_quantize_chain",
           "mxfp4_qema_quantize", "mxfp4_dequantize", "mxfp4_gemm", "mxfp4_gemm_quant", "mxfp4_gemm_static", "mxfp4_linear_fwd",
           "mxfp4_linear_bwd", "mxfp4_linear_fwd_ex", "mxfp4_linear_bwd_ex", "mxfp4_qramp_adamw", "mxfp4_qramp_detect", "mxfp4_quant_conf_hist", "mxfp4_change_sums",
           "mxfp4_change_sums_q", "mxfp4_mma_issue_ceiling", "mxfp4_gemm_wait_selftest", "mxfp4_quantize_wait_selftest"]


class MxError(RuntimeError):
    def __init__(self, fn, status):
        super().__init__("%s returned %s (%d)" % (fn, STATUS_NAMES.get(status, "?"), status))
        self.status = status


class CMat(C.Structure):
    _fields_ = [("data", C.c_void_p), ("scales", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64)]


class CQParams(C.Structure):
    _fields_ = [("scale_mode", C.c_int32), ("rounding", C.c_int32), ("seed", C.c_uint64),
                ("stream_id", C.c_uint32), ("reserved", C.c_uint32)]


class COsc(C.Structure):
    _fields_ = [("w_prev", C.c_void_p), ("wq_prev", CMat), ("dist_w", C.c_void_p), ("dist_q", C.c_void_p)]


class CAdamW(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float), ("weight_decay", C.c_float),
                ("bias_corr1", C.c_float), ("bias_corr2", C.c_float)]


class CEpilogue(C.Structure):
    _fields_ = [("hook", C.c_int32), ("chain", C.c_int32), ("aux", C.c_void_p), ("ld_aux", C.c_int64), ("y", C.c_void_p), ("ldy", C.c_int64),
                ("z", C.c_void_p), ("ldz", C.c_int64), ("zq", CMat), ("qp_row", CQParams), ("zq_t", CMat), ("qp_t", CQParams)]


class CCtx(C.Structure):
    _fields_ = [("xq", CMat), ("wq", CMat), ("xq_t", CMat), ("xq_t_seed", C.c_uint64), ("wq_t", CMat), ("wq_t_seed", C.c_uint64)]


_lib = None

# Where this binding allocates an output or scratch buffer for the caller it goes through _new(); a test harness may
# install a hook here (shape, dtype, device) -> tensor, e.g. to surround every buffer with guard bytes.
ALLOC_HOOK = None


def _new(shape, dtype, device):
    if ALLOC_HOOK is not None:
        return ALLOC_HOOK(shape, dtype, device)
    return torch.empty(shape, dtype=dtype, device=device)


def lib():
    """Load libmxfp4.so; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libmxfp4.so is missing: run `python -m paper_2502_20853_b200.build` "
                           "(there is no CPU or library fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i64, i32, u64, sz = C.c_void_p, C.c_int64, C.c_int32, C.c_uint64, C.c_size_t
    L.mxfp4_launch_count.restype = u64
    L.mxfp4_launch_count.argtypes = []
    L.mxfp4_scale_bytes.restype = sz
    L.mxfp4_scale_bytes.argtypes = [i64, i64]
    L.mxfp4_scale_offset.restype = sz
    L.mxfp4_scale_offset.argtypes = [i64, i64, i64]
    L.mxfp4_gemm_workspace_bytes.restype = sz
    L.mxfp4_gemm_workspace_bytes.argtypes = [i64, i64, i64]
    L.mxfp4_gemm_chain_mmas.restype = i64
    L.mxfp4_gemm_chain_mmas.argtypes = [i64, i64, i64]
    L.mxfp4_linear_workspace_bytes.restype = sz
    L.mxfp4_linear_workspace_bytes.argtypes = [i64, i64, i64]
    L.mxfp4_quantize.restype = i32
    L.mxfp4_quantize.argtypes = [vp, i64, i64, i64, CMat, C.POINTER(CQParams), vp, vp]
    L.mxfp4_quantize_t.restype = i32
    L.mxfp4_quantize_t.argtypes = [vp, C.POINTER(CMat), i64, i64, i64, CMat, C.POINTER(CQParams), vp, vp]
    L.mxfp4_quantize_2axis.restype = i32
    L.mxfp4_quantize_2axis.argtypes = [vp, i64, i64, i64, CMat, C.POINTER(CQParams), CMat, C.POINTER(CQParams), vp, vp]
    L.mxfp4_quantize_chain.restype = i32
    L.mxfp4_quantize_chain.argtypes = L.mxfp4_quantize_2axis.argtypes
    L.mxfp4_qema_quantize.restype = i32
    L.mxfp4_qema_quantize.argtypes = [vp, vp, C.c_float, i32, i64, i64, CMat, i32, C.POINTER(COsc), vp, vp]
    L.mxfp4_dequantize.restype = i32
    L.mxfp4_dequantize.argtypes = [CMat, vp, i64, vp]
    L.mxfp4_gemm.restype = i32
    L.mxfp4_gemm.argtypes = [CMat, CMat, vp, i64, i32, vp, vp, sz, vp, vp]
    L.mxfp4_gemm_quant.restype = i32
    L.mxfp4_gemm_quant.argtypes = [CMat, CMat, vp, C.POINTER(CEpilogue), vp, vp]
    L.mxfp4_gemm_static.restype = i32
    L.mxfp4_gemm_static.argtypes = [CMat, CMat, vp, i64, i32, vp, vp, vp]
    L.mxfp4_linear_fwd.restype = i32
    L.mxfp4_linear_fwd.argtypes = [vp, i64, i64, i64, vp, i64, vp, vp, i64, C.POINTER(CCtx), i32, vp, vp]
    L.mxfp4_linear_bwd.restype = i32
    L.mxfp4_linear_bwd.argtypes = [vp, i64, C.POINTER(CCtx), u64, i32, vp, i64, vp, i64, i32, vp, sz, vp, vp]
    L.mxfp4_gemm_wait_selftest.restype = i32
    L.mxfp4_gemm_wait_selftest.argtypes = [CMat, CMat, vp, i64, i32, vp, sz, C.c_uint32, vp, vp]
    L.mxfp4_quantize_wait_selftest.restype = i32
    L.mxfp4_quantize_wait_selftest.argtypes = [vp, i64, i64, i64, CMat, CMat, C.c_uint32, vp, vp]
    L.mxfp4_linear_fwd_ex.restype = i32
    L.mxfp4_linear_fwd_ex.argtypes = [vp, i64, i64, i64, vp, i64, vp, vp, i64, C.POINTER(CCtx), i32, C.POINTER(CEpilogue), vp, vp]
    L.mxfp4_linear_bwd_ex.restype = i32
    L.mxfp4_linear_bwd_ex.argtypes = [vp, i64, C.POINTER(CMat), C.POINTER(CMat), C.POINTER(CCtx), u64, i32, vp, i64, vp, i64, i32,
                                      C.POINTER(CEpilogue), vp, sz, vp, vp]
    L.mxfp4_quant_conf_hist.restype = i32
    L.mxfp4_quant_conf_hist.argtypes = [vp, i64, i64, i32, i32, vp, vp]
    L.mxfp4_change_sums.restype = i32
    L.mxfp4_change_sums.argtypes = [vp, vp, i64, vp, vp]
    L.mxfp4_change_sums_q.restype = i32
    L.mxfp4_change_sums_q.argtypes = [CMat, CMat, vp, vp]
    L.mxfp4_mma_issue_ceiling.restype = i32
    L.mxfp4_mma_issue_ceiling.argtypes = [i32, i32, vp, vp]
    L.mxfp4_qramp_detect.restype = i32
    L.mxfp4_qramp_detect.argtypes = [vp, vp, i64, C.c_float, i32, i32, vp, vp, vp]
    L.mxfp4_qramp_adamw.restype = i32
    L.mxfp4_qramp_adamw.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, C.POINTER(CAdamW), vp]
    _lib = L
    return L


def _check(fn, status):
    if status != 0:
        raise MxError(fn, status)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def launch_count():
    """Kernels the library has launched in this process so far (its own count, taken at the launch sites)."""
    return int(lib().mxfp4_launch_count())


def scale_bytes(rows, cols):
    return int(lib().mxfp4_scale_bytes(rows, cols))


def scale_offset(row, block, cols):
    return int(lib().mxfp4_scale_offset(row, block, cols))


class QMat:
    """A quantized matrix in device memory: packed E2M1 codes + E8M0 scales in tiled order."""

    def __init__(self, rows, cols, device="cuda", data=None, scales=None):
        self.rows, self.cols = int(rows), int(cols)
        self.data = data if data is not None else _new((self.rows, self.cols // 2), torch.uint8, device)
        nbytes = max(scale_bytes(self.rows, self.cols), 16)
        self.scales = scales if scales is not None else _new((nbytes,), torch.uint8, device)

    def c(self):
        return CMat(self.data.data_ptr(), self.scales.data_ptr(), self.rows, self.cols)

    def scales_linear(self):
        """Scale bytes gathered into [rows, cols/32] order (index arithmetic only; for inspection)."""
        nblk = self.cols // 32
        nblk4 = (nblk + 3) // 4
        r = torch.arange(self.rows, device=self.scales.device).view(-1, 1)
        b = torch.arange(nblk, device=self.scales.device).view(1, -1)
        off = ((r // 128) * nblk4 + b // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + b % 4
        return self.scales[off.reshape(-1)].view(self.rows, nblk)


def _qp(scale_mode, rounding, seed, stream_id):
    return CQParams(scale_mode, rounding, seed & 0xFFFFFFFFFFFFFFFF, stream_id, 0)


def _bf16_2d(x):
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    return x


def new_status(device="cuda"):
    return torch.zeros(1, dtype=torch.int32, device=device)


def quantize(x, scale_mode=SCALE_TRUNCATION_FREE, rounding=ROUND_NEAREST, seed=0, stream_id=0, out=None,
             dev_status=None):
    x = _bf16_2d(x)
    rows, cols = x.shape
    out = out if out is not None else QMat(rows, cols, x.device)
    qp = _qp(scale_mode, rounding, seed, stream_id)
    _check("mxfp4_quantize", lib().mxfp4_quantize(_ptr(x), rows, cols, x.stride(0), out.c(), C.byref(qp),
                                                  _ptr(dev_status), _stream()))
    return out


def quantize_t(src, scale_mode=SCALE_TRUNCATION_FREE, rounding=ROUND_NEAREST, seed=0, stream_id=0, out=None,
               dev_status=None):
    """Quantize along rows, emit the transposed matrix.  ``src`` is a bf16 tensor or a QMat (double quantization)."""
    qp = _qp(scale_mode, rounding, seed, stream_id)
    if isinstance(src, QMat):
        rows, cols = src.rows, src.cols
        out = out if out is not None else QMat(cols, rows, src.data.device)
        cm = src.c()
        st = lib().mxfp4_quantize_t(None, C.byref(cm), rows, cols, cols, out.c(), C.byref(qp), _ptr(dev_status), _stream())
    else:
        x = _bf16_2d(src)
        rows, cols = x.shape
        out = out if out is not None else QMat(cols, rows, x.device)
        st = lib().mxfp4_quantize_t(_ptr(x), None, rows, cols, x.stride(0), out.c(), C.byref(qp), _ptr(dev_status), _stream())
    _check("mxfp4_quantize_t", st)
    return out


def quantize_2axis(x, qp_row, qp_t, out=None, out_t=None, dev_status=None):
    """Both layouts from one read.  qp_* = (scale_mode, rounding, seed, stream_id)."""
    x = _bf16_2d(x)
    rows, cols = x.shape
    out = out if out is not None else QMat(rows, cols, x.device)
    out_t = out_t if out_t is not None else QMat(cols, rows, x.device)
    a, b = _qp(*qp_row), _qp(*qp_t)
    _check("mxfp4_quantize_2axis", lib().mxfp4_quantize_2axis(_ptr(x), rows, cols, x.stride(0), out.c(), C.byref(a),
                                                              out_t.c(), C.byref(b), _ptr(dev_status), _stream()))
    return out, out_t


def quantize_chain(x, seed, scale_mode=SCALE_TRUNCATION_FREE, rounding=ROUND_NEAREST, stream_id=0, rounding_t=ROUND_STOCHASTIC,
                   stream_id_t=6, out=None, out_t=None, dev_status=None):
    """out = Q(x) and out_t = Q(deq(out)^T) (double quantization) from one read of x; defaults: Q1 and Q6 of the linear layer."""
    x = _bf16_2d(x)
    rows, cols = x.shape
    out = out if out is not None else QMat(rows, cols, x.device)
    out_t = out_t if out_t is not None else QMat(cols, rows, x.device)
    a, b = _qp(scale_mode, rounding, seed, stream_id), _qp(scale_mode, rounding_t, seed, stream_id_t)
    _check("mxfp4_quantize_chain", lib().mxfp4_quantize_chain(_ptr(x), rows, cols, x.stride(0), out.c(), C.byref(a),
                                                              out_t.c(), C.byref(b), _ptr(dev_status), _stream()))
    return out, out_t


class OscState:
    """Oscillation-counter state of one weight (caller-owned device buffers)."""

    def __init__(self, w_prev, wq_prev, dist_w, dist_q):
        self.w_prev, self.wq_prev, self.dist_w, self.dist_q = w_prev, wq_prev, dist_w, dist_q

    def c(self):
        return COsc(self.w_prev.data_ptr(), self.wq_prev.c(), self.dist_w.data_ptr(), self.dist_q.data_ptr())


def qema_quantize(w, ema, beta=0.998, update_ema=True, scale_mode=SCALE_TRUNCATION_FREE, osc=None, out=None,
                  dev_status=None):
    w = _bf16_2d(w)
    assert w.is_contiguous() and ema.is_cuda and ema.dtype == torch.float32 and ema.is_contiguous() and ema.shape == w.shape
    n, k = w.shape
    out = out if out is not None else QMat(n, k, w.device)
    co = osc.c() if osc is not None else None
    _check("mxfp4_qema_quantize",
           lib().mxfp4_qema_quantize(_ptr(w), _ptr(ema), C.c_float(beta), int(bool(update_ema)), n, k, out.c(), scale_mode,
                                     C.byref(co) if co is not None else None, _ptr(dev_status), _stream()))
    return out


def dequantize(q):
    out = _new((q.rows, q.cols), torch.float32, q.data.device)
    _check("mxfp4_dequantize", lib().mxfp4_dequantize(q.c(), _ptr(out), q.cols, _stream()))
    return out


def gemm_workspace_bytes(m, n, kc):
    return int(lib().mxfp4_gemm_workspace_bytes(m, n, kc))


def gemm_chain_mmas(m, n, kc):
    """Longest accumulation chain (MMAs of 64 contraction elements) of the product's plan: the error bound depends on it."""
    return int(lib().mxfp4_gemm_chain_mmas(m, n, kc))


def linear_workspace_bytes(m, k, n):
    return int(lib().mxfp4_linear_workspace_bytes(m, k, n))


def gemm(a, b, out_dtype=OUT_BF16, bias=None, out=None, workspace=None, dev_status=None):
    """D[M, N] = deq(a)[M, kc] @ deq(b)[N, kc]^T."""
    dt = torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16
    out = out if out is not None else _new((a.rows, b.rows), dt, a.data.device)
    need = gemm_workspace_bytes(a.rows, b.rows, a.cols)
    if workspace is None and need:
        workspace = _new((need,), torch.uint8, a.data.device)
    _check("mxfp4_gemm", lib().mxfp4_gemm(a.c(), b.c(), _ptr(out), out.stride(0), out_dtype, _ptr(bias), _ptr(workspace),
                                          workspace.numel() if workspace is not None else 0, _ptr(dev_status), _stream()))
    return out


class Epilogue:
    """What mxfp4_gemm_quant does with the accumulator tile: Y = bf16(product + bias), Z = bf16(hook(Y)), and the
    quantizations of Z.  qp_* = (scale_mode, rounding, seed, stream_id); zq / zq_t: QMat to fill (None: not emitted);
    y / z: bf16 tensors to fill (None: not written); chain: zq_t re-quantizes deq(zq) (double quantization)."""

    def __init__(self, hook=HOOK_IDENTITY, aux=None, y=None, z=None, zq=None, qp_row=(0, 0, 0, 0), zq_t=None, qp_t=(0, 0, 0, 0), chain=False):
        self.hook, self.aux, self.y, self.z, self.zq, self.qp_row, self.zq_t, self.qp_t, self.chain = hook, aux, y, z, zq, qp_row, zq_t, qp_t, chain

    def c(self):
        none = CMat(None, None, 0, 0)
        return CEpilogue(self.hook, int(bool(self.chain)),
                         self.aux.data_ptr() if self.aux is not None else None, self.aux.stride(0) if self.aux is not None else 0,
                         self.y.data_ptr() if self.y is not None else None, self.y.stride(0) if self.y is not None else 0,
                         self.z.data_ptr() if self.z is not None else None, self.z.stride(0) if self.z is not None else 0,
                         self.zq.c() if self.zq is not None else none, _qp(*self.qp_row),
                         self.zq_t.c() if self.zq_t is not None else none, _qp(*self.qp_t))


def gemm_quant(a, b, epi, bias=None, dev_status=None):
    """The product deq(a) deq(b)^T with the next quantization fused into its epilogue (see Epilogue); fills the
    tensors / QMats named in ``epi``."""
    ce = epi.c()
    _check("mxfp4_gemm_quant", lib().mxfp4_gemm_quant(a.c(), b.c(), _ptr(bias), C.byref(ce), _ptr(dev_status), _stream()))
    return epi


def gemm_wait_selftest(a, b, dev_status, out_dtype=OUT_BF16, spin_limit=2048):
    """The kernels gemm() would launch for (a, b), with their loads withheld and every bounded wait limited to
    ``spin_limit`` polls: the waits run out, DEV_TIMEOUT is raised in ``dev_status`` and the kernels drain and return.
    The output is undefined and is thrown away."""
    dt = torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16
    out = _new((a.rows, b.rows), dt, a.data.device)
    need = gemm_workspace_bytes(a.rows, b.rows, a.cols)
    ws = _new((max(need, 16),), torch.uint8, a.data.device)
    _check("mxfp4_gemm_wait_selftest", lib().mxfp4_gemm_wait_selftest(a.c(), b.c(), _ptr(out), out.stride(0), out_dtype, _ptr(ws), ws.numel(),
                                                                      spin_limit, _ptr(dev_status), _stream()))


def quantize_wait_selftest(x, dev_status, spin_limit=2048):
    """The two-axis quantizer's kernel for ``x`` with its loads withheld: see gemm_wait_selftest."""
    x = _bf16_2d(x)
    rows, cols = x.shape
    out, out_t = QMat(rows, cols, x.device), QMat(cols, rows, x.device)
    _check("mxfp4_quantize_wait_selftest", lib().mxfp4_quantize_wait_selftest(_ptr(x), rows, cols, x.stride(0), out.c(), out_t.c(), spin_limit,
                                                                              _ptr(dev_status), _stream()))


STATIC_SCRATCH_BYTES = 16 << 20


def gemm_static(a, b, out, out_dtype=OUT_BF16, bias=None, dev_status=None):
    """gemm() for callers that must not allocate: ``out`` is required, the split-K scratch is the
    library's own fixed device array (STATIC_SCRATCH_BYTES; larger needs raise WORKSPACE_TOO_SMALL).
    Nothing is allocated here or in the library.  Calls on one GPU share the array: do not overlap them."""
    _check("mxfp4_gemm_static", lib().mxfp4_gemm_static(a.c(), b.c(), _ptr(out), out.stride(0), out_dtype, _ptr(bias),
                                                        _ptr(dev_status), _stream()))
    return out


class LinearCtx:
    """Forward operands kept for the backward pass.  With ``xq_t`` (a QMat [K, M]) and ``seed`` the forward pass also
    makes the backward operand Q6 of this step in its pass over X.  ``wq_t`` (a QMat [K, N]) is the backward operand Q4:
    made ahead by the caller with ``quantize_t(wq, rounding=ROUND_STOCHASTIC, seed=seed, stream_id=4)``, or written by
    ``linear_fwd`` itself when that is given the weight ``w`` (one pass over W then makes Q2 and Q4)."""

    def __init__(self, xq, wq, xq_t=None, seed=0, wq_t=None):
        self.xq, self.wq, self.xq_t, self.seed, self.wq_t = xq, wq, xq_t, seed, wq_t

    def c(self):
        none = CMat(None, None, 0, 0)
        t = self.xq_t.c() if self.xq_t is not None else none
        wt = self.wq_t.c() if self.wq_t is not None else none
        sd = self.seed & 0xFFFFFFFFFFFFFFFF
        return CCtx(self.xq.c(), self.wq.c(), t, sd, wt, sd)


def linear_fwd(x, w=None, wq=None, bias=None, scale_mode=SCALE_TRUNCATION_FREE, ctx=None, out=None, dev_status=None,
               bwd_seed=None, epi=None):
    """Y = Q1(X) Q2(W)^T.  Give ``w`` (bf16 [N, K]) or an already quantized ``wq`` (e.g. from qema_quantize).
    ``bwd_seed``: also make Q6 for the backward pass that will be called with this seed.
    ``x = None``: ``ctx.xq`` (and ``ctx.xq_t``) already hold the quantized input (written by the previous layer's
    epilogue).  ``epi`` (an Epilogue): the product runs with that quantizing epilogue, which names its own outputs;
    the first return value is then ``epi``."""
    if x is not None:
        x = _bf16_2d(x)
        m, k = x.shape
        dev = x.device
    else:
        m, k = ctx.xq.rows, ctx.xq.cols
        dev = ctx.xq.data.device
    if ctx is None:
        if wq is None:
            wq = QMat(w.shape[0], k, dev)
        ctx = LinearCtx(QMat(m, k, dev), wq)
        if bwd_seed is not None:
            ctx.xq_t, ctx.seed = QMat(k, m, dev), bwd_seed
    elif bwd_seed is not None:
        ctx.seed = bwd_seed
        if ctx.xq_t is None:
            ctx.xq_t = QMat(k, m, dev)
    n = ctx.wq.rows
    if epi is None:
        out = out if out is not None else _new((m, n), torch.bfloat16, dev)
    cc = ctx.c()
    if w is not None:
        w = _bf16_2d(w)
        assert w.is_contiguous()
    ce = epi.c() if epi is not None else None
    _check("mxfp4_linear_fwd_ex", lib().mxfp4_linear_fwd_ex(_ptr(x), x.stride(0) if x is not None else 0, m, k, _ptr(w), n, _ptr(bias),
                                                            _ptr(out) if epi is None else None, out.stride(0) if epi is None else 0,
                                                            C.byref(cc), scale_mode, C.byref(ce) if ce is not None else None,
                                                            _ptr(dev_status), _stream()))
    return (epi if epi is not None else out), ctx


def linear_bwd(dy, ctx, seed, scale_mode=SCALE_TRUNCATION_FREE, dw_dtype=OUT_FP32, dx=None, dw=None, workspace=None,
               dev_status=None, dyq=None, dyq_t=None, epi_dx=None):
    """dX = Q3(dY) Q4(Wq^T..), dW = Q5(dY^T) Q6(Xq)  (Eq. 4-5).
    ``dy = None``: ``dyq`` / ``dyq_t`` already hold Q3(dY) / Q5(dY^T) (written by the next layer's epilogue).
    ``epi_dx`` (an Epilogue): the input-gradient product runs with that quantizing epilogue; the first return value is
    then ``epi_dx``."""
    m, k, n = ctx.xq.rows, ctx.xq.cols, ctx.wq.rows
    dev = ctx.xq.data.device
    if dy is not None:
        dy = _bf16_2d(dy)
    if epi_dx is None:
        dx = dx if dx is not None else _new((m, k), torch.bfloat16, dev)
    dwt = torch.float32 if dw_dtype == OUT_FP32 else torch.bfloat16
    dw = dw if dw is not None else _new((n, k), dwt, dev)
    if workspace is None:
        workspace = _new((linear_workspace_bytes(m, k, n),), torch.uint8, dev)
    cc = ctx.c()
    ce = epi_dx.c() if epi_dx is not None else None
    cq, cqt = (dyq.c(), dyq_t.c()) if dy is None else (None, None)
    _check("mxfp4_linear_bwd_ex", lib().mxfp4_linear_bwd_ex(_ptr(dy), dy.stride(0) if dy is not None else 0,
                                                            C.byref(cq) if cq is not None else None, C.byref(cqt) if cqt is not None else None,
                                                            C.byref(cc), seed & 0xFFFFFFFFFFFFFFFF, scale_mode,
                                                            _ptr(dx) if epi_dx is None else None, dx.stride(0) if epi_dx is None else 0,
                                                            _ptr(dw), dw.stride(0), dw_dtype, C.byref(ce) if ce is not None else None,
                                                            _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream()))
    return (epi_dx if epi_dx is not None else dx), dw


def qramp_detect(dist_w, dist_q, k1=16.0, k2=5, n_max=255, out=None, oscillating=None):
    """Algorithm 2, OscillationDetection: the ramp factor n_w (uint8, same shape) of every element from its trajectory
    lengths, and (added to ``oscillating``, a one-element int64 device tensor) the number of elements with R_w > k1."""
    assert dist_w.dtype == torch.float32 and dist_q.dtype == torch.float32 and dist_w.is_contiguous() and dist_q.is_contiguous()
    n_w = out if out is not None else _new(tuple(dist_w.shape), torch.uint8, dist_w.device)
    if oscillating is None:
        oscillating = torch.zeros(1, dtype=torch.int64, device=dist_w.device)
    _check("mxfp4_qramp_detect", lib().mxfp4_qramp_detect(_ptr(dist_w), _ptr(dist_q), dist_w.numel(), k1, k2, n_max, _ptr(n_w),
                                                          _ptr(oscillating), _stream()))
    return n_w, oscillating


def qramp_adamw(w, grad, m, v, acc, cnt, n_w=None, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.05, step=1,
                w_bf16=None):
    """One step of the customized AdamW of Algorithm 2, in place on the FP32 tensors w, m, v, acc and the uint8 cnt;
    ``step`` is the global step count of the bias corrections; ``w_bf16`` (optional) receives the bf16 copy of every
    weight that changed."""
    for t in (w, grad, m, v, acc):
        assert t.dtype == torch.float32 and t.is_contiguous()
    assert cnt.dtype == torch.uint8 and cnt.is_contiguous()
    hp = CAdamW(lr, beta1, beta2, eps, weight_decay, 1.0 - beta1 ** step, 1.0 - beta2 ** step)
    _check("mxfp4_qramp_adamw", lib().mxfp4_qramp_adamw(_ptr(w), _ptr(w_bf16), _ptr(grad), _ptr(m), _ptr(v), _ptr(acc), _ptr(cnt),
                                                        _ptr(n_w), w.numel(), C.byref(hp), _stream()))


def quant_conf_hist(w, bins=20, scale_mode=SCALE_TRUNCATION_FREE, out=None):
    """Histogram (int64[bins], added to ``out``) of the quantization confidence (Sec. 4.2) of the bf16 weight matrix w."""
    w = _bf16_2d(w)
    hist = out if out is not None else torch.zeros(bins, dtype=torch.int64, device=w.device)
    assert w.is_contiguous()
    _check("mxfp4_quant_conf_hist", lib().mxfp4_quant_conf_hist(_ptr(w), w.shape[0], w.shape[1], scale_mode, bins, _ptr(hist), _stream()))
    return hist


def change_sums(cur, prev, out=None):
    """(sum (cur - prev)^2, sum prev^2) as a float64[2] device tensor (added to ``out``): one term of the rate of change of
    App. A.3.  cur / prev: two bf16 tensors of one shape, or two QMat of one shape."""
    dev = cur.data.device if isinstance(cur, QMat) else cur.device
    res = out if out is not None else torch.zeros(2, dtype=torch.float64, device=dev)
    if isinstance(cur, QMat):
        _check("mxfp4_change_sums_q", lib().mxfp4_change_sums_q(cur.c(), prev.c(), _ptr(res), _stream()))
    else:
        assert cur.dtype == torch.bfloat16 and prev.dtype == torch.bfloat16 and cur.is_contiguous() and prev.is_contiguous()
        assert cur.shape == prev.shape
        _check("mxfp4_change_sums", lib().mxfp4_change_sums(_ptr(cur), _ptr(prev), cur.numel(), _ptr(res), _stream()))
    return res


def mma_issue_ceiling(bn=256, iters=2000, reps=5):
    """TFLOP/s of an MMA-only loop (128 x bn x 64 block-scaled MXFP4 MMAs on shared-memory resident operands) over all
    SMs: the tensor pipe's ceiling on this GPU, best of ``reps`` timings with CUDA events."""
    st = new_status()
    sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    best = 0.0
    for _ in range(reps + 1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        _check("mxfp4_mma_issue_ceiling", lib().mxfp4_mma_issue_ceiling(bn, iters, _ptr(st), _stream()))
        e1.record()
        e1.synchronize()
        t = e0.elapsed_time(e1) * 1e-3
        best = max(best, sms * iters * 4 * 2.0 * 128 * bn * 64 / t / 1e12)
    if int(st.item()) != 0:
        raise RuntimeError("device status %d in the MMA ceiling loop" % int(st.item()))
    return best
