"""Helpers shared by the GPU parity tests: tensor conversion between the oracle's numpy world and torch."""
import numpy as np
import torch

import workloads


def to_dev_bf16(a: np.ndarray) -> torch.Tensor:
    """float32 numpy array of bf16-exact values -> bf16 CUDA tensor with the same values."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    tb = t.to(torch.bfloat16)
    assert torch.equal(tb.float(), t) or np.isnan(a).any()
    return tb.cuda()


def qmat_to_numpy(q):
    """(packed [rows, cols/2], scales [rows, cols/32]) of a device QMat as numpy uint8."""
    return q.data.cpu().numpy(), q.scales_linear().cpu().numpy()


def numpy_to_qmat(mx, packed: np.ndarray, scales: np.ndarray):
    """Build a device QMat from oracle-format arrays (scales get tiled; padding = 0x7F)."""
    rows, half = packed.shape
    cols = half * 2
    q = mx.QMat(rows, cols, "cuda")
    q.data.copy_(torch.from_numpy(np.ascontiguousarray(packed)))
    nblk = cols // 32
    nblk4 = (nblk + 3) // 4
    buf = np.full(q.scales.numel(), 0x7F, dtype=np.uint8)
    r = np.arange(rows).reshape(-1, 1)
    b = np.arange(nblk).reshape(1, -1)
    off = ((r // 128) * nblk4 + b // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + b % 4
    buf[off.reshape(-1)] = scales.reshape(-1)
    q.scales.copy_(torch.from_numpy(buf))
    return q


def assert_qmat_equal(q, packed_ref, scales_ref, what=""):
    p, s = qmat_to_numpy(q)
    bad_s = np.argwhere(s != scales_ref)
    assert bad_s.size == 0, "%s: %d scale bytes differ, first at %s: got %d want %d" % (
        what, len(bad_s), bad_s[0], s[tuple(bad_s[0])], scales_ref[tuple(bad_s[0])])
    bad_p = np.argwhere(p != packed_ref)
    assert bad_p.size == 0, "%s: %d packed bytes differ, first at %s: got %#x want %#x" % (
        what, len(bad_p), bad_p[0], p[tuple(bad_p[0])], packed_ref[tuple(bad_p[0])])


def check_gemm_bound(d_gpu: np.ndarray, d_ref: np.ndarray, t_ref: np.ndarray, bf16_out: bool, what="", factor=1.0):
    """|err| <= factor * 2^-20 * sum|a*b| per element; a bf16 output must be the rounding of a value inside that band.
    factor = 1 is the tolerance of the configurations; the library's general bound for chains of more than 8 MMAs into
    one accumulator is max(1, chain / 8) (see mxfp4_gemm in the header)."""
    tol = t_ref * 2.0 ** -20 * factor
    d_gpu = d_gpu.astype(np.float64)
    if bf16_out:
        lo = workloads.round_to_bf16((d_ref - tol).astype(np.float32)).astype(np.float64)
        hi = workloads.round_to_bf16((d_ref + tol).astype(np.float32)).astype(np.float64)
        lo = np.minimum(lo, d_ref - tol)
        hi = np.maximum(hi, d_ref + tol)
        ok = (d_gpu >= lo) & (d_gpu <= hi)
    else:
        ok = np.abs(d_gpu - d_ref) <= tol
    if not ok.all():
        idx = np.argwhere(~ok)
        i = tuple(idx[0])
        raise AssertionError("%s: %d of %d outside the bound; first %s: got %r want %r tol %r" % (
            what, len(idx), ok.size, i, d_gpu[i], d_ref[i], tol[i]))
