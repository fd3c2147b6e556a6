"""Time one kernel of the library on synthetic device-resident data (CUDA events, L2-sized inputs).

  python -m paper_2502_20853_b200.microbench --kernel quantize_2axis --rows 16384 --cols 4096 --iters 5
  python -m paper_2502_20853_b200.microbench --kernel gemm --m 8192 --n 4096 --k 1024 --out bf16

Kernels: quantize, quantize_sr, quantize_t, quantize_t_sr, quantize_2axis, quantize_chain, requant (double quantization), qema,
qema_osc, qramp_detect, qramp_adamw (all elements update every step), qramp_adamw_ramped (a tenth of the elements
accumulate over 6 steps), quant_conf_hist, change_sums, mma_ceiling (MMA-only loop, --n = tile width), gemm.  Prints one line with the mean time and the algorithmic GB/s or TFLOP/s.
"""
import argparse

import torch

from . import binding as mx

Q = 0.5 + 1.0 / 32.0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", required=True)
    ap.add_argument("--rows", type=int, default=16384)
    ap.add_argument("--cols", type=int, default=4096)
    ap.add_argument("--m", type=int, default=8192)
    ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--k", type=int, default=1024)
    ap.add_argument("--out", default="bf16", choices=["bf16", "fp32"])
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args()
    mx.lib()
    torch.manual_seed(0)
    R, C = a.rows, a.cols
    flops = 0.0
    if a.kernel == "mma_ceiling":
        bn = a.n if a.n in (128, 192, 256) else 256
        print("mma_ceiling: 128 x %d x 64 kind::mxf4 MMAs from shared memory, all SMs: %.1f TFLOP/s" % (bn, mx.mma_issue_ceiling(bn=bn)))
        return
    if a.kernel in ("gemm_quant_gelu_chain", "gemm_quant_mul_2axis", "gemm_quant_chain"):
        # the product with the fused quantizing epilogue: forward (Y kept, GELU, Q1 + Q6 of the next layer), backward
        # (times the activation's derivative, Q3 + Q5 of the previous layer), or the plain chain with Z kept
        A, B = mx.QMat(a.m, a.k), mx.QMat(a.n, a.k)
        A.data.random_(0, 256)
        B.data.random_(0, 256)
        A.scales.random_(124, 130)
        B.scales.random_(124, 130)
        y = torch.empty((a.m, a.n), dtype=torch.bfloat16, device="cuda")
        zq, zqt = mx.QMat(a.m, a.n), mx.QMat(a.n, a.m)
        st = mx.new_status()
        if a.kernel == "gemm_quant_gelu_chain":
            epi = mx.Epilogue(hook=mx.HOOK_GELU, y=y, zq=zq, zq_t=zqt, qp_t=(0, 1, 1, 6), chain=True)
            out_bytes = 2 + 2 * Q
        elif a.kernel == "gemm_quant_chain":
            epi = mx.Epilogue(z=y, zq=zq, zq_t=zqt, qp_t=(0, 1, 1, 6), chain=True)
            out_bytes = 2 + 2 * Q
        else:
            aux = torch.rand((a.m, a.n), device="cuda").to(torch.bfloat16)
            epi = mx.Epilogue(hook=mx.HOOK_MULTIPLY, aux=aux, zq=zq, qp_row=(0, 1, 1, 3), zq_t=zqt, qp_t=(0, 1, 1, 5))
            out_bytes = 2 + 2 * Q          # the second factor read, two sets of codes written
        fn = lambda: mx.gemm_quant(A, B, epi, dev_status=st)  # noqa: E731
        nbytes = Q * a.k * (a.m + a.n) + out_bytes * a.m * a.n
        flops = 2.0 * a.m * a.n * a.k
    elif a.kernel == "gemm":
        A, B = mx.QMat(a.m, a.k), mx.QMat(a.n, a.k)
        A.data.random_(0, 256)
        B.data.random_(0, 256)
        A.scales.random_(120, 134)
        B.scales.random_(120, 134)
        od = mx.OUT_FP32 if a.out == "fp32" else mx.OUT_BF16
        out = torch.empty((a.m, a.n), dtype=torch.float32 if od else torch.bfloat16, device="cuda")
        ws = torch.empty(max(16, mx.gemm_workspace_bytes(a.m, a.n, a.k)), dtype=torch.uint8, device="cuda")
        st = mx.new_status()
        fn = lambda: mx.gemm(A, B, out_dtype=od, out=out, workspace=ws, dev_status=st)  # noqa: E731
        nbytes = Q * a.k * (a.m + a.n) + out.element_size() * a.m * a.n
        flops = 2.0 * a.m * a.n * a.k
    else:
        x = torch.randn(R, C, device="cuda", dtype=torch.bfloat16)
        q, qt = mx.QMat(R, C), mx.QMat(C, R)
        el = R * C
        if a.kernel == "quantize":
            fn, nbytes = (lambda: mx.quantize(x, out=q)), el * (2 + Q)
        elif a.kernel == "quantize_sr":
            fn, nbytes = (lambda: mx.quantize(x, rounding=1, seed=1, stream_id=3, out=q)), el * (2 + Q)
        elif a.kernel == "quantize_t":
            fn, nbytes = (lambda: mx.quantize_t(x, out=qt)), el * (2 + Q)
        elif a.kernel == "quantize_t_sr":
            fn, nbytes = (lambda: mx.quantize_t(x, rounding=1, seed=1, stream_id=5, out=qt)), el * (2 + Q)
        elif a.kernel == "quantize_2axis":
            fn, nbytes = (lambda: mx.quantize_2axis(x, (0, 1, 1, 3), (0, 1, 1, 5), out=q, out_t=qt)), el * (2 + 2 * Q)
        elif a.kernel == "quantize_2axis_rne":
            fn, nbytes = (lambda: mx.quantize_2axis(x, (0, 0, 0, 0), (0, 0, 0, 0), out=q, out_t=qt)), el * (2 + 2 * Q)
        elif a.kernel == "quantize_chain":
            fn, nbytes = (lambda: mx.quantize_chain(x, seed=1, out=q, out_t=qt)), el * (2 + 2 * Q)
        elif a.kernel == "requant":
            mx.quantize(x, out=q)
            fn, nbytes = (lambda: mx.quantize_t(q, rounding=1, seed=1, stream_id=6, out=qt)), el * 2 * Q
        elif a.kernel in ("qema", "qema_osc"):
            ema = x.float().contiguous()
            osc = None
            if a.kernel == "qema_osc":
                osc = mx.OscState(x.clone(), mx.quantize(x), torch.zeros_like(ema), torch.zeros_like(ema))
            fn = lambda: mx.qema_quantize(x, ema, out=q, osc=osc)  # noqa: E731
            nbytes = el * (2 + 8 + Q + ((2 + 2 + 2 * Q + 16) if osc is not None else 0))
        elif a.kernel == "qramp_detect":
            dw, dq = torch.rand(el, device="cuda") + 0.1, torch.rand(el, device="cuda") * 40
            nw, osc = torch.empty(el, dtype=torch.uint8, device="cuda"), torch.zeros(1, dtype=torch.int64, device="cuda")
            fn, nbytes = (lambda: mx.qramp_detect(dw, dq, out=nw, oscillating=osc)), el * (4 + 4 + 1)
        elif a.kernel in ("qramp_adamw", "qramp_adamw_ramped"):
            w, g = x.float().reshape(-1).contiguous() * 0.02, torch.randn(el, device="cuda") * 1e-3
            m, v, acc = torch.zeros_like(w), torch.zeros_like(w), torch.zeros_like(w)
            cnt, wb = torch.zeros(el, dtype=torch.uint8, device="cuda"), x.reshape(-1).clone()
            nw = None
            if a.kernel == "qramp_adamw_ramped":
                nw = torch.where(torch.rand(el, device="cuda") < 0.1, 6, 1).to(torch.uint8)
            fn = lambda: mx.qramp_adamw(w, g, m, v, acc, cnt, nw, w_bf16=wb)  # noqa: E731
            # every element: read w, grad, m, v, acc (4 each) + cnt (+ n_w), write acc + cnt; updated ones: write w, m, v, bf16
            nbytes = el * (20 + 1 + (1 if nw is not None else 0) + 4 + 1 + 14)
        elif a.kernel == "quant_conf_hist":
            w, hist = x * 0.02, torch.zeros(20, dtype=torch.int64, device="cuda")
            fn, nbytes = (lambda: mx.quant_conf_hist(w, bins=20, out=hist)), el * 2
        elif a.kernel == "change_sums":
            y, res = x + 0.01, torch.zeros(2, dtype=torch.float64, device="cuda")
            fn, nbytes = (lambda: mx.change_sums(x, y, out=res)), el * 4
        else:
            raise SystemExit("unknown kernel " + a.kernel)
    for _ in range(a.warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    t = e0.elapsed_time(e1) * 1e-3 / a.iters
    msg = "%s: %.2f us  %.1f GB/s (algorithmic)" % (a.kernel, t * 1e6, nbytes / t / 1e9)
    if flops:
        msg += "  %.1f TFLOP/s" % (flops / t / 1e12)
    print(msg)


if __name__ == "__main__":
    main()
