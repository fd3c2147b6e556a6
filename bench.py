#!/usr/bin/env python
"""Benchmark of the MXFP4 quantized linear layer, forward + backward (Eq. 3-5), on B200.

One "step" = the whole hot path over one batch of the DeiT-Small MLP pair (fc1 384->1536, fc2 1536->384,
25216 tokens): per layer the Q-EMA weight quantizer (with EMA update), Q1 + GEMM-1 (forward),
Q3/Q5 (one pass over dY), Q4, Q6, GEMM-2, GEMM-3 (backward).  Metric: useful TFLOP/s = 6*M*N*K per layer / time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads  # noqa: E402

METRIC = "mxfp4_linear_fwd_bwd_tflops"
UNIT = "TFLOP/s"
Q = 0.5 + 1.0 / 32.0  # bytes per MXFP4 element (packed nibble + scale share)


def source_digest():
    """Digest of the CUDA sources of the profiled kernels (the quantizers and the GEMMs): ncu traffic figures are only
    quoted while those kernels are the ones that were profiled."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2502_20853_b200", "csrc")
    for f in ("common.cuh", "gemm.cu", "quantize.cu"):
        with open(os.path.join(d, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def read_traffic(kernel_key):
    """DRAM bytes per launch of one kernel from the committed ncu capture (profiles/traffic.json), or None when there is
    no capture for it or the sources have changed since."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(p):
        return None
    with open(p) as f:
        d = json.load(f)
    if d.get("source_digest") != source_digest():
        return None
    return d.get("dram_bytes_per_launch", {}).get(kernel_key)


def read_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return dict(hbm=float(d["hbm_gbs"]), bf16=float(d["bf16_tflops"]), bf16_sustained=float(d["bf16_tflops_sustained"]),
                    source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx_, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx_.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx_) if mx_ else None,
                    power_w_max=max(power) if power else None, samples=len(sm), reasons=sorted(reasons))


def layer_flops(L, rows=None):
    m = L.M if rows is None else rows
    return 6.0 * m * L.N * L.K


# ---------------------------------------------------------------------------------------------------
# reference arm / cpu_baseline: the oracle, as it stands, on the host cores, on a bounded sample
# ---------------------------------------------------------------------------------------------------
def oracle_step(layers_data, sample_rows):
    import oracle as orc
    for (L, x, w, dy, ema, seed) in layers_data:
        f = orc.linear_fwd(x, w, ema=ema if L.qema else None, beta=0.998, want_bound=False)
        orc.linear_bwd(dy, f["xq"], f["wq"], seed, want_bound=False)


def oracle_inputs(config, sample_rows):
    data = []
    for li, L in enumerate(workloads.CONFIGS[config]):
        _, x, w, dy = workloads.make_layer(config, li, rows=sample_rows)
        data.append((L, x, w, dy, w.astype(np.float32).copy(), workloads.sr_seed(config, li)))
    return data


def time_oracle(config, sample_rows, steps, warmup):
    import oracle as orc
    orc.lib()
    data = oracle_inputs(config, sample_rows)
    for _ in range(warmup):
        oracle_step(data, sample_rows)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(data, sample_rows)
    dt = (time.perf_counter() - t0) / steps
    flops = sum(layer_flops(L, sample_rows) for L in workloads.CONFIGS[config])
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    return dict(value=flops / dt / 1e12, seconds_per_step=dt, cores=cores, flops=flops)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample_rows = 1024
    r = time_oracle(args.config, sample_rows, max(1, args.steps), max(0, min(args.warmup, 1)))
    sample = "config %d layers at %d of their token rows (all quantizers + 3 FP64 products per layer)" % (args.config, sample_rows)
    line = dict(impl="reference", metric=METRIC, value=r["value"], unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=r["seconds_per_step"] * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload="config%d: %s" % (args.config, "+".join(L.name for L in workloads.CONFIGS[args.config])),
                            sample=sample),
                cpu_baseline=dict(value=r["value"], unit=UNIT, cores=r["cores"], kind="oracle", sample=sample),
                e2e=dict(value=r["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------------
def max_over_ranks(values, device):
    """The replicas run independently; what is reported is the slowest one: element-wise maximum over the ranks of the
    process group (the values themselves when there is no group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


class LayerState:
    """Device-resident tensors and scratch of one linear layer."""

    def __init__(self, mx, torch, config, li):
        L, x, w, dy = workloads.make_layer(config, li)
        self.L = L
        bf = lambda a: torch.from_numpy(a).to(torch.bfloat16).cuda()  # noqa: E731
        self.host = dict(x=torch.from_numpy(x).to(torch.bfloat16).pin_memory(), w=torch.from_numpy(w).to(torch.bfloat16).pin_memory(),
                         dy=torch.from_numpy(dy).to(torch.bfloat16).pin_memory())
        self.x, self.w, self.dy = bf(x), bf(w), bf(dy)
        self.ema = self.w.float().contiguous()
        self.seed = workloads.sr_seed(config, li)
        self.wq = mx.QMat(L.N, L.K)
        self.wq_t = mx.QMat(L.K, L.N)
        self.ctx = mx.LinearCtx(mx.QMat(L.M, L.K), self.wq, xq_t=mx.QMat(L.K, L.M), seed=self.seed, wq_t=self.wq_t)
        self.weights_ready = torch.cuda.Event()
        self.ev_in, self.ev_done, self.ev_copied = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()
        self.y = torch.empty((L.M, L.N), dtype=torch.bfloat16, device="cuda")
        self.dx = torch.empty((L.M, L.K), dtype=torch.bfloat16, device="cuda")
        self.dw = torch.empty((L.N, L.K), dtype=torch.float32, device="cuda")
        self.ws = torch.empty(mx.linear_workspace_bytes(L.M, L.K, L.N), dtype=torch.uint8, device="cuda")
        self.host_out = dict(y=torch.empty((L.M, L.N), dtype=torch.bfloat16).pin_memory(),
                             dx=torch.empty((L.M, L.K), dtype=torch.bfloat16).pin_memory(),
                             dw=torch.empty((L.N, L.K), dtype=torch.float32).pin_memory())

    def weight_step(self, mx, status):
        """The weight side of a step: Q2 (Q-EMA with its EMA update, or round to nearest) and, from it, the backward
        operand Q4.  It depends on the weight alone, so the benchmark runs it on a second stream beside the activation
        quantizers."""
        if self.L.qema:
            mx.qema_quantize(self.w, self.ema, beta=0.998, update_ema=True, out=self.wq, dev_status=status)
        else:
            mx.quantize(self.w, out=self.wq, dev_status=status)
        mx.quantize_t(self.wq, rounding=1, seed=self.seed, stream_id=4, out=self.wq_t, dev_status=status)

    def step(self, mx, status):
        mx.linear_fwd(self.x, wq=self.wq, ctx=self.ctx, out=self.y, dev_status=status)
        mx.linear_bwd(self.dy, self.ctx, self.seed, dx=self.dx, dw=self.dw, workspace=self.ws, dev_status=status)

    def copy_in(self):
        self.x.copy_(self.host["x"], non_blocking=True)
        self.w.copy_(self.host["w"], non_blocking=True)
        self.dy.copy_(self.host["dy"], non_blocking=True)

    def copy_out(self):
        self.host_out["y"].copy_(self.y, non_blocking=True)
        self.host_out["dx"].copy_(self.dx, non_blocking=True)
        self.host_out["dw"].copy_(self.dw, non_blocking=True)

    def io_bytes(self):
        h2d = sum(t.numel() * t.element_size() for t in self.host.values())
        d2h = sum(t.numel() * t.element_size() for t in self.host_out.values())
        return h2d, d2h


def kernel_breakdown(mx, torch, layers, flush, reps=5):
    """Per-kernel device time (CUDA events on the launching stream, L2 flushed before every launch)
    and algorithmic bytes / flops of each launch of the step."""
    out = []

    def timed(name, fn, alg_bytes, flops, bound):
        ts = []
        for _ in range(reps):
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e-3)
        t = float(np.mean(ts[1:])) if len(ts) > 1 else ts[0]
        out.append(dict(kernel=name, seconds=t, alg_bytes=alg_bytes, flops=flops, bound=bound))

    for S in layers:
        L = S.L
        M, K, N = L.M, L.K, L.N
        tag = L.name
        if L.qema:
            timed(tag + ":qema", lambda: mx.qema_quantize(S.w, S.ema, out=S.wq), N * K * (2 + 4 + 4 + Q), 0, "hbm")
        else:
            timed(tag + ":quantize_w", lambda: mx.quantize(S.w, out=S.wq), N * K * (2 + Q), 0, "hbm")
        # Q1 and Q6 (the double quantization of Q1's result) in one pass over X
        timed(tag + ":quantize_x_q1_q6", lambda: mx.quantize_chain(S.x, seed=S.seed, out=S.ctx.xq, out_t=S.ctx.xq_t), M * K * (2 + 2 * Q), 0, "hbm")
        timed(tag + ":gemm_y", lambda: mx.gemm(S.ctx.xq, S.wq, out=S.y), Q * K * (M + N) + 2 * M * N, 2.0 * M * N * K, "tensor")
        dyq, dyq_t = mx.QMat(M, N), mx.QMat(N, M)
        wq_t, xq_t = mx.QMat(K, N), S.ctx.xq_t
        sr = lambda s: (0, 1, S.seed, s)  # noqa: E731
        timed(tag + ":quantize_2axis_dy", lambda: mx.quantize_2axis(S.dy, sr(3), sr(5), out=dyq, out_t=dyq_t), M * N * (2 + 2 * Q), 0, "hbm")
        timed(tag + ":requant_w", lambda: mx.quantize_t(S.wq, rounding=1, seed=S.seed, stream_id=4, out=wq_t), N * K * 2 * Q, 0, "hbm")
        timed(tag + ":gemm_dx", lambda: mx.gemm(dyq, wq_t, out=S.dx), Q * N * (M + K) + 2 * M * K, 2.0 * M * N * K, "tensor")
        ws = torch.empty(max(16, mx.gemm_workspace_bytes(N, K, M)), dtype=torch.uint8, device="cuda")
        timed(tag + ":gemm_dw", lambda: mx.gemm(dyq_t, xq_t, out_dtype=mx.OUT_FP32, out=S.dw, workspace=ws),
              Q * M * (N + K) + 4 * N * K, 2.0 * M * N * K, "tensor")
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2502_20853_b200 as mx
    from paper_2502_20853_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    mx.lib()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    peaks = read_peaks()
    cfg_layers = workloads.CONFIGS[args.config]
    layers = [LayerState(mx, torch, args.config, li) for li in range(len(cfg_layers))]
    status = mx.new_status()
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")  # > 126 MB L2

    def flush():
        flush_buf.fill_(1)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    graph = None
    weight_stream = torch.cuda.Stream()

    def one_step():
        """One training step of every layer, inputs resident in HBM: the weight quantizers on their own stream, forward
        and backward on the current one, which waits for each layer's weights before that layer's forward pass."""
        main = torch.cuda.current_stream()
        weight_stream.wait_stream(main)
        with torch.cuda.stream(weight_stream):
            for S in layers:
                S.weight_step(mx, status)
                S.weights_ready.record(weight_stream)
        for S in layers:
            main.wait_event(S.weights_ready)
            S.step(mx, status)
        main.wait_stream(weight_stream)

    h2d_stream, d2h_stream = torch.cuda.Stream(), torch.cuda.Stream()

    def run_e2e(n):
        """n end-to-end steps timed as one block: every step copies its inputs from pinned host memory and its results
        back, as a training loop does it: the copies of one step overlap the compute and the copies of its neighbours
        (the next step's inputs travel while this step's results go back; the two directions have their own engines).
        An input buffer is refilled only after the step that reads it has finished, an output buffer is overwritten only
        after its copy to the host has."""
        main = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(main)
        h2d_stream.wait_stream(main)
        d2h_stream.wait_stream(main)
        for _ in range(n):
            for S in layers:
                h2d_stream.wait_event(S.ev_done)          # the previous step has finished reading these inputs
                with torch.cuda.stream(h2d_stream):
                    S.copy_in()
                    S.ev_in.record(h2d_stream)
            for S in layers:
                main.wait_event(S.ev_in)
                main.wait_event(S.ev_copied)              # the previous step's results have left the output buffers
                weight_stream.wait_stream(main)
                with torch.cuda.stream(weight_stream):
                    S.weight_step(mx, status)
                    S.weights_ready.record(weight_stream)
                main.wait_event(S.weights_ready)
                S.step(mx, status)
                S.ev_done.record(main)
                d2h_stream.wait_event(S.ev_done)
                with torch.cuda.stream(d2h_stream):
                    S.copy_out()
                    S.ev_copied.record(d2h_stream)
        main.wait_stream(h2d_stream)
        main.wait_stream(d2h_stream)
        main.wait_stream(weight_stream)
        e1.record(main)
        e1.synchronize()
        return e0.elapsed_time(e1) * 1e-3

    def run_steps(n):
        total = 0.0
        for _ in range(n):
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            if graph is not None:
                graph.replay()
            else:
                one_step()
            e1.record()
            e1.synchronize()
            total += e0.elapsed_time(e1) * 1e-3
        return total

    # one eager step first (function attributes, lazy module loading), then the step is captured in a CUDA graph:
    # the launch sequence of a training step is fixed, so replaying it takes the host out of the timed region
    run_steps(1)
    launches_per_step = 0
    if not args.no_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            one_step()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        l0 = binding.LAUNCHES
        with torch.cuda.graph(graph):
            one_step()
        launches_per_step = binding.LAUNCHES - l0

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # warm-up; kept going for at least 1.5 s so that the clock sampler has samples under load before timing starts
    t_warm = time.perf_counter()
    run_steps(max(3, args.warmup))
    while time.perf_counter() - t_warm < 1.5:
        run_steps(3)
    barrier()
    launches0 = binding.LAUNCHES
    total = run_steps(args.steps)
    launches = (binding.LAUNCHES - launches0) if graph is None else launches_per_step * args.steps
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    run_e2e(2)
    barrier()
    total_e2e = run_e2e(args.steps)
    barrier()
    if int(status.item()) != 0:
        raise RuntimeError("device status %d during the benchmark" % int(status.item()))

    total, total_e2e = max_over_ranks([total, total_e2e], "cuda")
    flops_step = sum(layer_flops(L) for L in cfg_layers) * world
    value = flops_step * args.steps / total / 1e12
    value_e2e = flops_step * args.steps / total_e2e / 1e12
    h2d = sum(S.io_bytes()[0] for S in layers)
    d2h = sum(S.io_bytes()[1] for S in layers)

    if rank == 0:
        kb = kernel_breakdown(mx, torch, layers, flush)
        ksum = sum(k["seconds"] for k in kb)
        for k in kb:
            k["share"] = k["seconds"] / ksum
            k["gbs"] = k["alg_bytes"] / k["seconds"] / 1e9
            k["tflops"] = k["flops"] / k["seconds"] / 1e12
        dom = max(kb, key=lambda k: k["seconds"])
        fp4_peak = 4.0 * peaks["bf16"]  # dense FP4 = 4 x dense bf16 (the ratio the paper quotes), burst figure: kernel timed alone
        if dom["bound"] == "hbm":
            roof = dict(bound="hbm", kernel=dom["kernel"], achieved=dom["gbs"], peak=peaks["hbm"], unit="GB/s",
                        frac=dom["gbs"] / peaks["hbm"], traffic=read_traffic(dom["kernel"]), peak_source=peaks["source"])
        else:
            roof = dict(bound="tensor", kernel=dom["kernel"], achieved=dom["tflops"], peak=fp4_peak, unit="TFLOP/s",
                        frac=dom["tflops"] / fp4_peak, traffic=read_traffic(dom["kernel"]), peak_source=peaks["source"] + " bf16 x 4")
        cpu = time_oracle(args.config, 4096, 1, 0)
        sample = "config %d layers at 4096 of their %d token rows (all quantizers + 3 FP64 products per layer), 1 pass" % (
            args.config, cfg_layers[0].M)
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(3, args.warmup),
                    ms_per_step=total / args.steps * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="mxfp4 (e2m1 x e8m0), f32 accumulate", data="synthetic",
                    config=dict(workload="config%d: %s" % (args.config, " + ".join(
                        "%s [M=%d,K=%d,N=%d]" % (L.name, L.M, L.K, L.N) for L in cfg_layers)),
                        l2="flushed between steps (256 MB write)", qema=True, replicas=world,
                        launch="eager" if graph is None else "CUDA graph replay of one step", streams="weight quantizers (Q2 by Q-EMA, Q4) on a second stream beside the activation quantizers"),
                    clocks=clocks,
                    e2e=dict(value=value_e2e, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                             ms_per_step=total_e2e / args.steps * 1e3,
                             note="steps timed as one block; every step copies all inputs in from pinned host memory and all "
                                  "results out; copies of neighbouring steps overlap on their own streams; inputs (196 MB per "
                                  "step for config 2) exceed the L2"),
                    gpu_launches=launches, roofline=roof,
                    cpu_baseline=dict(value=cpu["value"], unit=UNIT, cores=cpu["cores"], kind="oracle", sample=sample),
                    kernels=[dict(kernel=k["kernel"], us=round(k["seconds"] * 1e6, 2), share=round(k["share"], 4),
                                  gbs=round(k["gbs"], 1), tflops=round(k["tflops"], 1), bound=k["bound"]) for k in kb],
                    peaks=dict(hbm_gbs=peaks["hbm"], bf16_tflops=peaks["bf16"], fp4_tflops_proxy=fp4_peak, source=peaks["source"],
                               fp4_mma_issue_ceiling_tflops=round(mx.mma_issue_ceiling(bn=256), 1),
                               fp4_mma_issue_ceiling_note="measured here: MMA-only loop, 128x256x64 kind::mxf4, operands resident in shared memory"))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=sorted(workloads.CONFIGS))
    ap.add_argument("--no-graph", action="store_true", help="launch every step from the host instead of replaying a CUDA graph")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
