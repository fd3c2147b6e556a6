#!/usr/bin/env python
"""Benchmark of the MXFP4 quantized linear layer, forward + backward (Eq. 3-5), on B200.

One "step" = the whole hot path over one batch of a workload's layers: per layer the weight quantizer (Q-EMA with its
EMA update, or round to nearest) and Q4, Q1 + Q6 + GEMM-1 (forward), Q3/Q5 (one pass over dY), GEMM-2, GEMM-3
(backward).  Metric: useful TFLOP/s = 6*M*N*K per layer / time.  The headline is config 4 (ViT-Large MLP, 50432
tokens: the largest workload that the method's configurations name); the other configurations are timed in the same
run and reported under "configs".

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 4] [--others 1,2,3,5,6]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads  # noqa: E402

METRIC = "mxfp4_linear_fwd_bwd_tflops"
UNIT = "TFLOP/s"
Q = 0.5 + 1.0 / 32.0  # bytes per MXFP4 element (packed nibble + scale share)
CPU_SAMPLE_ROWS = 1024  # token rows per layer of the oracle's timed sample (reference arm and cpu_baseline alike)
KERNEL_REPS = 50        # timed launches per kernel of the breakdown (after 3 untimed ones)


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
    """Samples nvidia-smi clocks / throttle reasons every 100 ms while a timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def mark(self):
        return time.perf_counter()

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, t0=None, t1=None):
        """Median SM clock, maximum clock and the reasons seen among the samples taken between t0 and t1."""
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        sm, mx_, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for (t, ln) in list(self.lines):
            if (t0 is not None and t < t0) or (t1 is not None and t > t1):
                continue
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


def measure_stream_rates(torch, nbytes=1 << 30, reps=5):
    """Write-only and read-only HBM rates measured here (best of `reps`, CUDA events): a 1 GiB fill and a 1 GiB sum.
    The roofline denominator stays the measured copy rate; these two say what a kernel whose traffic is mostly output
    (the short-contraction products write 8 times what they read) or mostly input can reach on this part."""
    buf = torch.empty(nbytes // 4, dtype=torch.float32, device="cuda")
    out = {}
    for name, fn in (("write_only_gbs", lambda: buf.fill_(1.0)), ("read_only_gbs", lambda: buf.sum())):
        best = 1e9
        for _ in range(reps + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            e1.synchronize()
            best = min(best, e0.elapsed_time(e1) * 1e-3)
        out[name] = round(nbytes / best / 1e9, 1)
    del buf
    return out


def layer_flops(L, rows=None):
    m = L.M if rows is None else rows
    return 6.0 * m * L.N * L.K


def workload_name(config):
    return "config%d: %s" % (config, " + ".join("%s [M=%d,K=%d,N=%d]" % (L.name, L.M, L.K, L.N) for L in workloads.CONFIGS[config]))


# ---------------------------------------------------------------------------------------------------
# reference arm / cpu_baseline: the oracle, as it stands, on the host cores, on a bounded sample
# ---------------------------------------------------------------------------------------------------
def oracle_step(layers_data):
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


def oracle_sample_text(config, rows):
    return ("config %d layers at %d of their %d token rows: all quantizers + 3 FP64 products per layer; TFLOP/s counts the "
            "sampled rows' flops, i.e. it is the full workload's figure extrapolated linearly in the rows (the weight-gradient "
            "contraction is %d long instead of %d)" % (config, rows, workloads.CONFIGS[config][0].M, rows, workloads.CONFIGS[config][0].M))


def time_oracle(config, sample_rows, steps, warmup):
    import oracle as orc
    orc.lib()
    data = oracle_inputs(config, sample_rows)
    for _ in range(warmup):
        oracle_step(data)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(data)
    dt = (time.perf_counter() - t0) / steps
    flops = sum(layer_flops(L, sample_rows) for L in workloads.CONFIGS[config])
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    return dict(value=flops / dt / 1e12, seconds_per_step=dt, cores=cores, flops=flops)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    r = time_oracle(args.config, CPU_SAMPLE_ROWS, max(1, args.steps), max(0, min(args.warmup, 1)))
    sample = oracle_sample_text(args.config, CPU_SAMPLE_ROWS)
    line = dict(impl="reference", metric=METRIC, value=r["value"], unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=r["seconds_per_step"] * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=workload_name(args.config), sample=sample, extrapolated=True),
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


def make_inputs(config):
    """The seeded tensors of every layer of a configuration; the three tensors of every layer are generated side by side
    (numpy's generators release the interpreter lock)."""
    layers = workloads.CONFIGS[config]
    jobs = []
    with ThreadPoolExecutor(max_workers=min(8, 3 * len(layers))) as ex:
        for li, L in enumerate(layers):
            jobs.append((ex.submit(workloads.make_x, L, workloads.tensor_seed(config, li, "X")),
                         ex.submit(workloads.make_w, L, workloads.tensor_seed(config, li, "W")),
                         ex.submit(workloads.make_dy, L, workloads.tensor_seed(config, li, "dY"))))
        return [tuple(f.result() for f in j) for j in jobs]


class LayerState:
    """Device-resident tensors and scratch of one linear layer."""

    def __init__(self, mx, torch, config, li, tensors, host_io):
        L = workloads.CONFIGS[config][li]
        x, w, dy = tensors
        self.L = L
        hb = lambda a: torch.from_numpy(a).to(torch.bfloat16)  # noqa: E731
        xb, wb, dyb = hb(x), hb(w), hb(dy)
        self.x, self.w, self.dy = xb.cuda(), wb.cuda(), dyb.cuda()
        self.host = dict(x=xb.pin_memory(), w=wb.pin_memory(), dy=dyb.pin_memory()) if host_io else None
        self.ema = self.w.float().contiguous()
        self.seed = workloads.sr_seed(config, li)
        self.wq = mx.QMat(L.N, L.K)
        self.wq_t = mx.QMat(L.K, L.N)
        self.osc = None
        if L.osc:
            # the oscillation counters of Sec. 6.1 ride along with Q-EMA: previous weight and quantized weight, two trajectory lengths
            self.osc = mx.OscState(self.w.clone(), mx.quantize(self.w), torch.zeros((L.N, L.K), device="cuda"),
                                   torch.zeros((L.N, L.K), device="cuda"))
        self.ctx = mx.LinearCtx(mx.QMat(L.M, L.K), self.wq, xq_t=mx.QMat(L.K, L.M), seed=self.seed, wq_t=self.wq_t)
        self.weights_ready = torch.cuda.Event()
        self.ev_in, self.ev_done, self.ev_copied = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()
        self.y = torch.empty((L.M, L.N), dtype=torch.bfloat16, device="cuda")
        self.dx = torch.empty((L.M, L.K), dtype=torch.bfloat16, device="cuda")
        self.dw = torch.empty((L.N, L.K), dtype=torch.float32, device="cuda")
        self.ws = torch.empty(mx.linear_workspace_bytes(L.M, L.K, L.N), dtype=torch.uint8, device="cuda")
        self.host_out = None
        if host_io:
            self.host_out = dict(y=torch.empty((L.M, L.N), dtype=torch.bfloat16).pin_memory(),
                                 dx=torch.empty((L.M, L.K), dtype=torch.bfloat16).pin_memory(),
                                 dw=torch.empty((L.N, L.K), dtype=torch.float32).pin_memory())

    def weight_step(self, mx, status):
        """The weight side of a step: Q2 (Q-EMA with its EMA update and, where the workload keeps them, the oscillation
        counters; or round to nearest) and, from it, the backward operand Q4.  It depends on the weight alone, so the
        benchmark runs the first layer's on the step's stream and the others beside it on a second stream."""
        if self.L.qema:
            mx.qema_quantize(self.w, self.ema, beta=0.998, update_ema=True, osc=self.osc, out=self.wq, dev_status=status)
            mx.quantize_t(self.wq, rounding=1, seed=self.seed, stream_id=4, out=self.wq_t, dev_status=status)
        else:
            # Q2 (round to nearest) and its double quantization Q4 from one read of the weight: the same kernel that makes
            # Q1 and Q6 of the activations, with Q4's random stream
            mx.quantize_chain(self.w, seed=self.seed, stream_id_t=4, out=self.wq, out_t=self.wq_t, dev_status=status)

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


def kernel_breakdown(mx, torch, layers, flush, reps=KERNEL_REPS):
    """Per-kernel device time (CUDA events on the launching stream, L2 flushed before every launch): median and best of
    `reps` timed launches after 3 untimed ones, with the algorithmic bytes / flops of each launch of the step."""
    out = []

    def timed(name, fn, alg_bytes, flops, bound):
        ts = []
        for i in range(reps + 3):
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            e1.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1) * 1e-3)
        out.append(dict(kernel=name, seconds=float(np.median(ts)), best=float(np.min(ts)), mean=float(np.mean(ts)),
                        launches=len(ts), alg_bytes=alg_bytes, flops=flops, bound=bound))

    for S in layers:
        L = S.L
        M, K, N = L.M, L.K, L.N
        tag = L.name
        if L.qema:
            per = (2 + 4 + 4 + Q) + ((2 + 2 + Q + 16 + Q) if S.osc is not None else 0)
            timed(tag + ":qema" + ("_osc" if S.osc is not None else ""), lambda: mx.qema_quantize(S.w, S.ema, osc=S.osc, out=S.wq), N * K * per, 0, "hbm")
        else:
            timed(tag + ":quantize_w_q2_q4", lambda: mx.quantize_chain(S.w, seed=S.seed, stream_id_t=4, out=S.wq, out_t=S.wq_t), N * K * (2 + 2 * Q), 0, "hbm")
        # Q1 and Q6 (the double quantization of Q1's result) in one pass over X
        timed(tag + ":quantize_x_q1_q6", lambda: mx.quantize_chain(S.x, seed=S.seed, out=S.ctx.xq, out_t=S.ctx.xq_t), M * K * (2 + 2 * Q), 0, "hbm")
        timed(tag + ":gemm_y", lambda: mx.gemm(S.ctx.xq, S.wq, out=S.y), Q * K * (M + N) + 2 * M * N, 2.0 * M * N * K, "tensor")
        dyq, dyq_t = mx.QMat(M, N), mx.QMat(N, M)
        wq_t, xq_t = mx.QMat(K, N), S.ctx.xq_t
        sr = lambda s: (0, 1, S.seed, s)  # noqa: E731
        timed(tag + ":quantize_2axis_dy", lambda: mx.quantize_2axis(S.dy, sr(3), sr(5), out=dyq, out_t=dyq_t), M * N * (2 + 2 * Q), 0, "hbm")
        if L.qema:
            timed(tag + ":requant_w", lambda: mx.quantize_t(S.wq, rounding=1, seed=S.seed, stream_id=4, out=wq_t), N * K * 2 * Q, 0, "hbm")
        else:
            wq_t = S.wq_t
        timed(tag + ":gemm_dx", lambda: mx.gemm(dyq, wq_t, out=S.dx), Q * N * (M + K) + 2 * M * K, 2.0 * M * N * K, "tensor")
        ws = torch.empty(max(16, mx.gemm_workspace_bytes(N, K, M)), dtype=torch.uint8, device="cuda")
        timed(tag + ":gemm_dw", lambda: mx.gemm(dyq_t, xq_t, out_dtype=mx.OUT_FP32, out=S.dw, workspace=ws),
              Q * M * (N + K) + 4 * N * K, 2.0 * M * N * K, "tensor")
        del dyq, dyq_t, wq_t, ws
    return out


def summarise_kernels(kb, peaks):
    """Shares, rates and roofline fractions of the kernels of one step; the dominant kernel's roofline object."""
    fp4_peak = 4.0 * peaks["bf16"]  # dense FP4 = 4 x dense bf16 (the ratio the paper quotes), burst figure: kernels are timed alone
    ksum = sum(k["seconds"] for k in kb)
    rows = []
    for k in kb:
        t = k["seconds"]
        row = dict(kernel=k["kernel"], us=round(t * 1e6, 2), us_best=round(k["best"] * 1e6, 2), launches=k["launches"],
                   share=round(t / ksum, 4), gbs=round(k["alg_bytes"] / t / 1e9, 1), bound=k["bound"])
        if k["bound"] == "hbm":
            row["frac_hbm"] = round(k["alg_bytes"] / t / 1e9 / peaks["hbm"], 4)
        else:
            tf = k["flops"] / t / 1e12
            ai = k["flops"] / k["alg_bytes"]
            cap = min(fp4_peak, ai * peaks["hbm"] * 1e9 / 1e12)   # min(peak, arithmetic intensity x HBM rate)
            row.update(tflops=round(tf, 1), frac_fp4_peak=round(tf / fp4_peak, 4), ai_flop_per_byte=round(ai, 1),
                       cap_tflops=round(cap, 1), frac_of_cap=round(tf / cap, 4))
        rows.append(row)
    dom = max(kb, key=lambda k: k["seconds"])
    if dom["bound"] == "hbm":
        ach = dom["alg_bytes"] / dom["seconds"] / 1e9
        roof = dict(bound="hbm", kernel=dom["kernel"], achieved=ach, peak=peaks["hbm"], unit="GB/s", frac=ach / peaks["hbm"],
                    traffic=read_traffic(dom["kernel"]), peak_source=peaks["source"],
                    timing="median of %d launches, L2 flushed before each" % dom["launches"],
                    achieved_best=dom["alg_bytes"] / dom["best"] / 1e9)
    else:
        ach = dom["flops"] / dom["seconds"] / 1e12
        roof = dict(bound="tensor", kernel=dom["kernel"], achieved=ach, peak=fp4_peak, unit="TFLOP/s", frac=ach / fp4_peak,
                    traffic=read_traffic(dom["kernel"]), peak_source=peaks["source"] + " bf16 x 4",
                    timing="median of %d launches, L2 flushed before each" % dom["launches"],
                    achieved_best=dom["flops"] / dom["best"] / 1e12)
    return rows, roof


class ConfigRun:
    """One configuration resident on the device: its step (eager or as a CUDA graph) and its timing."""

    def __init__(self, mx, torch, binding, config, host_io, use_graph, flush):
        self.mx, self.torch, self.binding, self.config, self.flush = mx, torch, binding, config, flush
        tensors = make_inputs(config)
        self.layers = [LayerState(mx, torch, config, li, tensors[li], host_io) for li in range(len(tensors))]
        del tensors
        self.status = mx.new_status()
        self.weight_stream = torch.cuda.Stream()
        self.graph = None
        self.launches_per_step = 0
        self.run_steps(1)   # one eager step first: function attributes, lazy module loading
        if use_graph:
            # the launch sequence of a training step is fixed, so replaying it takes the host out of the timed region
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                self.one_step()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            self.graph = torch.cuda.CUDAGraph()
            l0 = mx.launch_count()
            with torch.cuda.graph(self.graph):
                self.one_step()
            self.launches_per_step = mx.launch_count() - l0
        else:
            l0 = mx.launch_count()
            self.one_step()
            self.launches_per_step = mx.launch_count() - l0

    def one_step(self):
        """One training step of every layer, inputs resident in HBM.  The first layer's weight quantizers run on the current
        stream (its forward pass would only wait for them), those of the other layers beside them on a second stream;
        forward and backward follow on the current stream, which waits for a later layer's weights before that layer's
        forward pass (they are long done by then)."""
        torch, mx = self.torch, self.mx
        main = torch.cuda.current_stream()
        self.weight_stream.wait_stream(main)
        with torch.cuda.stream(self.weight_stream):
            for S in self.layers[1:]:
                S.weight_step(mx, self.status)
                S.weights_ready.record(self.weight_stream)
        self.layers[0].weight_step(mx, self.status)
        for i, S in enumerate(self.layers):
            if i:
                main.wait_event(S.weights_ready)
            S.step(mx, self.status)
        main.wait_stream(self.weight_stream)

    def run_steps(self, n):
        torch = self.torch
        total = 0.0
        for _ in range(n):
            self.flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            if self.graph is not None:
                self.graph.replay()
            else:
                self.one_step()
            e1.record()
            e1.synchronize()
            total += e0.elapsed_time(e1) * 1e-3
        return total

    def flops_per_step(self):
        return sum(layer_flops(S.L) for S in self.layers)

    def check_status(self):
        if int(self.status.item()) != 0:
            raise RuntimeError("device status %d during the benchmark of config %d" % (int(self.status.item()), self.config))


def run_e2e(torch, mx, run, n, h2d_stream, d2h_stream):
    """n end-to-end steps timed as one block: every step copies its inputs from pinned host memory and its results
    back, as a training loop does it: the copies of one step overlap the compute and the copies of its neighbours
    (the next step's inputs travel while this step's results go back; the two directions have their own engines).
    An input buffer is refilled only after the step that reads it has finished, an output buffer is overwritten only
    after its copy to the host has."""
    layers, status, weight_stream = run.layers, run.status, run.weight_stream
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


def time_mlp_pair(mx, torch, config, flush, steps, use_graph=True):
    """fc1 -> GELU -> fc2, forward and backward with the data flowing between the two layers, timed two ways:
    `unfused`: every quantization by its stand-alone kernel, GELU and the multiplication by its derivative as separate
    elementwise passes (plain torch bf16 kernels, the harness around the library); `fused`: fc1's forward product emits
    Q1 / Q6 of fc2's input behind the GELU in its epilogue, fc2's input-gradient product multiplies by the derivative and
    emits Q3 / Q5 of fc1's output gradient (mxfp4_linear_fwd_ex / _bwd_ex).  The derivative GELU'(Y1) is a tensor made
    once, outside the timed step, in both variants."""
    tensors = make_inputs(config)
    L1, L2 = workloads.CONFIGS[config]
    assert L1.N == L2.K and L1.M == L2.M
    M, K1, N1, N2 = L1.M, L1.K, L1.N, L2.N
    hb = lambda a: torch.from_numpy(a).to(torch.bfloat16).cuda()  # noqa: E731
    x, w1, w2, dy2 = hb(tensors[0][0]), hb(tensors[0][1]), hb(tensors[1][1]), hb(tensors[1][2])
    del tensors
    s1, s2 = workloads.sr_seed(config, 0), workloads.sr_seed(config, 1)
    st = mx.new_status()
    wq1, wq2 = mx.quantize(w1), mx.quantize(w2)
    wq1_t = mx.quantize_t(wq1, rounding=1, seed=s1, stream_id=4)
    wq2_t = mx.quantize_t(wq2, rounding=1, seed=s2, stream_id=4)
    ctx1 = mx.LinearCtx(mx.QMat(M, K1), wq1, xq_t=mx.QMat(K1, M), seed=s1, wq_t=wq1_t)
    ctx2 = mx.LinearCtx(mx.QMat(M, N1), wq2, xq_t=mx.QMat(N1, M), seed=s2, wq_t=wq2_t)
    bf = lambda r, c: torch.empty((r, c), dtype=torch.bfloat16, device="cuda")  # noqa: E731
    y1, z1, y2, dz, dy1, dx1 = bf(M, N1), bf(M, N1), bf(M, N2), bf(M, N1), bf(M, N1), bf(M, K1)
    dw1 = torch.empty((N1, K1), dtype=torch.float32, device="cuda")
    dw2 = torch.empty((N2, N1), dtype=torch.float32, device="cuda")
    ws1 = torch.empty(mx.linear_workspace_bytes(M, K1, N1), dtype=torch.uint8, device="cuda")
    ws2 = torch.empty(mx.linear_workspace_bytes(M, N1, N2), dtype=torch.uint8, device="cuda")
    dyq1, dyq1_t = mx.QMat(M, N1), mx.QMat(N1, M)
    gprime = torch.rand((M, N1), device="cuda").to(torch.bfloat16)      # stands in for GELU'(Y1): values in [0, 1)

    def unfused():
        mx.linear_fwd(x, wq=wq1, ctx=ctx1, out=y1, dev_status=st)
        torch.ops.aten.gelu.out(y1, out=z1)
        mx.linear_fwd(z1, wq=wq2, ctx=ctx2, out=y2, dev_status=st)
        mx.linear_bwd(dy2, ctx2, s2, dx=dz, dw=dw2, workspace=ws2, dev_status=st)
        torch.mul(dz, gprime, out=dy1)
        mx.linear_bwd(dy1, ctx1, s1, dx=dx1, dw=dw1, workspace=ws1, dev_status=st)

    epi_f = mx.Epilogue(hook=mx.HOOK_GELU, y=y1, zq=ctx2.xq, qp_row=(0, 0, 0, 0), zq_t=ctx2.xq_t, qp_t=(0, 1, s2, 6), chain=True)
    epi_b = mx.Epilogue(hook=mx.HOOK_MULTIPLY, aux=gprime, zq=dyq1, qp_row=(0, 1, s1, 3), zq_t=dyq1_t, qp_t=(0, 1, s1, 5))

    def fused():
        mx.linear_fwd(x, wq=wq1, ctx=ctx1, dev_status=st, epi=epi_f)
        mx.linear_fwd(None, wq=wq2, ctx=ctx2, out=y2, dev_status=st)
        mx.linear_bwd(dy2, ctx2, s2, dw=dw2, workspace=ws2, dev_status=st, epi_dx=epi_b)
        mx.linear_bwd(None, ctx1, s1, dx=dx1, dw=dw1, workspace=ws1, dev_status=st, dyq=dyq1, dyq_t=dyq1_t)

    out = {}
    for name, fn in (("unfused", unfused), ("fused", fused)):
        fn()
        torch.cuda.synchronize()
        graph = None
        if use_graph:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                fn()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                fn()
        ts = []
        for i in range(steps + 3):
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay() if graph is not None else fn()
            e1.record()
            e1.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1))
        out[name + "_ms"] = float(np.median(ts))
        del graph
    if int(st.item()) != 0:
        raise RuntimeError("device status %d in the MLP-pair benchmark" % int(st.item()))
    flops = layer_flops(L1) + layer_flops(L2)
    out.update(workload="config%d as a chain: %s -> GELU -> %s, %d tokens" % (config, L1.name, L2.name, M),
               unfused_tflops=flops / out["unfused_ms"] / 1e9, fused_tflops=flops / out["fused_ms"] / 1e9,
               speedup=out["unfused_ms"] / out["fused_ms"], steps=steps,
               note="weight quantizers (Q2, Q4) made ahead in both variants; unfused includes the GELU and the multiplication by "
                    "its derivative as separate bf16 elementwise passes (torch kernels), fused does them in the products' epilogues")
    return out


def time_block(mx, torch, binding, flush, steps, use_graph=True):
    """The fifth workload as stated: one DeiT-Small block training step (batch 128 x 197 tokens) with its four linear
    layers in the library (Q-EMA weight quantizer and oscillation counters included) and attention, LayerNorm, GELU and
    residuals as PyTorch bf16 kernels with autograd (workloads/block_harness.py)."""
    from workloads import block_harness as bh
    blk = bh.Block(mx)
    x, dout = bh.make_block_inputs(128)
    blk.weight_step()
    blk.perturb_weights(seed=77)
    for _ in range(2):
        blk.step(x, dout)
    torch.cuda.synchronize()
    graph, launch = None, "eager"
    l0 = mx.launch_count()
    blk.step(x, dout)
    lib_launches = mx.launch_count() - l0
    if use_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                blk.step(x, dout)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                blk.step(x, dout)
            graph, launch = g, "CUDA graph replay of one step"
        except Exception as e:  # noqa: BLE001  (the harness falls back to eager launches; the library is not involved)
            torch.cuda.synchronize()
            launch = "eager (graph capture of the autograd harness failed: %s)" % type(e).__name__
    ts = []
    for i in range(steps + 3):
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay() if graph is not None else blk.step(x, dout)
        e1.record()
        e1.synchronize()
        if i >= 3:
            ts.append(e0.elapsed_time(e1))
    for layer in blk.layers.values():
        if int(layer.status.item()) != 0:
            raise RuntimeError("device status %d in the block benchmark" % int(layer.status.item()))
    ms = float(np.median(ts))
    flops = sum(layer_flops(L) for L in workloads.CONFIGS[5])
    return dict(workload="DeiT-Small block, batch 128 x 197 tokens: qkv, proj, fc1, fc2 in the library; LayerNorm, attention, GELU, residuals in PyTorch bf16",
                ms_per_step=ms, linear_tflops=flops / ms / 1e9, library_launches_per_step=lib_launches, launch=launch, steps=steps)


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
    fp4_burst, fp4_sustained = 4.0 * peaks["bf16"], 4.0 * peaks["bf16_sustained"]
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")  # > 126 MB L2

    def flush():
        flush_buf.fill_(1)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local).start() if rank == 0 else None
    warmup = max(3, args.warmup)

    # ---------------- the headline configuration ----------------
    run = ConfigRun(mx, torch, binding, args.config, host_io=True, use_graph=not args.no_graph, flush=flush)
    # warm-up; kept going for at least 1.5 s so that the clocks have settled under load before timing starts
    t_warm = time.perf_counter()
    run.run_steps(warmup)
    while time.perf_counter() - t_warm < 1.5:
        run.run_steps(3)
    barrier()
    c0 = time.perf_counter()
    launches0 = mx.launch_count()
    total = run.run_steps(args.steps)
    launches = (mx.launch_count() - launches0) if run.graph is None else run.launches_per_step * args.steps
    # the timed region of a short run ends before the sampler's next tick: keep the same load going (untimed) until it has ticked
    while time.perf_counter() - c0 < 0.6:
        run.run_steps(3)
    c1 = time.perf_counter()
    barrier()
    clocks = sampler.summary(t_warm + 0.5, c1) if rank == 0 else None
    h2d_stream, d2h_stream = torch.cuda.Stream(), torch.cuda.Stream()
    run_e2e(torch, mx, run, 2, h2d_stream, d2h_stream)
    barrier()
    total_e2e = run_e2e(torch, mx, run, args.steps, h2d_stream, d2h_stream)
    barrier()
    run.check_status()

    total, total_e2e = max_over_ranks([total, total_e2e], "cuda")
    flops_step = run.flops_per_step() * world
    value = flops_step * args.steps / total / 1e12
    value_e2e = flops_step * args.steps / total_e2e / 1e12
    h2d = sum(S.io_bytes()[0] for S in run.layers)
    d2h = sum(S.io_bytes()[1] for S in run.layers)

    line = None
    if rank == 0:
        kb = kernel_breakdown(mx, torch, run.layers, flush)
        kernels, roof = summarise_kernels(kb, peaks)
        main_summary = dict(workload=workload_name(args.config), ms_per_step=total / args.steps * 1e3, tflops=value / world,
                            pct_fp4_peak_burst=100.0 * value / world / fp4_burst, pct_fp4_peak_sustained=100.0 * value / world / fp4_sustained,
                            dominant_kernel=roof["kernel"], dominant_frac=roof["frac"], dominant_bound=roof["bound"],
                            launches_per_step=run.launches_per_step, sm_mhz=clocks["sm_mhz"], steps=args.steps)
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=warmup,
                    ms_per_step=total / args.steps * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="mxfp4 (e2m1 x e8m0), f32 accumulate", data="synthetic",
                    config=dict(workload=workload_name(args.config),
                                l2="flushed between steps (256 MB write)", qema=any(S.L.qema for S in run.layers), replicas=world,
                                launch="eager" if run.graph is None else "CUDA graph replay of one step",
                                streams="weight quantizers (Q2 + Q4, one launch per weight without Q-EMA): the first layer's on the step's stream, the others beside it on a second stream"),
                    pct_fp4_peak=dict(burst=main_summary["pct_fp4_peak_burst"], sustained=main_summary["pct_fp4_peak_sustained"],
                                      note="step TFLOP/s over 4 x the measured bf16 GEMM rate (burst / sustained); the quantizer passes are inside the step"),
                    clocks=clocks,
                    e2e=dict(value=value_e2e, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                             ms_per_step=total_e2e / args.steps * 1e3,
                             note="steps timed as one block; every step copies all inputs in from pinned host memory and all "
                                  "results out; copies of neighbouring steps overlap on their own streams"),
                    gpu_launches=launches, roofline=roof, kernels=kernels)
    del run
    torch.cuda.empty_cache()

    # ---------------- the other configurations, one after the other (rank 0 reports; every replica runs them) ----------------
    configs = {}
    if line is not None:
        configs[str(args.config)] = main_summary
    for c in args.others:
        if c == args.config:
            continue
        r = ConfigRun(mx, torch, binding, c, host_io=False, use_graph=not args.no_graph, flush=flush)
        r.run_steps(warmup)
        (one,) = max_over_ranks([r.run_steps(5) / 5], "cuda")   # every replica times the same number of steps
        n = int(min(2000, max(20, 1.0 / max(one, 1e-6))))   # about a second of steps, so that the clock sampler sees them
        c0 = time.perf_counter()
        tot = r.run_steps(n)
        c1 = time.perf_counter()
        r.check_status()
        (tot,) = max_over_ranks([tot], "cuda")
        if rank == 0:
            kb = kernel_breakdown(mx, torch, r.layers, flush)
            krows, kroof = summarise_kernels(kb, peaks)
            tf = r.flops_per_step() * n / tot / 1e12   # per replica, like the headline's pct_fp4_peak
            ck = sampler.summary(c0, c1)
            configs[str(c)] = dict(workload=workload_name(c), ms_per_step=tot / n * 1e3, tflops=tf,
                                   pct_fp4_peak_burst=100.0 * tf / fp4_burst, pct_fp4_peak_sustained=100.0 * tf / fp4_sustained,
                                   dominant_kernel=kroof["kernel"], dominant_frac=kroof["frac"], dominant_bound=kroof["bound"],
                                   launches_per_step=r.launches_per_step, sm_mhz=ck["sm_mhz"], reasons=ck["reasons"], steps=n,
                                   kernels=[{k: v for k, v in row.items() if k in ("kernel", "us", "us_best", "share", "gbs", "tflops", "frac_hbm", "frac_fp4_peak", "frac_of_cap")}
                                            for row in krows])
        del r
        torch.cuda.empty_cache()

    mlp_pair = {}
    if rank == 0 and 5 in args.others and "5" in configs:
        blk = time_block(mx, torch, binding, flush, 30, use_graph=not args.no_graph)
        blk["linears_ms"] = configs["5"]["ms_per_step"]
        blk["harness_ms"] = blk["ms_per_step"] - blk["linears_ms"]
        blk["note"] = "linears_ms: the same four layers' step on resident tensors (configs['5']); harness_ms: the rest of the block step"
        configs["5"]["block"] = blk
        torch.cuda.empty_cache()
    if rank == 0:
        for c in args.mlp_pairs:
            mlp_pair[str(c)] = time_mlp_pair(mx, torch, c, flush, 30, use_graph=not args.no_graph)
            torch.cuda.empty_cache()

    if rank == 0:
        sampler.stop()
        cpu = time_oracle(args.config, CPU_SAMPLE_ROWS, args.cpu_passes, 0)
        line["configs"] = configs
        line["mlp_pair"] = mlp_pair
        line["cpu_baseline"] = dict(value=cpu["value"], unit=UNIT, cores=cpu["cores"], kind="oracle",
                                    sample=oracle_sample_text(args.config, CPU_SAMPLE_ROWS) + "; %d passes" % args.cpu_passes)
        line["peaks"] = dict(measure_stream_rates(torch), hbm_gbs=peaks["hbm"], bf16_tflops=peaks["bf16"], bf16_tflops_sustained=peaks["bf16_sustained"],
                             fp4_tflops_proxy=fp4_burst, fp4_tflops_proxy_sustained=fp4_sustained, source=peaks["source"],
                             fp4_mma_issue_ceiling_tflops=round(mx.mma_issue_ceiling(bn=256), 1),
                             fp4_mma_issue_ceiling_note="measured here: MMA-only loop, 128x256x64 kind::mxf4, operands resident in shared memory")
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4, choices=sorted(workloads.CONFIGS))
    ap.add_argument("--others", default="auto", help="configurations timed after the headline one and reported under 'configs' (comma separated; empty for none; "
                                                      "auto: 1,2,3,5,6 on one GPU, none when several replicas run)")
    ap.add_argument("--mlp-pairs", default="auto", help="two-layer configurations also timed as a chain fc1 -> GELU -> fc2, with and without the fused epilogues "
                                                         "(auto: 4,2 on one GPU, none when several replicas run)")
    ap.add_argument("--cpu-passes", type=int, default=5, help="passes of the oracle over its row sample for cpu_baseline")
    ap.add_argument("--no-graph", action="store_true", help="launch every step from the host instead of replaying a CUDA graph")
    args = ap.parse_args()
    single = int(os.environ.get("WORLD_SIZE", "1")) == 1
    if args.others == "auto":
        args.others = "1,2,3,5,6" if single else ""
    if args.mlp_pairs == "auto":
        args.mlp_pairs = "4,2" if single else ""
    args.others = [int(t) for t in args.others.split(",") if t.strip()]
    args.mlp_pairs = [int(t) for t in args.mlp_pairs.split(",") if t.strip()]
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
