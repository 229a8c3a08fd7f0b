"""Benchmark of the COD-TDQ hot path on B200: token-group quantizer -> W4A4 linear.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl tdq|reference] [--workload cfg4|cfg3|cfg2]

A step is one pass of the whole path over one batch of the workload: tdq_quantize_act on X,
then tdq_w4a4_linear on the codes (weights are quantized once, before timing: they are
static).  The default workload is the ViT-B-style MLP fc1 case, X bf16 [32, 577, 768] and
W [3072, 768], the largest of the single-layer workloads.  One JSON line is printed.

  value / unit       quantizer throughput in GB/s: algorithmic bytes (2 B read + 0.5 B codes +
                     0.125 B scale per element) / device time of the quantizer kernel, summed
                     over all ranks.  The linear layer's TOPS and both roofline fractions are
                     in "kernels"; ms_per_step is the whole step.
  e2e                the same quantity through tdq_quant_linear_host with pinned HOST input and
                     output, copies inside the timed region.
  roofline           for the kernel that takes most of the step.
  cpu_baseline       the CPU oracle on the host cores, on a bounded sample, rank 0, N=1 only.

--impl reference times the CPU oracle as it stands (rank 0 only).
Multi-GPU: rows are independent, every rank runs its own full batch (weak scaling, no
collective on the data path); the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "quantizer GB/s and W4A4 linear TOPS at 1 B200, % of HBM / INT8 roofline"
L2_BYTES = 126 * 2 ** 20


def kernel_source_hash(files):
    """sha256 over the named source files of the package's csrc directory, in the given order."""
    import hashlib
    h = hashlib.sha256()
    for name in files:
        with open(os.path.join(ROOT, "paper_2604_16855_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def profiled_traffic(kernel, workload_name, files):
    """DRAM bytes per launch of `kernel` on `workload_name` from the committed profile summary, or None.  A summary
    counts only while the kernel's sources still hash to what the summary records (the counters were taken on that
    code); its lines `kernel:`, `workload:`, `dram_bytes_per_launch:` and `kernel_source_sha256:` are read."""
    d = os.path.join(ROOT, "profiles")
    if not os.path.isdir(d):
        return None
    want = kernel_source_hash(files)
    for name in sorted(os.listdir(d)):
        fields = {}
        try:
            for line in open(os.path.join(d, name)):
                if ":" in line:
                    k, v = line.split(":", 1)
                    fields[k.strip().strip("`*- ")] = v.strip().strip("`* ")
        except OSError:
            continue
        if fields.get("kernel") == kernel and fields.get("workload") == workload_name and \
                fields.get("kernel_source_sha256") == want:
            try:
                return float(fields["dram_bytes_per_launch"])
            except (KeyError, ValueError):
                return None
    return None


LINEAR_G32_SOURCES = ["tdq_linear_g32.cu", "tdq_tc.cuh"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def workload(name):
    return {"cfg1": si.config1, "cfg2": si.config2, "cfg3": si.config3, "cfg4": si.config4}[name]()


def quant_bytes(M, C, esize, g=32):
    return M * C * esize + M * C // 2 + M * (C // g) * 4


def linear_bytes(M, I, O, g=32, ysize=4):
    return M * I // 2 + M * (I // g) * 4 + O * I // 2 + O * 4 + M * O * ysize


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        for l in self.lines:
            f = [v.strip() for v in l.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        # the busiest samples are the ones taken under load
        load = sorted(sm)[len(sm) // 2:]
        return dict(sm_mhz=float(np.median(load)), sm_max_mhz=float(max(mx)), power_w_max=float(max(pw)),
                    samples=len(sm), reasons=sorted(reasons))


def cpu_oracle_leg(case, rows, repeats=1):
    """Times the oracle (quantizer + linear) on the first `rows` token rows.  Returns a dict."""
    import oracle
    x = case.x.reshape(-1, case.C)[:rows]
    wq = oracle.quantize_weight(case.w, pad_to=32)
    best_q, best_l = 1e30, 1e30
    for _ in range(repeats):
        t0 = time.perf_counter()
        xa = oracle.quantize_act(x)
        t1 = time.perf_counter()
        oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"])
        t2 = time.perf_counter()
        best_q, best_l = min(best_q, t1 - t0), min(best_l, t2 - t1)
    esize = 2 if case.x_is_bf16 else 4
    return dict(rows=int(x.shape[0]), quant_s=best_q, linear_s=best_l,
                quant_gbs=quant_bytes(x.shape[0], case.C, esize) / best_q / 1e9,
                linear_tops=2.0 * x.shape[0] * case.C * case.O / best_l / 1e12,
                cores=oracle.num_threads())


def cpu_oracle_single_thread(workload_name, rows):
    """The same oracle leg on one host thread (a child process, because the thread count of the oracle's OpenMP
    runtime is fixed when it starts)."""
    env = dict(os.environ, OMP_NUM_THREADS="1")
    try:
        r = subprocess.run([sys.executable, os.path.abspath(__file__), "--oracle-leg", str(rows), "--workload", workload_name],
                           env=env, capture_output=True, text=True, timeout=600)
        return json.loads(r.stdout.strip().splitlines()[-1])
    except (subprocess.SubprocessError, ValueError, IndexError, OSError):
        return None


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    case = workload(args.workload)
    # a step is a bounded sample: at most 2048 rows, fewer when many steps are asked for, so that the
    # whole run stays within about two minutes
    rows = 2048
    t0 = time.perf_counter()
    cpu_oracle_leg(case, rows)
    t_leg = time.perf_counter() - t0
    budget_s = 120.0
    if (args.steps + args.warmup) * t_leg > budget_s:
        rows = int(rows * budget_s / ((args.steps + args.warmup) * t_leg)) // 64 * 64
        rows = max(64, rows)
    for _ in range(args.warmup):
        cpu_oracle_leg(case, rows)
    t0 = time.perf_counter()
    legs = [cpu_oracle_leg(case, rows) for _ in range(args.steps)]
    wall = time.perf_counter() - t0
    qs = sum(l["quant_s"] for l in legs)
    ls = sum(l["linear_s"] for l in legs)
    esize = 2 if case.x_is_bf16 else 4
    value = args.steps * quant_bytes(rows, case.C, esize) / qs / 1e9
    sample = "first %d of %d token rows of %s per step, quantizer + linear" % (rows, case.M, case.name)
    out = dict(metric=METRIC, impl="reference", value=value, unit="GB/s", n_gpus=args.gpus, steps=args.steps,
               warmup=args.warmup, ms_per_step=1e3 * wall / args.steps, higher_is_better=True, scaling="weak",
               vs_baseline=None, dtype="f32", data="synthetic",
               config=dict(workload=case.name, x=[int(v) for v in case.x.shape], w=[int(v) for v in case.w.shape],
                           g=32, tau=1.0, zr=0.2, sample=sample),
               kernels=dict(linear=dict(tops=2.0 * args.steps * rows * case.C * case.O / ls / 1e12)),
               cpu_baseline=dict(value=value, unit="GB/s", cores=legs[0]["cores"], kind="oracle", sample=sample),
               e2e=dict(value=value, unit="GB/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(out))


def max_over_ranks(values, device, world):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the time)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_rate(units_per_rank, world, ms):
    """Units all ranks processed per second, given the slowest rank's time in milliseconds."""
    return world * units_per_rank / (ms * 1e-3)


def shard_rows(M, rank, world):
    """The token rows [start, stop) rank `rank` of `world` takes when one batch is split over the ranks (rows are
    independent, weights are replicated, nothing is exchanged): whole 128-row blocks, the remainder to the last ranks."""
    blocks = (M + 127) // 128
    lo = (blocks * rank) // world * 128
    hi = M if rank == world - 1 else (blocks * (rank + 1)) // world * 128
    return min(lo, M), min(hi, M)


def graph_steps(K, nsets, cap=64):
    """Steps per graph: the largest divisor of K that is a multiple of the buffer rotation and at
    most `cap`; K itself (one graph, one replay) when there is none."""
    for d in range(min(K, cap), 0, -1):
        if K % d == 0 and d % nsets == 0:
            return d
    return K


def time_graph(fn, n_inner, replays=5):
    """Captures n_inner calls of fn(i) into a CUDA graph, replays it, returns ms per call (device events)."""
    import torch
    fn(0)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(n_inner):
            fn(i)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (replays * n_inner)


def fused_leg(tdq, xs, wcodes, wscale, ys, wsp, M, C, O, esize):
    """The fused entry point on the same workload and buffer rotation: ms per call and its bytes."""
    n = len(xs)
    ms = time_graph(lambda i: tdq.quant_linear_fused(xs[i % n], wcodes, wscale, y=ys[i % n], workspace=wsp), 4 * n)
    bytes_ = M * C * esize + O * C // 2 + O * 4 + M * O * 4
    return dict(name="tdq_quant_linear_fused", ms=ms, gbs=bytes_ / (ms * 1e-3) / 1e9, tops=2.0 * M * C * O / (ms * 1e-3) / 1e12,
                algorithmic_bytes=bytes_)


def sweep_leg(tdq, dev):
    """The 32-layer sweep (two blocks of qkv, proj, fc1, fc2 in each of four encoder stages, batch 8): every layer
    quantizes its own input and runs its linear layer; total time per pass, launched from the host and from a graph."""
    import torch
    import synth_inputs as si
    layers = []
    max_y = max_codes = max_scale = max_ws = 0
    for li in range(32):
        case = si.config5_layer(li, batch=8)
        x = torch.from_numpy(case.x.reshape(case.M, case.C).view(np.int16).copy()).view(torch.bfloat16).to(dev)
        wc, ws = tdq.quantize_weight(torch.from_numpy(case.w).to(dev), 32)
        layers.append((x, wc, ws, case.M, case.C, case.O))
        max_y = max(max_y, case.M * case.O)
        max_codes = max(max_codes, case.M * case.C // 2)
        max_scale = max(max_scale, case.M * case.C // 32)
        max_ws = max(max_ws, tdq.linear_workspace(case.M, case.C, case.O, 32, dev).numel())
    ybuf = torch.empty((max_y,), dtype=torch.float32, device=dev)
    cbuf = torch.empty((max_codes,), dtype=torch.uint8, device=dev)
    sbuf = torch.empty((max_scale,), dtype=torch.float32, device=dev)
    wsp = torch.empty((max_ws,), dtype=torch.uint8, device=dev)
    params = tdq.default_act_params()

    def one_pass(_=0):
        for (x, wc, ws, M, C, O) in layers:
            codes = cbuf[:M * C // 2].view(M, C // 2)
            scale = sbuf[:M * C // 32].view(M, C // 32)
            tdq.quantize_act(x, params, codes=codes, scale=scale)
            tdq.w4a4_linear(codes, scale, wc, ws, y=ybuf[:M * O].view(M, O), workspace=wsp)

    def one_pass_fused(_=0):
        n_two = 0
        for (x, wc, ws, M, C, O) in layers:
            if C <= 768:
                tdq.quant_linear_fused(x, wc, ws, y=ybuf[:M * O].view(M, O), workspace=wsp)
            else:                     # the fused kernel keeps a row block's operand in shared memory: C <= 768
                codes = cbuf[:M * C // 2].view(M, C // 2)
                scale = sbuf[:M * C // 32].view(M, C // 32)
                tdq.quantize_act(x, params, codes=codes, scale=scale)
                tdq.w4a4_linear(codes, scale, wc, ws, y=ybuf[:M * O].view(M, O), workspace=wsp)
                n_two += 1
        return n_two

    for _ in range(3):
        one_pass()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        one_pass()
    e1.record()
    torch.cuda.synchronize()
    eager_ms = e0.elapsed_time(e1) / 5
    graph_ms = time_graph(one_pass, 1)
    n_two = one_pass_fused()
    fused_ms = time_graph(one_pass_fused, 1)
    macs = sum(M * C * O for (_, _, _, M, C, O) in layers)
    xbytes = sum(M * C * 2 for (_, _, _, M, C, O) in layers)
    ybytes = sum(M * O * 4 for (_, _, _, M, C, O) in layers)
    return dict(layers=32, batch=8, eager_us=eager_ms * 1e3, graph_us=graph_ms * 1e3, fused_graph_us=fused_ms * 1e3,
                fused_layers=32 - n_two, macs=macs, x_bytes=xbytes, y_bytes=ybytes,
                graph_tops=2.0 * macs / (graph_ms * 1e-3) / 1e12, graph_gbs=(xbytes + ybytes) / (graph_ms * 1e-3) / 1e9)


def small_configs_leg(tdq, dev, peaks):
    """cfg1-cfg3 (launch-bound sizes): per call from a graph over rotating buffers, with both roofline fractions."""
    import torch
    out = {}
    for name in ("cfg1", "cfg2", "cfg3"):
        case = workload(name)
        M, C, O = case.M, case.C, case.O
        esz = 2 if case.x_is_bf16 else 4
        xh = torch.from_numpy(case.x.reshape(M, C).view(np.int16).copy()).view(torch.bfloat16) if case.x_is_bf16 \
            else torch.from_numpy(case.x.reshape(M, C).copy())
        n = max(2, int(np.ceil(2.5 * L2_BYTES / (quant_bytes(M, C, esz) + M * O * 4))))
        n = min(n, 48)
        xs = [xh.to(dev) for _ in range(n)]
        wc, ws = tdq.quantize_weight(torch.from_numpy(case.w).to(dev), 32)
        codes = [torch.empty((M, C // 2), dtype=torch.uint8, device=dev) for _ in range(n)]
        scales = [torch.empty((M, C // 32), dtype=torch.float32, device=dev) for _ in range(n)]
        ys = [torch.empty((M, O), dtype=torch.float32, device=dev) for _ in range(n)]
        wsp = tdq.linear_workspace(M, C, O, 32, dev)
        p = tdq.default_act_params()
        q_ms = time_graph(lambda i: tdq.quantize_act(xs[i % n], p, codes=codes[i % n], scale=scales[i % n]), 2 * n)
        l_ms = time_graph(lambda i: tdq.w4a4_linear(codes[i % n], scales[i % n], wc, ws, y=ys[i % n], workspace=wsp), 2 * n)
        f_ms = time_graph(lambda i: tdq.quant_linear_fused(xs[i % n], wc, ws, y=ys[i % n], workspace=wsp), 2 * n)
        qb, lb, ops = quant_bytes(M, C, esz), linear_bytes(M, C, O), 2.0 * M * C * O
        out[name] = dict(x=[int(v) for v in case.x.shape], O=O, buffer_sets=n,
                         quantize_us=q_ms * 1e3, quantize_gbs=qb / (q_ms * 1e-3) / 1e9, quantize_frac_hbm=qb / (q_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                         linear_us=l_ms * 1e3, linear_tops=ops / (l_ms * 1e-3) / 1e12, linear_gbs=lb / (l_ms * 1e-3) / 1e9,
                         linear_frac_hbm=lb / (l_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], linear_bound="hbm", fused_us=f_ms * 1e3)
    return out


def pow2_leg(tdq, dev, workload_name):
    """The power-of-two variant alone on a workload's shape: its quantizer once, then its linear layer from a graph."""
    import torch
    case = workload(workload_name)
    M, C, O = case.M, case.C, case.w.shape[0]
    x = torch.from_numpy(case.x.reshape(M, C).view(np.int16).copy()).view(torch.bfloat16).to(dev) if case.x_is_bf16 \
        else torch.from_numpy(case.x.reshape(M, C)).to(dev)
    wcodes, wscale = tdq.quantize_weight(torch.from_numpy(case.w).to(dev), 32)
    p2 = tdq.act_params(flags=tdq.ENABLE_C1 | tdq.ENABLE_C2 | tdq.POW2_STEP)
    codes, scale = tdq.quantize_act(x, p2)
    ys = [torch.empty((M, O), dtype=torch.float32, device=dev) for _ in range(2)]
    wsp = tdq.linear_workspace(M, C, O, 32, dev)
    ms = time_graph(lambda i: tdq.w4a4_linear_pow2(codes, scale, wcodes, wscale, y=ys[i % 2], workspace=wsp), 8, replays=3)
    st, detail = tdq.workspace_status(wsp)
    if st != tdq.OK:
        raise RuntimeError("tdq_w4a4_linear_pow2 reported 0x%x" % detail)
    return dict(name="tdq_w4a4_linear_pow2", workload=workload_name, shape=[M, C, O], ms=ms,
                tops=2.0 * M * C * O / (ms * 1e-3) / 1e12)


def probe_leg(tdq, dev, peaks):
    """A compute-bound shape (16384 x 4096 -> 4096, bf16 output) with per-32 groups and with one group per token."""
    import torch
    M = I = 16384
    I = O = 4096
    torch.manual_seed(1)
    xc = torch.randint(0, 256, (M, I // 2), dtype=torch.uint8, device=dev)
    wc = torch.randint(0, 256, (O, I // 2), dtype=torch.uint8, device=dev)
    ws = torch.rand((O,), device=dev) + 0.5
    ys = [torch.empty((M, O), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    out = {}
    for g in (32, I):
        xs = torch.rand((M, I // g), device=dev) + 0.5
        wsp = tdq.linear_workspace(M, I, O, g, dev)
        ms = time_graph(lambda i: tdq.w4a4_linear(xc, xs, wc, ws, g=g, y=ys[i % 2], workspace=wsp), 4, replays=3)
        tops = 2.0 * M * I * O / (ms * 1e-3) / 1e12
        out["g%d" % g] = dict(ms=ms, tops=tops, frac_int8=tops / (2.0 * peaks["bf16_tflops"]), frac_int8_4500=tops / 4500.0)
    out["shape"] = [M, I, O]
    out["y_dtype"] = "bf16"
    return out


def run_tdq(args):
    import torch
    import torch.distributed as dist
    from paper_2604_16855_b200 import tdq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    case = workload(args.workload)
    M, C, O = case.M, case.C, case.O
    esize = 2 if case.x_is_bf16 else 4
    x_host = torch.from_numpy(case.x.reshape(M, C).view(np.int16).copy()).view(torch.bfloat16) if case.x_is_bf16 \
        else torch.from_numpy(case.x.reshape(M, C).copy())
    w = torch.from_numpy(case.w).to(dev)
    wcodes, wscale = tdq.quantize_weight(w, 32)

    # rotating buffer sets: a step touches X, codes, scales and Y; keep the rotation larger than L2
    step_bytes = quant_bytes(M, C, esize) + M * O * 4
    nsets = max(2, int(np.ceil(2.5 * L2_BYTES / step_bytes)))
    xs = [x_host.to(dev) for _ in range(nsets)]
    codes = [torch.empty((M, C // 2), dtype=torch.uint8, device=dev) for _ in range(nsets)]
    scales = [torch.empty((M, C // 32), dtype=torch.float32, device=dev) for _ in range(nsets)]
    ys = [torch.empty((M, O), dtype=torch.float32, device=dev) for _ in range(nsets)]
    wsp = tdq.linear_workspace(M, C, O, 32, dev)
    params = tdq.default_act_params()

    def step(i, ev=None):
        s = i % nsets
        if ev:
            ev[0].record()
        tdq.quantize_act(xs[s], params, codes=codes[s], scale=scales[s])
        if ev:
            ev[1].record()
        tdq.w4a4_linear(codes[s], scales[s], wcodes, wscale, y=ys[s], workspace=wsp)
        if ev:
            ev[2].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    st, detail = tdq.workspace_status(wsp)
    if st != tdq.OK:
        raise RuntimeError("linear kernel reported a device-side timeout: 0x%x" % detail)

    # The timed steps are replayed from a CUDA graph, so that the kernels run back to back and the
    # events measure kernels, not the host's launch path.  A graph holds G steps (a multiple of the
    # buffer rotation) and is replayed K / G times between two events: the step time.  The graph has
    # no event nodes inside: an event record between two kernel nodes costs about 7 us on this
    # hardware (cfg4: 157.8 us per step with two of them per step, 143.8 us without), which is
    # measurement, not the path.  Each kernel's own duration is timed the same way right after, from a
    # graph of that call alone over rotating buffers (inputs beyond 2.5 x L2), events around its launches.
    G = graph_steps(args.steps, nsets) if not args.eager else 0
    sampler = ClockSampler(local)
    launches0 = tdq.kernel_launch_count()
    if G:
        evs = None
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(G):
                step(args.warmup + i)
        launches_per_replay = tdq.kernel_launch_count() - launches0
        graph.replay()                       # untimed: uploads the graph
        barrier()
        st, detail = tdq.workspace_status(wsp)
        if st != tdq.OK:
            raise RuntimeError("linear kernel reported a device-side timeout: 0x%x" % detail)
    else:
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record()
    if G:
        for _ in range(args.steps // G):
            graph.replay()
    else:
        for i in range(args.steps):
            step(args.warmup + i, evs[i])
    t_end.record()
    barrier()
    if G:
        launches = launches_per_replay * (args.steps // G)
    else:
        launches = tdq.kernel_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    total_ms = t_begin.elapsed_time(t_end)
    n_iso = min(64, max(nsets, int(np.ceil(2.5 * L2_BYTES / (M * C * esize)))))   # input sets of the quantizer alone
    if G:
        xi = xs + [xs[0].clone() for _ in range(n_iso - nsets)]
        n_q = n_iso * max(1, min(args.steps, 64) // n_iso)
        q_call_ms = time_graph(lambda i: tdq.quantize_act(xi[i % n_iso], params, codes=codes[i % nsets], scale=scales[i % nsets]),
                               n_q, replays=max(1, args.steps // n_q))
        l_call_ms = time_graph(lambda i: tdq.w4a4_linear(codes[i % nsets], scales[i % nsets], wcodes, wscale, y=ys[i % nsets],
                                                         workspace=wsp), G, replays=args.steps // G)
        q_ms, l_ms = q_call_ms * args.steps, l_call_ms * args.steps
        barrier()
    else:
        n_ev = len(evs)
        q_ms = sum(e[0].elapsed_time(e[1]) for e in evs) * args.steps / n_ev
        l_ms = sum(e[1].elapsed_time(e[2]) for e in evs) * args.steps / n_ev

    # Sustained leg: the same step graph replayed for about two seconds with the clock sampler running.  The
    # 20-step region above lasts a few milliseconds, too short for a 100 ms sampler and for the power cap to act;
    # here the step time is read beside the SM clock it ran at, and their product (SM clocks per step) is what
    # stays comparable when the clock moves.
    sustained = None
    if G and rank == 0 and world == 1 and not args.no_extras:
        n_rep = max(1, int(2.0 / max(1e-6, (total_ms / args.steps) * 1e-3 * G)))
        s2 = ClockSampler(local)
        s2.start()
        time.sleep(0.25)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_rep):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        c2 = s2.stop()
        ms_step = e0.elapsed_time(e1) / (n_rep * G)
        sustained = dict(seconds=e0.elapsed_time(e1) * 1e-3, steps=n_rep * G, ms_per_step=ms_step, clocks=c2,
                         sm_clocks_per_step=(ms_step * 1e-3 * c2["sm_mhz"] * 1e6) if c2.get("sm_mhz") else None)
    # warm-cache figures: the same call on one buffer set, launched back to back (inputs stay in L2 where they fit)
    warm = None
    if G and world == 1:
        warm = dict(
            quantize_ms=time_graph(lambda i: tdq.quantize_act(xs[0], params, codes=codes[0], scale=scales[0]), 16),
            linear_ms=time_graph(lambda i: tdq.w4a4_linear(codes[0], scales[0], wcodes, wscale, y=ys[0], workspace=wsp), 8))

    # end to end: pinned host X in, host Y out, through the host-buffer entry point
    xh = x_host.pin_memory()
    yh = torch.empty((M, O), dtype=torch.float32).pin_memory()
    stream = torch.cuda.current_stream().cuda_stream
    import ctypes

    def e2e_step():
        rc = tdq.lib().tdq_quant_linear_host(
            ctypes.c_void_p(xh.data_ptr()), tdq.BF16 if case.x_is_bf16 else tdq.F32, 1, M, C, ctypes.byref(params),
            ctypes.c_void_p(wcodes.data_ptr()), ctypes.c_void_p(wscale.data_ptr()), None, O,
            ctypes.c_void_p(yh.data_ptr()), tdq.F32, ctypes.c_void_p(xs[0].data_ptr()),
            ctypes.c_void_p(codes[0].data_ptr()), ctypes.c_void_p(scales[0].data_ptr()),
            ctypes.c_void_p(ys[0].data_ptr()), ctypes.c_void_p(wsp.data_ptr()), wsp.numel(), ctypes.c_void_p(stream))
        if rc != tdq.OK:
            raise RuntimeError("tdq_quant_linear_host: " + tdq.status_string(rc))

    e2e_steps = max(2, min(args.steps, 5))
    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    total_ms, q_ms, l_ms, e2e_ms = max_over_ranks([total_ms, q_ms, l_ms, e2e_ms], dev, world)
    fused = sweep = small = probe = None
    q_iso_ms = l_iso_ms = None
    q_switch_ms = None
    q_nchw = None
    pow2 = None
    if world == 1 and not args.no_extras:
        # each kernel on its own, launched back to back from a graph over rotating buffers: no other
        # kernel and no event node between two launches (the in-step figures above include those gaps)
        if not G:
            xi = xs + [xs[0].clone() for _ in range(n_iso - nsets)]
        # the same steps with an event record in front of and behind every call (what a graph with event
        # nodes measures; kept to show the difference)
        evx = [[torch.cuda.Event(enable_timing=True, external=True) for _ in range(3)] for _ in range(2 * nsets)]
        gx = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gx):
            for i in range(2 * nsets):
                step(i, evx[i])
        gx.replay()
        gx.replay()
        torch.cuda.synchronize()
        q_iso_ms = sum(e[0].elapsed_time(e[1]) for e in evx) / len(evx)
        l_iso_ms = sum(e[1].elapsed_time(e[2]) for e in evx) / len(evx)
        del gx
        # the quantizer with one or both bounds switched off (the paper's C1-only, C2-only and
        # DSTG-only ablation settings), back to back like the line above
        q_switch_ms = {}
        for label, flags in (("c1_only", tdq.ENABLE_C1), ("c2_only", tdq.ENABLE_C2), ("dstg_only", 0)):
            pf = tdq.act_params(flags=flags)
            q_switch_ms[label] = time_graph(lambda i: tdq.quantize_act(xi[i % n_iso], pf, codes=codes[i % nsets],
                                                                       scale=scales[i % nsets]), 4 * n_iso)
        pp = tdq.act_params(p=0.95)     # base radius = 31st of the 32 magnitudes (Supp. S4.8's percentile option)
        q_switch_ms["percentile_0.95"] = time_graph(lambda i: tdq.quantize_act(xi[i % n_iso], pp, codes=codes[i % nsets],
                                                                               scale=scales[i % nsets]), 4 * n_iso)
        # the fixed-radius control: no reductions, the speed limit of a one-pass quantizer of this size
        q_switch_ms["fixed_radius"] = time_graph(lambda i: tdq.quantize_act_fixed(xi[i % n_iso], 1.0, 32, codes=codes[i % nsets],
                                                                                 scale=scales[i % nsets]), 4 * n_iso)
        del xi
        # channel-major input of the same volume: a [B, C, 24, 24] feature map quantized along C in place
        fm = [torch.randn((32, C, 24, 24), device=dev).mul_(torch.randn((32, 1, 24, 24), device=dev).exp_())
              .to(torch.bfloat16 if case.x_is_bf16 else torch.float32) for _ in range(n_iso)]
        Mf = 32 * 24 * 24
        fcodes = torch.empty((Mf, C // 2), dtype=torch.uint8, device=dev)
        fscale = torch.empty((Mf, C // 32), dtype=torch.float32, device=dev)
        q_nchw_ms = time_graph(lambda i: tdq.quantize_act_nchw(fm[i % n_iso], params, codes=fcodes, scale=fscale), 4 * n_iso)
        q_nchw = dict(name="tdq_quantize_act_nchw", x=[32, C, 24, 24], ms=q_nchw_ms,
                      gbs=quant_bytes(Mf, C, esize) / (q_nchw_ms * 1e-3) / 1e9)
        del fm, fcodes, fscale
        # the power-of-two step variant (not the paper's quantizer): its quantizer and its linear layer
        p2 = tdq.act_params(flags=tdq.ENABLE_C1 | tdq.ENABLE_C2 | tdq.POW2_STEP)
        tdq.quantize_act(xs[0], p2, codes=codes[0], scale=scales[0])
        pl_ms = time_graph(lambda i: tdq.w4a4_linear_pow2(codes[0], scales[0], wcodes, wscale, y=ys[i % nsets], workspace=wsp),
                           8 * nsets)
        pow2 = dict(name="tdq_w4a4_linear_pow2", ms=pl_ms, tops=2.0 * M * C * O / (pl_ms * 1e-3) / 1e12,
                    gbs=linear_bytes(M, C, O) / (pl_ms * 1e-3) / 1e9)
        fused = fused_leg(tdq, xs, wcodes, wscale, ys, wsp, M, C, O, esize)
        del xs, codes, scales, ys
        torch.cuda.empty_cache()
        sweep = sweep_leg(tdq, dev)
        torch.cuda.empty_cache()
        peaks_x = load_peaks()
        small = small_configs_leg(tdq, dev, peaks_x)
        probe = probe_leg(tdq, dev, peaks_x)

    if rank == 0:
        peaks = load_peaks()
        K = args.steps
        qb, lb = quant_bytes(M, C, esize), linear_bytes(M, C, O)
        ops = 2.0 * M * C * O
        q_gbs = qb * K / (q_ms * 1e-3) / 1e9
        l_gbs = lb * K / (l_ms * 1e-3) / 1e9
        l_tops = ops * K / (l_ms * 1e-3) / 1e12
        int8_peak = 2.0 * peaks["bf16_tflops"]            # nominal int8 : bf16 ratio on the measured bf16 peak
        # the library's own figure: clocks per 128 x 128 x 32 instruction with operands resident in shared memory
        mma_peak = None
        if world == 1 and not args.no_extras:
            n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
            clk_max = (clocks or {}).get("sm_max_mhz") or 1965.0
            mma_peak = {}
            for label, kind in (("e4m3_f32acc", False), ("int8_int32acc", True)):
                cpm = tdq.measure_mma_clocks(kind, 8192, dev)
                mma_peak[label] = dict(clocks_per_mma=cpm, tops_at_max_clock=2.0 * 128 * 128 * 32 * n_sm * clk_max * 1e6 / cpm / 1e12)
            mma_peak["sm_max_mhz"] = clk_max
        q_kernel = dict(name="tdq_quantize_act", ms=q_ms / K, gbs=q_gbs, frac_hbm=q_gbs / peaks["hbm_gbs"],
                        frac_hbm_8tbs=q_gbs / 8000.0, algorithmic_bytes=qb)
        timing = ("events around launches of this call alone, replayed from a CUDA graph over rotating buffers" if G
                  else "events around every call, launched from the host")
        q_kernel["timing"] = timing
        if q_iso_ms:
            q_kernel.update(ms_between_event_nodes_in_step=q_iso_ms, ms_by_setting=q_switch_ms)
        l_kernel = dict(name="tdq_w4a4_linear", ms=l_ms / K, tops=l_tops, frac_int8=l_tops / int8_peak,
                        frac_int8_4500=l_tops / 4500.0, gbs=l_gbs, frac_hbm=l_gbs / peaks["hbm_gbs"],
                        algorithmic_bytes=lb, ops=ops,
                        bound="hbm" if lb / peaks["hbm_gbs"] / 1e9 > ops / int8_peak / 1e12 else "tensor")
        l_kernel["timing"] = timing
        if mma_peak:
            l_kernel["frac_int8_measured_issue_rate"] = l_tops / mma_peak["e4m3_f32acc"]["tops_at_max_clock"]
        if warm:
            q_kernel["ms_warm"], l_kernel["ms_warm"] = warm["quantize_ms"], warm["linear_ms"]
        if l_iso_ms:
            l_kernel.update(ms_between_event_nodes_in_step=l_iso_ms)
        if l_ms >= q_ms:
            if l_kernel["bound"] == "hbm":
                roof = dict(kernel="tdq_w4a4_linear", bound="hbm", achieved=l_gbs, peak=peaks["hbm_gbs"],
                            unit="GB/s", frac=l_gbs / peaks["hbm_gbs"],
                            traffic=profiled_traffic("w4a4_g32_kernel", args.workload, LINEAR_G32_SOURCES))
            else:
                roof = dict(kernel="tdq_w4a4_linear", bound="tensor", achieved=l_tops, peak=int8_peak,
                            unit="TOP/s", frac=l_tops / int8_peak, traffic=None)
        else:
            roof = dict(kernel="tdq_quantize_act", bound="hbm", achieved=q_gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=q_gbs / peaks["hbm_gbs"], traffic=None)
        roof["peak_source"] = peaks["source"]
        e2e_value = world * qb * e2e_steps / (e2e_ms * 1e-3) / 1e9
        out = dict(metric=METRIC, value=world * q_gbs, unit="GB/s", n_gpus=world, steps=K, warmup=args.warmup,
                   ms_per_step=total_ms / K, higher_is_better=True, scaling="weak", vs_baseline=None,
                   dtype="f32",
                   data="synthetic",
                   config=dict(workload=case.name, x=[int(v) for v in case.x.shape], w=[int(v) for v in case.w.shape],
                               g=32, tau=1.0, zr=0.2, y_dtype="f32",
                               cache="rotating %d buffer sets, %.0f MB per step (L2 is 126 MB)" % (nsets, step_bytes / 1e6),
                               launch=("CUDA graph of %d steps without event nodes, replayed %d times; each kernel timed from a graph of its call alone" % (G, args.steps // G)) if G else "eager",
                               parallelism="rows sharded, %d replica(s)" % world),
                   kernels=dict(quantize_act=q_kernel, quantize_act_nchw=q_nchw, w4a4_linear=l_kernel, w4a4_linear_pow2=pow2, fused=fused, sweep_cfg5=sweep, configs_1_to_3=small, compute_probe=probe,
                                step_tokens_per_s=world * M * K / (total_ms * 1e-3)),
                   roofline=roof, clocks=clocks, sustained=sustained, mma_peak=mma_peak, gpu_launches=int(launches),
                   e2e=dict(value=e2e_value, unit="GB/s", ms_per_step=e2e_ms / e2e_steps,
                            h2d_bytes_per_step=int(M * C * esize), d2h_bytes_per_step=int(M * O * 4),
                            api="tdq_quant_linear_host"))
        if world == 1 and not args.no_cpu_baseline:
            leg = cpu_oracle_leg(case, min(M, args.cpu_rows))
            out["cpu_baseline"] = dict(value=leg["quant_gbs"], unit="GB/s", cores=leg["cores"], kind="oracle",
                                       sample="first %d of %d token rows of %s, quantizer then linear, once"
                                              % (leg["rows"], M, case.name),
                                       linear_tops=leg["linear_tops"], quant_s=leg["quant_s"],
                                       linear_s=leg["linear_s"])
            one = cpu_oracle_single_thread(args.workload, min(M, 1024))
            if one:
                out["cpu_baseline"]["single_thread"] = dict(value=one["quant_gbs"], unit="GB/s", linear_tops=one["linear_tops"],
                                                            sample="first %d token rows" % one["rows"])
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="default: 1000 (10 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="tdq", choices=["tdq", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=["cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--cpu-rows", type=int, default=18464)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="only the timed steps, the per-kernel timings and the end-to-end leg (for profiler runs)")
    ap.add_argument("--oracle-leg", type=int, default=0, help=argparse.SUPPRESS)
    ap.add_argument("--eager", action="store_true", help="launch every timed step from the host instead of replaying a CUDA graph")
    ap.add_argument("--probe-only", action="store_true", help="only the compute-bound probe shape of the linear layer (for profiler runs); prints that leg")
    ap.add_argument("--pow2-only", action="store_true", help="only the power-of-two variant of the linear layer on --workload (for profiler runs); prints that leg")
    args = ap.parse_args()
    if args.oracle_leg:                    # child of cpu_oracle_single_thread
        print(json.dumps(cpu_oracle_leg(workload(args.workload), args.oracle_leg)))
        return
    if args.probe_only:
        import torch
        from paper_2604_16855_b200 import tdq
        print(json.dumps(dict(compute_probe=probe_leg(tdq, torch.device("cuda", 0), load_peaks()))))
        return
    if args.pow2_only:
        import torch
        from paper_2604_16855_b200 import tdq
        print(json.dumps(dict(w4a4_linear_pow2=pow2_leg(tdq, torch.device("cuda", 0), args.workload))))
        return
    if args.steps is None:
        args.steps = 10 if args.impl == "reference" else 1000
    if args.impl == "reference":
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_tdq(args)


if __name__ == "__main__":
    main()
