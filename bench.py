#!/usr/bin/env python
"""Benchmark of the DSQ low-bit convolution path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole hot path over one batch of the
ResNet-18-shaped 4-bit workload (batch 64, 56x56x64 stem output): quantise the
fp32 activations to packed codes, then the 19 quantised convolutions with
fused dequantise / residual / requantise epilogues (20 kernel launches).  The
calls are captured in CUDA graphs and replayed; the input rotates over
several buffers whose total size exceeds L2.

Prints ONE JSON line.  `value` is images/s with inputs resident in HBM; `e2e`
is the same through the C-ABI calls with the input in pinned host memory and
the result read back.  `roofline` describes the dominant kernel (the
tensor-core convolution); `extras` carries the 4096^3 4-bit GEMM and the
quantise-kernel bandwidth; `cpu_baseline` is the CPU oracle timed on the host
cores on a bounded sample.  With N > 1 every rank runs the same step on its own
GPU (replicas; the path has no exchange step) and the images of all ranks are
summed over the slowest rank's time.
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import dsq_inputs  # noqa: E402

# DRAM traffic of the tensor-core convolution kernels per launch in this
# workload, from one ncu capture (profiles/bench_launch_list.txt); valid only
# for the kernel sources it was taken on (checked by hash)
TRAFFIC = {"bytes_per_launch": 4788042, "sources_sha256": "585f1a5645589bf21d02a3907c39fa0f79a688af8ef574aeb29a2ef435337442"}

WORKLOAD = "resnet18-shaped stack, 4-bit W/A, batch 64, 56x56x64 stem output, 19 convs"
METRIC = "4-bit ResNet-18 conv-stack throughput (effective low-bit conv TOPS alongside)"
INT8_NOMINAL_TOPS = 4500.0


# ---------------------------------------------------------------------------
# helpers
# ---------------------------------------------------------------------------
def kernel_sources_sha256():
    import hashlib
    h = hashlib.sha256()
    for f in ("dsq_tc.cu", "dsq_conv3.cu", "dsq_tc_common.cuh", "dsq_ptx.cuh", "dsq_epilogue.cuh",
              "dsq_common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_1908_05033_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def measured_traffic():
    if TRAFFIC["bytes_per_launch"] is None:
        return None
    return TRAFFIC["bytes_per_launch"] if TRAFFIC["sources_sha256"] == kernel_sources_sha256() else None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sustained=1400.0,
                source="fallback")


class ClockSampler:
    """Polls SM clock, power and the clock-event (throttle) reasons of one GPU
    through NVML from a thread of this process, every ~1 ms, read-only.
    Samples carry the phase that was current when they were taken ("timed",
    "e2e", ...), so that a timed region of a few milliseconds still gets its
    own record.  `sample_now()` takes one sample synchronously (used right
    after the timed launches have been enqueued, while the GPU is still
    running them)."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown",
               0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, torch_index):
        self.phase, self.samples, self.h, self.nv = "setup", [], None, None
        self._stop = threading.Event()
        self.thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(torch_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(torch_index)
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:          # no NVML: the record says so
            self.err = f"NVML unavailable: {e}"
            self.h = None

    def sample_now(self):
        if self.h is None:
            return
        nv = self.nv
        try:
            sm = float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            try:
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception:
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            pw = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
            self.samples.append((self.phase, sm, mask, pw))
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample_now()
            time.sleep(0.001)

    def start(self):
        if self.h is not None:
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()

    def stop(self):
        self._stop.set()
        if self.thread is not None:
            self.thread.join(timeout=2)

    def summary(self, phase):
        if self.h is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0,
                    "reasons": [getattr(self, "err", "NVML unavailable")]}
        rows = [r for r in self.samples if r[0] == phase]
        reasons = set()
        for _, _, mask, _ in rows:
            for bit, name in self.REASONS.items():
                if mask & bit:
                    reasons.add(name)
        return {"sm_mhz": statistics.median(r[1] for r in rows) if rows else None,
                "sm_max_mhz": self.max_sm,
                "power_w_max": max(r[3] for r in rows) if rows else None,
                "samples": len(rows), "reasons": sorted(reasons),
                "how": "NVML polled in-process every ~1 ms during the phase"}


def dist_setup(n_gpus):
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend)
    return rank, world, local


def aggregate(local_ms, local_units, device=None):
    """Whole-job figures over all ranks: (max time in ms, total units).  No
    data-path collective exists on this path; this is measurement only."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_ms), float(local_units)
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def barrier(device=None):
    import torch
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


# ---------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------
class OracleSample:
    """ONE definition of the CPU baseline, used by both the `cpu_baseline` leg
    and `--impl reference`: the oracle's run_stack (activation quantise, weight
    quantise, every convolution with S_a, bias, residual and requantise) on one
    synthetic image of the ResNet-18-shaped stack.  A sample is either a whole
    56x56 image or, where a bounded sample is needed, the same stack on a
    smaller crop (28, 14 or 8 pixels square); its work is counted in
    multiply-accumulates and converted to images of the full workload."""

    def __init__(self, wid=3):
        self.wid = wid
        self.full = dsq_inputs.resnet18_stack()
        self.params = dsq_inputs.stack_params(self.full, workload_id=wid)
        self.cache = {}

    def step(self, hw):
        """Runs one sample; returns the fraction of a full image it covers."""
        from oracle import stack as ostack
        if hw not in self.cache:
            st = dsq_inputs.resnet18_stack(hw=hw)
            x = dsq_inputs.stack_input(st, batch=1, workload_id=self.wid)
            self.cache[hw] = (st, x, st.macs_per_image() / self.full.macs_per_image())
        st, x, frac = self.cache[hw]
        ostack.run_stack(st, x, self.params, keep=[st.out])
        return frac

    def describe(self, hw, n, dt):
        what = "whole 56x56 images" if hw == 56 else f"{hw}x{hw} crops of the 56x56 input"
        return (f"{n} single-image passes of oracle.stack.run_stack over all 19 conv layers "
                f"(+ activation and weight quantise) on {what}, {dt:.1f} s")


def cpu_baseline_whole_images(budget_s=15.0):
    """The oracle as it stands on whole images for about `budget_s` seconds."""
    from oracle import native
    o = OracleSample()
    o.step(56)                                              # warm
    n, t0 = 0, time.perf_counter()
    while True:
        o.step(56)
        n += 1
        dt = time.perf_counter() - t0
        if dt > budget_s or n >= 200:
            break
    return {"value": n / dt, "unit": "img/s", "cores": native.num_threads(),
            "kind": "oracle", "sample": o.describe(56, n, dt)}


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores.  Each step is one
    bounded sample (OracleSample); the crop is chosen so that the whole run
    stays within about two minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import native
    o = OracleSample()
    o.step(56)                                              # warm (builds the weights' codes)
    t0 = time.perf_counter()
    o.step(56)
    t56 = time.perf_counter() - t0
    total = args.steps + args.warmup
    hw = 56
    for cand, cost in ((56, 1.0), (28, 0.25), (14, 1.0 / 16), (8, 1.0 / 49)):
        hw = cand
        if total * t56 * cost <= 120.0:
            break
    for _ in range(args.warmup):
        o.step(hw)
    t0 = time.perf_counter()
    imgs = 0.0
    for _ in range(args.steps):
        imgs += o.step(hw)
    dt = time.perf_counter() - t0
    value = imgs / dt
    macs = imgs * o.full.macs_per_image()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "img/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8xint8->int32 (4-bit codes)",
        "data": "synthetic",
        "config": workload_config(1),
        "effective_tops": 2.0 * macs / dt / 1e12,
        "cpu_baseline": {"value": value, "unit": "img/s", "cores": native.num_threads(),
                         "kind": "oracle", "sample": o.describe(hw, args.steps, dt)},
        "e2e": {"value": value, "unit": "img/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------
def time_graphs(graphs, steps, warmup, torch, sampler=None, phase="timed"):
    for i in range(warmup):
        graphs[i % len(graphs)].replay()
    barrier()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    if sampler is not None:
        sampler.phase = phase
    e0.record()
    for i in range(steps):
        graphs[i % len(graphs)].replay()
    e1.record()
    if sampler is not None:
        sampler.sample_now()        # enqueued, still running: one sure sample under load
    torch.cuda.synchronize()
    if sampler is not None:
        sampler.phase = "idle"
    barrier()
    return e0.elapsed_time(e1)


def workload_config(world, n_in=4, in_mb=206):
    return {"workload": WORKLOAD, "bits": 4, "global_batch": 64 * world,
            "parallelism": f"replicas x{world}", "cuda_graph": True,
            "l2": f"input rotates over {n_in} buffers ({in_mb} MB) > 126 MB L2",
            "w_offset": 0.5}


def kernel_times_eager(g, xs, torch, reps=5):
    """Per-kernel device time of one forward pass: CUDA events around every
    launch, on the launching stream, median over `reps` passes."""
    from paper_1908_05033_b200 import binding as B
    import paper_1908_05033_b200 as dsq
    names, evs = [], []
    orig = {n: getattr(B.lib, n) for n in ("dsq_quantize_act", "dsq_conv2d")}
    per_rep = []
    for r in range(reps):
        marks = []
        x = xs[r % len(xs)]
        # quantise
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record()
        dsq.dsq_quantize_act(x, g.bits, g.st.in_lo, g.st.in_hi, out=g.codes["in"])
        b.record()
        marks.append(("dsq_quantize_act", "in", a, b))
        for L, w in g.layers:
            H, W, Cc = g.shapes[L.src]
            shape = (g.batch, H, W, Cc)
            a_lo, a_hi = g.ranges[L.src]
            res = res_q = None
            if L.residual is not None:
                res = g.codes[L.residual]
                res_q = (g.bits,) + tuple(g.ranges[L.residual])
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record()
            dsq.dsq_conv2d(g.codes[L.src], shape, (g.bits, a_lo, a_hi), w["blob"], w["conv"],
                           w["scale"], w["bias"], g.ws, w_offset=g.w_offset, residual=res,
                           residual_q=res_q, requant=(g.bits, L.out_lo, L.out_hi),
                           out_codes=g.codes[L.dst])
            b.record()
            marks.append(("dsq_conv2d", L.name, a, b))
        torch.cuda.synchronize()
        per_rep.append([(k, n, a.elapsed_time(b)) for k, n, a, b in marks])
    out = []
    for i in range(len(per_rep[0])):
        k, n, _ = per_rep[0][i]
        out.append((k, n, statistics.median(rep[i][2] for rep in per_rep)))
    return out


def algorithmic_bytes_step(st, batch):
    """Packed code bytes every conv of the stack must move for one batch: its
    input codes, its residual codes, its output codes and its packed weights."""
    shapes = st.tensor_shapes()
    b = st.bits / 8.0
    total = 0.0
    for L in st.layers:
        if L.kind == "pool":
            continue
        Hi, Wi, Ci = shapes[L.src]
        Ho, Wo, Co = shapes[L.dst]
        total += batch * (Hi * Wi * Ci + Ho * Wo * Co) * b
        if L.residual is not None:
            total += batch * Ho * Wo * Co * b
        total += Co * L.ksize * L.ksize * (1 if L.kind == "dw" else Ci) * b
    return total


def time_other_stack(st, wid, torch, dev, steps=50):
    """ms per step and images/s of another workload's stack (graph replay)."""
    from paper_1908_05033_b200.stack import GpuStack
    params = dsq_inputs.stack_params(st, workload_id=wid)
    x = torch.from_numpy(dsq_inputs.stack_input(st, workload_id=wid)).to(dev)
    g = GpuStack(st, params, device=dev)
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        g.forward(x)
        torch.cuda.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=side):
            g.forward(x)
    torch.cuda.synchronize()
    for _ in range(5):
        gr.replay()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        gr.replay()
    e1.record(); torch.cuda.synchronize()
    g.check()
    ms = e0.elapsed_time(e1) / steps
    return {"ms_per_step": ms, "img_per_s": st.batch / (ms * 1e-3),
            "effective_tops": 2.0 * st.macs_per_image() * st.batch / (ms * 1e-3) / 1e12,
            "batch": st.batch, "bits": st.bits, "launches_per_step": g.n_launches()}


def run_ours(args):
    import torch
    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    import paper_1908_05033_b200 as dsq
    from paper_1908_05033_b200.stack import GpuStack
    peaks = load_peaks()

    st = dsq_inputs.resnet18_stack()
    wid = 3
    params = dsq_inputs.stack_params(st, workload_id=wid)
    x_host = dsq_inputs.stack_input(st, workload_id=wid)          # [64,56,56,64] fp32
    batch = st.batch
    g = GpuStack(st, params, device=dev)
    n_in = 4                                                      # 4 x 51 MB > L2
    xs = [torch.from_numpy(np.roll(x_host, i, axis=0)).to(dev) for i in range(n_in)]

    # capture one graph per input buffer: the whole step (quantise + 19 convs),
    # and the 19 convolutions alone (the dominant kernel, timed the same way)
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream())
    graphs, conv_graphs = [], []
    with torch.cuda.stream(side):
        g.forward(xs[0])
        torch.cuda.synchronize()
        for x in xs:
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=side):
                g.forward(x)
            graphs.append(gr)
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=side):
            g.forward(None)                     # codes["in"] as the last quantise left it
        conv_graphs.append(gr)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    ms = time_graphs(graphs, args.steps, args.warmup, torch, sampler, "timed")
    clocks = sampler.summary("timed")
    g.check()
    ms_all, imgs_all = aggregate(ms, batch * args.steps, dev)
    value = imgs_all / (ms_all * 1e-3)
    macs_step = st.macs_per_image() * batch
    eff_tops = 2.0 * macs_step * args.steps * world / (ms_all * 1e-3) / 1e12

    # ---- dominant kernel: the 19 tensor-core convolutions --------------------
    # Timed live with CUDA events over the same number of replays of a graph
    # that holds the 19 convolutions only (events cannot sit between the nodes
    # of the full step's graph).  Per-launch eager times go to extras.
    conv_ms_total = time_graphs(conv_graphs, args.steps, args.warmup, torch, sampler, "conv_only")
    kt = kernel_times_eager(g, xs, torch)
    conv_ms = sum(t for k, _, t in kt if k == "dsq_conv2d")
    quant_ms = sum(t for k, _, t in kt if k == "dsq_quantize_act")
    n_conv = g.n_launches() - 1
    step_ms = ms / args.steps
    conv_in_step_ms = conv_ms_total / args.steps
    # a region of well under a second runs at boost clocks without the power
    # cap: the burst figure of the measured peaks applies; the sustained one
    # is for regions of seconds
    burst = conv_ms_total < 1000.0
    bf16_peak = peaks["bf16_tflops"] if burst else peaks["bf16_sustained"]
    int8_peak = 2.0 * bf16_peak                 # int8 : bf16 nominal ratio 2
    achieved = 2.0 * macs_step / (conv_in_step_ms * 1e-3) / 1e12
    roofline = {
        "kernel": f"dsq_win3_kernel (3x3 stride 1) + dsq_tc_kernel (1x1, strided) behind dsq_conv2d, "
                  f"{n_conv} launches per step",
        "bound": "tensor", "achieved": achieved, "peak": int8_peak, "unit": "TOP/s",
        "frac": achieved / int8_peak,
        "peak_source": f"2 x bf16_tflops{'' if burst else '_sustained'} of {peaks['source']} peaks "
                       f"(int8:bf16 nominal ratio 2; {'burst' if burst else 'sustained'} figure: the "
                       f"timed region lasts {conv_ms_total:.1f} ms); nominal 4500, own MMA-only probe in extras",
        "frac_of_nominal_4500": achieved / INT8_NOMINAL_TOPS,
        "avg_launch_ms": conv_in_step_ms / n_conv,
        "how": f"CUDA events around {args.steps} replays of a graph holding the {n_conv} convolutions only",
        "clocks": sampler.summary("conv_only"),
        "traffic": measured_traffic(),
        "algorithmic_bytes_per_launch": algorithmic_bytes_step(st, batch) / n_conv,
    }

    line = {
        "metric": METRIC, "value": value, "unit": "img/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_all / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8xint8->int32 (4-bit codes)", "data": "synthetic",
        "config": workload_config(world, n_in, round(n_in * x_host.nbytes / 1e6)),
        "effective_tops": eff_tops,
        "pct_int8_nominal_peak": 100.0 * eff_tops / world / INT8_NOMINAL_TOPS,
        "clocks": clocks,
        "gpu_launches": g.n_launches() * args.steps,
        "roofline": roofline,
    }

    if rank == 0:
        # ---- end to end through the C ABI with host buffers ---------------
        # Every step copies its fp32 input from pinned host memory, runs the 20
        # calls and reads the output codes back.  The copy of step i+1 runs on a
        # second stream while step i computes (two device input buffers).
        pinned = [torch.from_numpy(np.roll(x_host, i, axis=0)).pin_memory() for i in range(2)]
        x_dev = [torch.empty_like(xs[0]) for _ in range(2)]
        out_host = torch.empty_like(g.codes[st.out], device="cpu").pin_memory()
        e2e_steps = max(3, min(args.steps, 40))
        main = torch.cuda.current_stream()
        copy_s = torch.cuda.Stream(device=dev)
        copied = [torch.cuda.Event() for _ in range(2)]
        consumed = [torch.cuda.Event() for _ in range(2)]

        def e2e_run(n):
            for b in range(2):
                consumed[b].record(main)
            with torch.cuda.stream(copy_s):
                copy_s.wait_event(consumed[0])
                x_dev[0].copy_(pinned[0], non_blocking=True)
                copied[0].record(copy_s)
            for i in range(n):
                b = i & 1
                if i + 1 < n:
                    with torch.cuda.stream(copy_s):
                        copy_s.wait_event(consumed[b ^ 1])
                        x_dev[b ^ 1].copy_(pinned[(i + 1) & 1], non_blocking=True)
                        copied[b ^ 1].record(copy_s)
                main.wait_event(copied[b])
                g.forward(x_dev[b])
                consumed[b].record(main)
                out_host.copy_(g.codes[st.out], non_blocking=True)

        e2e_run(3)
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        sampler.phase = "e2e"
        e0.record()
        e2e_run(e2e_steps)
        e1.record()
        torch.cuda.synchronize()
        sampler.phase = "idle"
        e2e_ms = e0.elapsed_time(e1)
        line["e2e"] = {"value": batch * e2e_steps / (e2e_ms * 1e-3) * world, "unit": "img/s",
                       "h2d_bytes_per_step": int(x_host.nbytes),
                       "d2h_bytes_per_step": int(out_host.numel()),
                       "steps": e2e_steps, "clocks": sampler.summary("e2e"),
                       "h2d_gbs": x_host.nbytes * e2e_steps / (e2e_ms * 1e-3) / 1e9,
                       "note": "per step: pinned fp32 input -> device (second stream, overlapping the "
                               "previous step), dsq_quantize_act + 19 dsq_conv2d, output codes -> host"}

        # ---- extras: quantise bandwidth, 4096^3 GEMM, MMA-only rate --------
        extras = {}
        ws = dsq.new_workspace(dev)
        try:
            tops, _ = dsq.dsq_probe_i8_mma_rate(20000, ws)
            extras["int8_mma_only_tops"] = tops
        except Exception as e:      # measurement aid only
            extras["int8_mma_only_tops"] = f"failed: {e}"
        # quantise kernel on a > L2 tensor (1 GiB fp32), b = 4
        big = torch.empty((64, 256, 256, 64), dtype=torch.float32, device=dev).normal_()
        outq = torch.empty((64, 256, 256, 32), dtype=torch.uint8, device=dev)
        for _ in range(3):
            dsq.dsq_quantize_act(big, 4, 0.0, 2.0, out=outq)
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            dsq.dsq_quantize_act(big, 4, 0.0, 2.0, out=outq)
        e1.record(); torch.cuda.synchronize()
        qms = e0.elapsed_time(e1) / 10
        gbs = big.numel() * 4.5 / (qms * 1e-3) / 1e9
        extras["quantize_act_b4_1GiB"] = {"GB/s": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
                                          "ms": qms, "bytes_per_element": 4.5}
        del big, outq
        # training-side soft quantiser (Eq. 5 forward, Eq. 10-13 backward), 512 MiB fp32
        xs_ = torch.empty(1 << 27, dtype=torch.float32, device=dev).normal_()
        gs_ = torch.empty_like(xs_).normal_()
        ys_ = torch.empty_like(xs_)
        gp_ = torch.empty(3, dtype=torch.float64, device=dev)
        for name, fn, bpe in (("fwd", lambda: dsq.dsq_soft_quantize_fwd(xs_, 4, -1.0, 2.0, 0.2, out=ys_), 8.0),
                              ("bwd", lambda: dsq.dsq_soft_quantize_bwd(xs_, gs_, 4, -1.0, 2.0, 0.2, out=ys_,
                                                                        grad_params=gp_), 12.0)):
            for _ in range(3):
                fn()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                fn()
            e1.record(); torch.cuda.synchronize()
            sms = e0.elapsed_time(e1) / 10
            sgbs = xs_.numel() * bpe / (sms * 1e-3) / 1e9
            extras["soft_quantize_" + name + "_b4_512MiB"] = {
                "GB/s": sgbs, "frac_of_hbm_peak": sgbs / peaks["hbm_gbs"], "ms": sms,
                "bytes_per_element": bpe}
        del xs_, gs_, ys_, gp_
        # 4-bit GEMMs: dsq_gemm with the workspace dsq_gemm_workspace_bytes asks for
        # (rows expanded to 8-bit once, then an 8-bit tensor-core GEMM fed by TMA)
        # and, beside it, with the small workspace (one fused kernel)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

        def time_gemm(size, gws):
            A, Bm, rs = dsq_inputs.gemm_case(size, size, size, 4)
            Ap = dsq.dsq_pack_codes(torch.from_numpy(A).to(dev), 4)
            Bp = dsq.dsq_pack_codes(torch.from_numpy(Bm).to(dev), 4)
            Cm = torch.empty((size, size), dtype=torch.int32, device=dev)
            times = []
            for i in range(13):
                flush.zero_()
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record()
                dsq.dsq_gemm(Ap, Bp, size, size, size, 4, gws, out_i32=Cm)
                e1.record(); torch.cuda.synchronize()
                if i >= 3:
                    times.append(e0.elapsed_time(e1))
            dsq.check_workspace(gws, "extras gemm")
            gms = statistics.median(times)
            gt = 2.0 * size ** 3 / (gms * 1e-3) / 1e12
            return {"ms": gms, "tops": gt, "frac_of_nominal_4500": gt / INT8_NOMINAL_TOPS,
                    "frac_of_2x_bf16_burst": gt / (2 * peaks["bf16_tflops"]),
                    "l2": "256 MB flush between launches"}

        for size in (4096, 8192):
            g2 = time_gemm(size, dsq.new_gemm_workspace(size, size, size, 4, dev))
            g2["path"] = "two passes (expand rows to int8, 8-bit GEMM); both timed"
            g2["fused_kernel"] = time_gemm(size, ws)
            extras[f"gemm_{size}_b4"] = g2
        # binary GEMM (1-bit rows, +-1 values) and weight-only GEMM (bf16 x 4-bit)
        Ab, Bb, _ = dsq_inputs.binary_gemm_case(4096, 4096, 4096)
        Abp = dsq.dsq_pack_codes(torch.from_numpy(Ab).to(dev), 1)
        Bbp = dsq.dsq_pack_codes(torch.from_numpy(Bb).to(dev), 1)
        Cb = torch.empty((4096, 4096), dtype=torch.int32, device=dev)
        bws = torch.zeros(dsq.lib.dsq_binary_gemm_workspace_bytes(4096, 4096, 4096),
                          dtype=torch.uint8, device=dev)
        xw, qw, uw, _ = dsq_inputs.weight_only_case(4096, 4096, 4096, 4)
        Xw = torch.from_numpy(xw).to(dev).to(torch.bfloat16)
        Ww = dsq.dsq_pack_codes(torch.from_numpy((qw.astype(np.int16) - 8).astype(np.int8)).to(dev), 4)
        sw = torch.from_numpy((uw / 15).astype(np.float32)).to(dev)
        Yw = torch.empty((4096, 4096), dtype=torch.float32, device=dev)
        wws = torch.zeros(dsq.lib.dsq_wgemm_workspace_bytes(4096, 4096), dtype=torch.uint8, device=dev)
        stream = torch.cuda.current_stream().cuda_stream

        def run_bgemm():
            st_ = dsq.lib.dsq_binary_gemm(Abp.data_ptr(), Bbp.data_ptr(), 4096, 4096, 4096,
                                          Cb.data_ptr(), None, None, bws.data_ptr(), bws.numel(), stream)
            assert st_ == 0

        def time_call(fn):
            times = []
            for i in range(13):
                flush.zero_()
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(); fn(); e1.record(); torch.cuda.synchronize()
                if i >= 3:
                    times.append(e0.elapsed_time(e1))
            return statistics.median(times)

        bms = time_call(run_bgemm)
        dsq.check_workspace(bws, "extras binary gemm")
        extras["binary_gemm_4096"] = {"ms": bms, "tops": 2.0 * 4096 ** 3 / (bms * 1e-3) / 1e12,
                                      "frac_of_nominal_4500": 2.0 * 4096 ** 3 / (bms * 1e-3) / 1e12 / INT8_NOMINAL_TOPS}
        wms = time_call(lambda: dsq.dsq_wgemm_bf16(Xw, Ww, 4096, 4096, 4096, 4, sw, ws=wws, out=Yw))
        dsq.check_workspace(wws, "extras weight-only gemm")
        wt = 2.0 * 4096 ** 3 / (wms * 1e-3) / 1e12
        extras["weight_only_gemm_4096_w4_bf16"] = {"ms": wms, "tflops": wt,
                                                   "frac_of_bf16_burst": wt / peaks["bf16_tflops"]}
        dsq.check_workspace(ws, "extras")
        del flush, Abp, Bbp, Cb, bws, Xw, Ww, Yw, wws
        extras["mobilenetv2_stack_b4_batch64"] = time_other_stack(
            dsq_inputs.mobilenetv2_stack(), 4, torch, dev)
        extras["vgg16_stack_b2_batch32"] = time_other_stack(dsq_inputs.vgg16_stack(), 5, torch, dev)
        extras["quantize_in_step_ms"] = quant_ms
        extras["conv_kernels_in_step_ms"] = conv_ms
        extras["per_layer_ms"] = {n: round(t, 4) for _, n, t in kt}
        line["extras"] = extras

        # ---- CPU oracle beside it ----------------------------------------------
        line["cpu_baseline"] = cpu_baseline_whole_images()
        sampler.stop()
        print(json.dumps(line))
    else:
        sampler.stop()
    barrier()
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
