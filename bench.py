#!/usr/bin/env python
"""Benchmark of the quantized layer: prints ONE JSON line.

Own arm (default): the DDIM-CIFAR-style 3x3 convolution, W8A8 (E4M3 weights with
rounding decisions, E4M3 activations), input FP32 NCHW [64,128,32,32] -> 128
channels, through the C-ABI library on the GPU.  A step is one fpq_conv2d call
(activation quantize + contraction + dequantize/bias); weights are encoded once
before the timed region (the encode's own time is reported separately).  The
steps rotate over several resident copies of (input, scratch, output) whose total
size is a multiple of the L2, so every step reads its input from HBM and its
writes push earlier steps' outputs out to HBM (inputs larger than L2); the K
timed steps are replayed as one CUDA graph so that host launch time is not part
of the number.  With N > 1 (torchrun) every rank runs its own copy of the layer on its own
batch: weak scaling, no collective on the data path.

Reference arm (--impl reference): the CPU oracle, as it stands, on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
import zlib

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "W8A8 and W4A8 quantized-layer TFLOP/s on 1 B200 and % of dense FP8/FP4 peak"
WORKLOAD = "ddim_cifar_conv3x3_w8a8: x fp32 NCHW [64,128,32,32] SiLU(N(0,1)), w [128,128,3,3] e4m3 + rounding bits, pad 1"
NOMINAL_FP8_TFLOPS = 4500.0
NOMINAL_FP4_TFLOPS = 9000.0
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_TF32_TFLOPS = 1100.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised under
# profiles/ (a kernel is absent here until a capture of its current form exists).
TRAFFIC = {
    # --cache-control none capture, second of three launches taken mid-rotation (write-backs included)
    "fpq_pair_conv_kernel (activation quantize + contraction + epilogue on CTA pairs)": 33718784 + 32794880,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ---------------------------------------------------------------------------------------------
# reference arm: the CPU oracle
# ---------------------------------------------------------------------------------------------
def oracle_sample_run(batch: int):
    """One pass of the oracle layer (quantize weights and activations, FP64 conv) on the
    first `batch` images of the workload.  Returns (seconds, flops, threads)."""
    import numpy as np
    import oracle as O
    from paper_2408_06995_b200 import inputs as I

    (L,) = I.config2(batch=batch)
    w2 = L.w.reshape(L.N, -1)
    ws = np.array([O.scale_from_max(v, O.E4M3) for v in np.abs(w2).max(axis=1)], dtype=np.float32)
    xs = O.scale_from_max(float(np.abs(L.x).max()), O.E4M3)
    rb = O.pack_bits(L.bits)
    O.lib()
    t0 = time.perf_counter()
    O.conv2d(L.x, L.w, ws, xs, O.E4M3, O.E4M3, L.bias, rb, L.pad, L.stride)
    dt = time.perf_counter() - t0
    return dt, L.flops, os.cpu_count()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # bounded sample per step, sized so that the whole run stays within a few minutes
    batch = 4 if args.steps <= 100 else (2 if args.steps <= 300 else 1)
    for _ in range(args.warmup):
        oracle_sample_run(batch)
    total, flops = 0.0, 0
    for _ in range(args.steps):
        dt, fl, cores = oracle_sample_run(batch)
        total += dt
        flops += fl
    value = flops / total / 1e12
    sample = f"first {batch} of 64 images of the workload per step, whole oracle layer"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# clock sampling during the timed region (NVML, read-only)
# ---------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.0005)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ---------------------------------------------------------------------------------------------
# own arm
# ---------------------------------------------------------------------------------------------
class LayerOnGpu:
    """Device-resident tensors of one quantized layer (conv or linear), weights already
    encoded.  Activations, scratch and outputs exist in several copies whose total size is a
    multiple of the L2; every call moves on to the next copy."""

    def __init__(self, L, fpq, torch, dev, l2_bytes=128 << 20, nsets=None):
        import numpy as np
        self.L, self.fpq, self.torch = L, fpq, torch
        self.fw = fpq.E4M3 if L.wfmt == "e4m3" else fpq.E2M1
        self.conv = L.kind == "conv"
        g = torch.Generator(device=dev)
        g.manual_seed(1000 + (zlib.crc32(L.name.encode()) & 0xffff))      # the same draws in every process
        if L.w is not None:
            self.w = torch.from_numpy(L.w.reshape(L.N, -1)).to(dev)
            self.bias = torch.from_numpy(L.bias).to(dev)
            x0 = torch.from_numpy(L.x).to(dev)
            self.rb = None if L.bits is None else torch.from_numpy(np.packbits(L.bits, axis=1, bitorder="little")).to(dev)
        else:
            # shape-only layer of a trace: seeded draws on the device (N(0,1) activations,
            # N(0,0.02) weights, Bernoulli(0.5) rounding decisions)
            xshape = (L.B, L.C, L.H, L.W) if self.conv else (L.M, L.K)
            x0 = torch.randn(xshape, generator=g, device=dev, dtype=torch.float32)
            self.w = torch.randn((L.N, L.K), generator=g, device=dev, dtype=torch.float32) * 0.02
            self.bias = torch.randn((L.N,), generator=g, device=dev, dtype=torch.float32) * 0.01
            self.rb = None
            if L.rounding:
                self.rb = torch.randint(0, 256, (L.N, (L.K + 7) // 8), generator=g, device=dev, dtype=torch.uint8)
        wmax = self.w.abs().amax(dim=1).cpu().numpy()
        self.ws = torch.tensor([fpq.fpq_scale_from_max(float(v), self.fw) for v in wmax], dtype=torch.float32, device=dev)
        self.xs = fpq.fpq_scale_from_max(float(x0.abs().max().item()), fpq.E4M3)
        if self.conv:
            self.ws_bytes = fpq.fpq_conv2d_workspace_size(L.B, L.C, L.H, L.W, L.N, L.R, L.S, L.pad, L.stride, fpq.E4M3, self.fw)
            yshape = (L.B, L.N, L.Ho, L.Wo)
        else:
            self.ws_bytes = fpq.fpq_linear_workspace_size(L.M, L.N, L.K, fpq.E4M3, self.fw)
            yshape = (L.M, L.N)
        self.x_elems = x0.numel()
        self.set_bytes = 4 * self.x_elems + 4 * L.M * L.N + self.ws_bytes
        self.nsets = nsets or max(2, -(-3 * l2_bytes // self.set_bytes))        # >= 3 x L2 in rotation
        self.xs_ = [x0] + [x0.clone() for _ in range(self.nsets - 1)]
        self.ys_ = [torch.empty(yshape, dtype=torch.float32, device=dev) for _ in range(self.nsets)]
        self.wss_ = [torch.empty(max(1, self.ws_bytes), dtype=torch.uint8, device=dev) for _ in range(self.nsets)]
        self.i = 0
        self._rot()
        self.encode()

    def _rot(self):
        self.i = (self.i + 1) % self.nsets
        self.x, self.y, self.workspace = self.xs_[self.i], self.ys_[self.i], self.wss_[self.i]

    def encode(self):
        f, L = self.fpq, self.L
        self.codes = f.fpq_quantize_weight(self.w, self.ws, self.fw, self.rb)
        if self.conv:
            self.prep = f.fpq_prepare_weight(self.codes, self.fw, f.CONV2D, L.N, L.C, L.R, L.S)
        else:
            self.prep = f.fpq_prepare_weight(self.codes, self.fw, f.LINEAR, L.N, L.K)

    def step(self):
        f, L = self.fpq, self.L
        self._rot()
        if self.conv:
            f.fpq_conv2d(self.x, self.prep, self.ws, self.xs, f.E4M3, self.fw, self.bias, L.N, L.R, L.S, L.pad,
                         L.stride, y=self.y, workspace=self.workspace)
        else:
            f.fpq_linear(self.x, self.prep, self.ws, self.xs, f.E4M3, self.fw, self.bias, L.N, y=self.y,
                         workspace=self.workspace)

    def stage1(self):
        f, L = self.fpq, self.L
        self._rot()
        if self.conv:
            f.fpq_conv2d_quantize_input(self.x, self.xs, f.E4M3, self.fw, L.N, L.R, L.S, L.pad, L.stride, self.workspace)
        else:
            f.fpq_linear_quantize_input(self.x, self.xs, f.E4M3, self.fw, L.N, self.workspace)

    def stage2(self):
        f, L = self.fpq, self.L
        self._rot()
        if self.conv:
            f.fpq_conv2d_contract(self.workspace, self.prep, self.ws, self.xs, f.E4M3, self.fw, self.bias, self.y,
                                  (L.B, L.C, L.H, L.W), L.R, L.S, L.pad, L.stride)
        else:
            f.fpq_linear_contract(self.workspace, self.prep, self.ws, self.xs, f.E4M3, self.fw, self.bias, self.y, L.K)

    def wbytes(self):
        return self.L.N * self.L.K * (1 if self.L.wfmt == "e4m3" else 0.5)

    # algorithmic bytes (FP32 activations in, FP32 out, encoded weights, scales + bias)
    def layer_bytes(self):
        return 4 * self.x_elems + self.wbytes() + 4 * self.L.M * self.L.N + 8 * self.L.N

    def stage1_bytes(self):
        return 4 * self.x_elems + self.ws_bytes

    def stage2_bytes(self):
        return self.ws_bytes + self.wbytes() + 4 * self.L.M * self.L.N + 8 * self.L.N


ConvLayerOnGpu = LayerOnGpu


class GraphOf:
    """n calls of fn captured once into a CUDA graph (the library only enqueues kernels, so the
    capture sees every launch); replay() then costs no per-launch host time."""

    def __init__(self, torch, fn, n):
        self.torch, self.n = torch, n
        self.g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()                                   # first call outside the capture (one-time set-up)
            torch.cuda.synchronize()
            with torch.cuda.graph(self.g, stream=side):
                for _ in range(n):
                    fn()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()

    def timed_replay(self):
        """Milliseconds of one replay, CUDA events on the launching stream."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        self.g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)


def per_launch_us(torch, fn, n, reps=3):
    g = GraphOf(torch, fn, n)
    g.timed_replay()
    return min(g.timed_replay() for _ in range(reps)) * 1e3 / n


def max_over_ranks(value: float, dist, device) -> float:
    """The slowest rank's time: what a weak-scaling run of independent replicas is charged."""
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_layer(I, rank: int, world: int):
    """Rank r's copy of the workload layer: same law, its own draws (tensor seeds offset by
    100 r), so that N ranks process N different batches with no exchange between them."""
    (L,) = I.config2()
    if world > 1:
        L = I.draw(L, 2, 100 * rank, "silu", 0.03, True)
    return L


def whole_job_value(flops_per_step: float, steps: int, world: int, slowest_ms: float) -> float:
    """TFLOP/s of the whole job: all ranks' work over the slowest rank's time."""
    return world * flops_per_step * steps / (slowest_ms * 1e-3) / 1e12


def run_own(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the quantized layer has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    from paper_2408_06995_b200 import build as fpq_build
    fpq_build.build()
    import paper_2408_06995_b200 as fpq
    from paper_2408_06995_b200 import inputs as I

    peaks = load_peaks()
    L = rank_layer(I, rank, world)      # every rank its own batch of the same law
    layer = ConvLayerOnGpu(L, fpq, torch, dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: W warm-up steps, then exactly K steps captured as one CUDA graph.  The graph is replayed
    # R >= 20 times (at least 50 ms of device time in all), every replay bracketed by its own pair of CUDA events;
    # ms_per_step is the median replay divided by K, the fastest replay is reported beside it.
    for _ in range(args.warmup):
        layer.step()
    torch.cuda.synchronize()
    steps_graph = GraphOf(torch, layer.step, args.steps)
    first_ms = steps_graph.timed_replay()              # untimed: graph upload, clocks, L2 turnover
    reps = max(20, int(50.0 / max(first_ms, 1e-3)) + 1)
    sampler = ClockSampler(physical_gpu_index(local))
    barrier()
    sampler.start()
    replay_ms = [steps_graph.timed_replay() for _ in range(reps)]
    barrier()
    clocks = sampler.stop()
    st = fpq.fpq_read_status()
    if st != fpq.OK:
        raise SystemExit(f"device status after the timed region: {fpq.status_string(st)}")
    total_ms = statistics.median(replay_ms)
    min_ms = min(replay_ms)
    if world > 1:
        total_ms = max_over_ranks(total_ms, dist, dev)
        min_ms = max_over_ranks(min_ms, dist, dev)
    flops_step = L.flops
    value = whole_job_value(flops_step, args.steps, world, total_ms)
    t_layer = total_ms * 1e-3 / args.steps

    # ---- the same graph replayed back to back for at least two seconds: the clocks settle under load, so the
    # figure is given as time x median SM clock as well
    sustained = None
    if rank == 0:
        n_sus = max(1, int(2000.0 / max(total_ms, 1e-3)))
        s2 = ClockSampler(physical_gpu_index(local))
        s2.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_sus):
            steps_graph.g.replay()
        e1.record()
        torch.cuda.synchronize()
        c2 = s2.stop()
        us = e0.elapsed_time(e1) * 1e3 / (n_sus * args.steps)
        sustained = {"seconds": e0.elapsed_time(e1) * 1e-3, "us_per_step": us, "sm_mhz_median": c2["sm_mhz"],
                     "reasons": c2["reasons"], "us_x_ghz": us * (c2["sm_mhz"] or 0) * 1e-3,
                     "tflops": flops_step / us / 1e6}

    # ---- L2-warm: the same step on ONE buffer set (input 33.5 MB + output 33.5 MB stay in the 126 MB L2)
    warm = None
    if rank == 0:
        lw = ConvLayerOnGpu(L, fpq, torch, dev, nsets=1)
        for _ in range(3):
            lw.step()
        warm = per_launch_us(torch, lw.step, 20)
        del lw
        torch.cuda.empty_cache()

    # ---- which kernels the step runs (the library's own choice), and each of them alone over the same buffer sets
    route = fpq.fpq_conv2d_route(L.B, L.C, L.H, L.W, L.N, L.R, L.S, L.pad, L.stride, fpq.E4M3, layer.fw)
    n_k = 10 * layer.nsets
    t_q = per_launch_us(torch, layer.stage1, n_k) * 1e-6
    t_c = per_launch_us(torch, layer.stage2, n_k) * 1e-6
    kernels_us = {"activation_quantize (two-kernel route)": t_q * 1e6, "contraction (two-kernel route)": t_c * 1e6}
    if route == fpq.ROUTE_TWO_KERNELS:
        launches_per_step = 2
        path = ("two kernels per step: activation quantize to framed channels-last codes, then the persistent "
                "TMA/tcgen05 implicit GEMM with fused dequantize + bias")
        if t_c >= t_q:
            dom, t_dom, b_dom = "fpq_gemm_kernel (contraction + epilogue)", t_c, layer.stage2_bytes()
        else:
            dom, t_dom, b_dom = "quantize_nchw_to_nhwc_e4m3_kernel (activation quantize)", t_q, layer.stage1_bytes()
        how = "each kernel replayed alone from a CUDA graph over the rotating buffer sets"
    else:
        launches_per_step = 1
        if route == fpq.ROUTE_PAIR_FUSED:
            dom = "fpq_pair_conv_kernel (activation quantize + contraction + epilogue on CTA pairs)"
            path = ("one kernel per step: FP32 activations staged by TMA, quantized to E4M3 in shared memory, "
                    "tcgen05 cta_group::2 MMAs with the weights resident in shared memory, fused dequantize + bias")
        else:
            dom = "fpq_gemm_kernel (fused form: activation quantize + contraction + epilogue)"
            path = "one kernel per step: activations quantized inside the contraction's operand staging"
        # the step IS the kernel: its duration is the timed region's, its bytes the layer's algorithmic bytes
        t_dom, b_dom = t_layer, layer.layer_bytes()
        kernels_us[dom] = t_dom * 1e6
        how = "the step is one kernel: CUDA events around the timed region's graph replays (median)"
    achieved = b_dom / t_dom / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"], "traffic": TRAFFIC.get(dom),
                "algorithmic_bytes_per_launch": b_dom, "us_per_launch": t_dom * 1e6,
                "kernels_us": kernels_us, "how": how}
    layer_roof = {"algorithmic_bytes": layer.layer_bytes(), "achieved_gbs": layer.layer_bytes() / t_layer / 1e9,
                  "frac_of_hbm_peak": layer.layer_bytes() / t_layer / 1e9 / peaks["hbm_gbs"],
                  "t_hbm_us": layer.layer_bytes() / (peaks["hbm_gbs"] * 1e9) * 1e6,
                  "t_tensor_us_nominal_fp8": flops_step / (NOMINAL_FP8_TFLOPS * 1e12) * 1e6}
    # every route of the library on the same step, for comparison
    routes_us = {}
    for name, pol in (("fused", fpq.PATH_FUSED), ("two_kernels", fpq.PATH_TWO_KERNELS)):
        fpq.fpq_set_path_policy(pol)
        for _ in range(2):
            layer.step()
        routes_us[name] = per_launch_us(torch, layer.step, n_k)
    fpq.fpq_set_path_policy(fpq.PATH_AUTO)

    # ---- the same K steps launched one by one from the host (launch-bound), for comparison
    evs = []
    for _ in range(min(args.steps, 200)):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        layer.step()
        e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    eager_us = statistics.median(a.elapsed_time(b) for a, b in evs) * 1e3

    # ---- weight encode (offline step), reported beside the metric
    enc_us = per_launch_us(torch, layer.encode, 20)

    # ---- end to end through the host-buffer C-ABI call
    xh = torch.from_numpy(L.x).pin_memory()
    yh = torch.empty(layer.ys_[0].shape, dtype=torch.float32).pin_memory()
    n_e2e = max(3, min(args.steps, 20))

    def e2e_call():
        layer._rot()
        fpq.fpq_conv2d_host(xh, layer.x, layer.prep, layer.ws, layer.xs, fpq.E4M3, layer.fw, layer.bias, layer.y, yh,
                            L.R, L.S, L.pad, L.stride, layer.workspace)

    for _ in range(3):
        e2e_call()
    barrier()
    t0 = time.perf_counter()
    for _ in range(n_e2e):
        e2e_call()
    t_e2e = time.perf_counter() - t0
    barrier()
    if world > 1:
        t_e2e = max_over_ranks(t_e2e, dist, dev)
    e2e = {"value": world * flops_step * n_e2e / t_e2e / 1e12, "unit": "TFLOP/s", "h2d_bytes_per_step": xh.numel() * 4,
           "d2h_bytes_per_step": yh.numel() * 4, "steps": n_e2e, "ms_per_step": 1e3 * t_e2e / n_e2e}

    # ---- W4A8 (the LDM-4-style pair), same protocol, reported beside the headline
    w4 = None
    if rank == 0 and not args.skip_w4:
        w4 = {}
        for L4 in I.config3():
            l4 = ConvLayerOnGpu(L4, fpq, torch, dev)
            for _ in range(3):
                l4.step()
            t4 = per_launch_us(torch, l4.step, 5 * l4.nsets) * 1e-6
            w4[L4.name] = {"tflops": L4.flops / t4 / 1e12, "us": t4 * 1e6,
                           "pct_dense_fp8_nominal": 100 * L4.flops / t4 / 1e12 / NOMINAL_FP8_TFLOPS,
                           "pct_dense_fp4_nominal": 100 * L4.flops / t4 / 1e12 / NOMINAL_FP4_TFLOPS,
                           "layer_frac_of_hbm_peak": l4.layer_bytes() / t4 / 1e9 / peaks["hbm_gbs"]}
            del l4
            torch.cuda.empty_cache()

    # ---- the standalone quantizers (HBM-bound): 2^26 FP32 elements, larger than L2
    quant = None
    if rank == 0 and not args.skip_w4:
        nq = 1 << 26
        xq = torch.randn(nq, device=dev, dtype=torch.float32)
        cq = torch.empty(nq, device=dev, dtype=torch.uint8)
        quant = {}
        for name, fmt, by in (("act_e4m3_hw_convert", fpq.E4M3, 5.0), ("act_e5m2_hw_convert", fpq.E5M2, 5.0),
                              ("act_e2m1_hw_convert", fpq.E2M1, 4.5), ("act_e3m4_general", fpq.E3M4, 5.0),
                              ("act_e1m2_general", fpq.E1M2, 4.5)):
            tq = per_launch_us(torch, lambda: fpq.fpq_quantize_act(xq, 0.01, fmt, cq), 10) * 1e-6
            quant[name] = {"elements": nq, "us": tq * 1e6, "gbs": by * nq / tq / 1e9,
                           "frac_of_hbm_peak": by * nq / tq / 1e9 / peaks["hbm_gbs"], "bytes_per_element": by}
        # the weight encoder (Sec. V-B: nearest, or signed floor + learned decision) on an 8192 x 8192 matrix
        wq = xq.view(8192, 8192)
        wsq = torch.full((8192,), 0.01, device=dev)
        rbq = torch.randint(0, 256, (8192, 1024), device=dev, dtype=torch.uint8)
        for name, fmt, rb, by in (("weight_e4m3_nearest", fpq.E4M3, None, 5.0), ("weight_e2m1_nearest", fpq.E2M1, None, 4.5),
                                  ("weight_e2m1_learned", fpq.E2M1, rbq, 4.625), ("weight_e3m4_learned", fpq.E3M4, rbq, 5.125)):
            out = fpq.fpq_quantize_weight(wq, wsq, fmt, rb)
            tq = per_launch_us(torch, lambda: fpq.fpq_quantize_weight(wq, wsq, fmt, rb, out), 10) * 1e-6
            quant[name] = {"elements": nq, "us": tq * 1e6, "gbs": by * nq / tq / 1e9,
                           "frac_of_hbm_peak": by * nq / tq / 1e9 / peaks["hbm_gbs"], "bytes_per_element": by}
        del wq, wsq, rbq, out
        del xq, cq
        torch.cuda.empty_cache()

    # ---- side measurements of the rows built around the layer (details: --suite round_learn / formats)
    side = None
    if rank == 0 and not args.skip_w4:
        side = {}
        M, N, K = 4096, 960, 320
        w = torch.randn((N, K), device=dev) * 0.02
        a = torch.randn((M, K), device=dev)
        alpha = torch.randn((N, K), device=dev) * 2.0
        sc = (w.abs().amax(dim=1) / 6.0).contiguous()
        grad, loss = torch.empty_like(alpha), torch.empty(2, dtype=torch.float64, device=dev)
        wk = torch.empty(fpq.fpq_round_learn_workspace_size(M, N, K), dtype=torch.uint8, device=dev)
        t = per_launch_us(torch, lambda: fpq.fpq_round_learn_step(w, sc, fpq.E2M1, alpha, a, 0.01, 1.0, grad, loss, wk),
                          10) * 1e-6
        fp32_peak = torch.cuda.get_device_properties(dev).multi_processor_count * 128 * 2 * \
            (clocks.get("sm_mhz") or 1965.0) * 1e6
        tf32_peak = peaks["bf16_tflops"] * (NOMINAL_TF32_TFLOPS / NOMINAL_BF16_TFLOPS)
        side["round_learn_step_qkv_320_960_m4096"] = {
            "us": t * 1e6, "tflops_fp32_equivalent": 4.0 * M * N * K / t / 1e12,
            "x_fp32_fma_peak": 4.0 * M * N * K / t / fp32_peak,
            "frac_of_tf32_peak_3_products": 3 * 4.0 * M * N * K / t / 1e12 / tf32_peak,
            "how": "both contractions on the tensor cores, three TF32 products per FP32 product"}
        M = 8192
        x = torch.randn((M, K), device=dev)
        y = torch.empty((M, N), device=dev)
        for fname, f in (("e4m3", fpq.E4M3), ("e1m2_reencoded", fpq.E1M2), ("e3m4_two_terms", fpq.E3M4),
                         ("e5m2_bias16_two_terms", fpq.Format(5, 2, 16, fpq.SAT_PAPER)),
                         ("e6m1_fp32_grid_values_tf32", fpq.Format(6, 1, 31, fpq.SAT_PAPER))):
            ws = (w.abs().amax(dim=1) / fpq.fpq_format_max(f)).contiguous()
            prep = fpq.fpq_prepare_weight(fpq.fpq_quantize_weight(w, ws, f, None), f, fpq.LINEAR, N, K)
            wk = torch.empty(max(256, fpq.fpq_linear_workspace_size(M, N, K, fpq.E4M3, f)), dtype=torch.uint8, device=dev)
            t = per_launch_us(torch, lambda: fpq.fpq_linear(x, prep, ws, 0.01, fpq.E4M3, f, None, N, y, wk), 10) * 1e-6
            side["linear_qkv_320_960_m8192_weights_" + fname] = {"us": t * 1e6, "tflops": 2.0 * M * N * K / t / 1e12}
        del w, a, alpha, x, y, wk
        torch.cuda.empty_cache()
        # the other workloads of the metric: the transformer-block linears and the whole U-Net step
        side["config4_transformer_linears_m8192"] = config4_measure(torch, fpq, I, dev, peaks)
        side["sd_v1_unet_step_trace"] = trace_measure(torch, fpq, I, dev, peaks, 5)

    # ---- CPU baseline: the oracle, as it stands, on the host cores (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not args.skip_cpu:
        dt_sum, fl_sum, passes, cores = 0.0, 0.0, 0, 0
        while dt_sum < 10.0 and passes < 32:          # about ten seconds of CPU work
            dt, fl, cores = oracle_sample_run(64)
            dt_sum, fl_sum, passes = dt_sum + dt, fl_sum + fl, passes + 1
        cpu = {"value": fl_sum / dt_sum / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
               "sample": f"the whole workload layer (64 images), {passes} passes", "seconds": dt_sum}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "e4m3 x e4m3 -> f32", "data": "synthetic",
            "config": {"workload": WORKLOAD,
                       "l2": f"inputs larger than L2: steps rotate over {layer.nsets} resident (x, scratch, y) sets, "
                             f"{layer.nsets * layer.set_bytes >> 20} MiB",
                       "launch": f"the K timed steps are one CUDA graph; {reps} replays, each timed by its own pair of "
                                 "CUDA events; ms_per_step = median replay / K",
                       "path": path},
            "pct_dense_fp8_peak_nominal": 100 * value / world / NOMINAL_FP8_TFLOPS,
            "pct_dense_fp8_peak_2x_measured_bf16": 100 * value / world / (2 * peaks["bf16_tflops"]),
            "roofline": roofline, "layer_roofline": layer_roof, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
            "min_ms_per_step": min_ms / args.steps, "replays": reps, "sustained": sustained, "l2_warm_us_per_step": warm,
            "routes_us": routes_us, "weight_encode_us": enc_us, "w4a8": w4, "standalone_quantizer": quant, "eager_step_us": eager_us,
            "side_measurements": side,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def trace_measure(torch, fpq, I, dev, peaks, reps):
    """One denoising step of the SD-v1-style U-Net as a layer trace: all 234 conv / linear
    layers (W4A8 with rounding decisions), each with its own buffers, launched back to back on one
    stream and replayed as one CUDA graph.  The buffers of one pass total several GB, so every
    layer finds its input in HBM."""
    trace = I.sd_v1_unet_layers()
    layers = [LayerOnGpu(L, fpq, torch, dev, nsets=1) for L in trace]
    torch.cuda.synchronize()

    def one_pass():
        for lay in layers:
            lay.step()

    for _ in range(2):
        one_pass()
    torch.cuda.synchronize()
    g = GraphOf(torch, one_pass, 1)
    g.timed_replay()
    ms = [g.timed_replay() for _ in range(reps)]
    st = fpq.fpq_read_status()
    if st != fpq.OK:
        raise SystemExit(f"device status: {fpq.status_string(st)}")
    flops = sum(L.flops for L in trace)
    bytes_ = sum(lay.layer_bytes() for lay in layers)
    bound_us = sum(max(lay.layer_bytes() / (peaks["hbm_gbs"] * 1e9), lay.L.flops / (NOMINAL_FP8_TFLOPS * 1e12)) * 1e6
                   for lay in layers)
    t = statistics.median(ms) * 1e-3
    out = {"suite": "sd_trace", "layers": len(layers), "gflop": flops / 1e9, "algorithmic_mb": bytes_ / 1e6,
           "ms_per_step": t * 1e3, "min_ms": min(ms), "aggregate_tflops": flops / t / 1e12,
           "pct_dense_fp8_peak_nominal": 100 * flops / t / 1e12 / NOMINAL_FP8_TFLOPS,
           "pct_dense_fp4_peak_nominal": 100 * flops / t / 1e12 / NOMINAL_FP4_TFLOPS,
           "sum_of_per_layer_bounds_us": bound_us, "frac_of_bound": bound_us * 1e-6 / t,
           "device_buffers_gb": sum(l.set_bytes for l in layers) / 1e9, "launch": "one CUDA graph replay"}
    del layers, g
    torch.cuda.empty_cache()
    return out


def config4_measure(torch, fpq, I, dev, peaks):
    """The eight SD-v1-style transformer-block linears (M = 8192; W8A8 and W4A8), each timed as a CUDA graph of
    calls that rotate over buffer sets larger than the L2: the sum against the sum of the per-layer bounds."""
    rows, tot, bound = {}, 0.0, 0.0
    for L in I.config4():
        lay = LayerOnGpu(L, fpq, torch, dev)
        for _ in range(2):
            lay.step()
        us = per_launch_us(torch, lay.step, max(4, min(40, 3 * lay.nsets)), reps=2)
        b = max(lay.layer_bytes() / (peaks["hbm_gbs"] * 1e9), L.flops / (NOMINAL_FP8_TFLOPS * 1e12)) * 1e6
        rows[L.name] = {"us": us, "bound_us": b}
        tot, bound = tot + us, bound + b
        del lay
        torch.cuda.empty_cache()
    return {"sum_us": tot, "sum_of_bounds_us": bound, "frac_of_bound": bound / tot, "layers": rows}


def run_trace(args):
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    from paper_2408_06995_b200 import build as fpq_build
    fpq_build.build()
    import paper_2408_06995_b200 as fpq
    from paper_2408_06995_b200 import inputs as I
    print(json.dumps(trace_measure(torch, fpq, I, dev, load_peaks(), max(3, min(args.steps, 20)))), flush=True)


def run_suite(args):
    """Per-shape table (not the headline line): every distinct layer shape of the chosen
    workload, each timed as a CUDA graph of rotating calls on both routes of the library."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    from paper_2408_06995_b200 import build as fpq_build
    fpq_build.build()
    import paper_2408_06995_b200 as fpq
    from paper_2408_06995_b200 import inputs as I
    peaks = load_peaks()
    if args.suite == "cifar":
        layers = I.config2()
    elif args.suite == "ldm":
        layers = I.config3()
    elif args.suite == "transformer":
        layers = I.config4()
    elif args.suite == "sd":
        layers = I.distinct_shapes(I.sd_v1_unet_layers())
    else:
        raise SystemExit("unknown suite")
    rows = []
    tot = {"auto": 0.0, "fused": 0.0, "two_kernels": 0.0, "two_kernels_narrow": 0.0, "best": 0.0, "flops": 0.0, "bytes": 0.0, "bound": 0.0}
    if args.only:
        layers = [L for L in layers if args.only in L.name]
        if not layers:
            raise SystemExit(f"no layer of suite {args.suite} has {args.only!r} in its name")
    for L in layers:
        lay = LayerOnGpu(L, fpq, torch, dev, l2_bytes=(128 << 20) if args.suite != "sd" else (48 << 20))
        n = max(4, min(40, 3 * lay.nsets))
        res = {}
        for name, pol in (("fused", fpq.PATH_FUSED), ("two_kernels", fpq.PATH_TWO_KERNELS),
                          ("two_kernels_narrow", fpq.PATH_TWO_KERNELS_NARROW), ("auto", fpq.PATH_AUTO)):
            fpq.fpq_set_path_policy(pol)
            for _ in range(2):
                lay.step()
            res[name] = per_launch_us(torch, lay.step, n, reps=2)
        fpq.fpq_set_path_policy(fpq.PATH_AUTO)
        st = fpq.fpq_read_status()
        if st != fpq.OK:
            raise SystemExit(f"{L.name}: device status {fpq.status_string(st)}")
        t_hbm = lay.layer_bytes() / (peaks["hbm_gbs"] * 1e9) * 1e6
        t_tc = L.flops / (NOMINAL_FP8_TFLOPS * 1e12) * 1e6
        best = min(res["fused"], res["two_kernels"], res["two_kernels_narrow"])
        rows.append({"name": L.name, "kind": L.kind, "M": L.M, "N": L.N, "K": L.K, "count": L.count, "wfmt": L.wfmt,
                     "us": res, "tflops_auto": L.flops / res["auto"] / 1e6, "t_hbm_us": t_hbm, "t_tensor_us": t_tc,
                     "frac_of_bound_auto": max(t_hbm, t_tc) / res["auto"]})
        for k in ("auto", "fused", "two_kernels", "two_kernels_narrow"):
            tot[k] += res[k] * L.count
        tot["best"] += best * L.count
        tot["flops"] += L.flops * L.count
        tot["bytes"] += lay.layer_bytes() * L.count
        tot["bound"] += max(t_hbm, t_tc) * L.count
        del lay
        torch.cuda.empty_cache()
    summary = {"suite": args.suite, "layers": sum(r["count"] for r in rows), "distinct_shapes": len(rows),
               "sum_us": {k: tot[k] for k in ("auto", "fused", "two_kernels", "two_kernels_narrow", "best")},
               "aggregate_tflops_auto": tot["flops"] / tot["auto"] / 1e6, "sum_bound_us": tot["bound"],
               "frac_of_bound_auto": tot["bound"] / tot["auto"], "gflop": tot["flops"] / 1e9, "rows": rows}
    print(json.dumps(summary), flush=True)


def run_search(args):
    """The encoding / bias search (Algorithm 1) on one tensor of 2^24 FP32 values: all FP8
    (4 x 111) and all FP4 (2 x 111) candidates.  ALU-bound: the roofline is instruction issue,
    9 lane instructions per element and candidate against 128 lanes per SM and clock."""
    import numpy as np
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    from paper_2408_06995_b200 import build as fpq_build
    fpq_build.build()
    import paper_2408_06995_b200 as fpq
    import oracle as O
    n = 1 << 24
    x = torch.randn(n, device=dev, dtype=torch.float32)
    maxabs = float(x.abs().max())
    clips = fpq.fpq_search_clip_candidates(maxabs, 111).to(dev)
    props = torch.cuda.get_device_properties(0)
    sampler = ClockSampler(physical_gpu_index(0))
    sampler.start()
    out = {"suite": "search", "elements": n, "rows": []}
    for name, encs_cpu in (("fp8_4x111", O.FP8_ENCODINGS), ("fp4_2x111", O.FP4_ENCODINGS)):
        encs = [fpq.Format(f.e, f.m, f.B, fpq.SAT_PAPER) for f in encs_cpu]
        ncand = len(encs) * 111
        mse = torch.empty((len(encs), 111), dtype=torch.float64, device=dev)
        best = torch.empty(2, dtype=torch.int32, device=dev)
        wk = torch.empty(fpq.fpq_search_workspace_size(len(encs), 111), dtype=torch.uint8, device=dev)
        t = per_launch_us(torch, lambda: fpq.fpq_search_format(x, encs, clips, mse, best, wk), 5) * 1e-6
        b = best.cpu().numpy()
        row = {"name": name, "candidates": ncand, "us": t * 1e6, "element_candidates_per_s": n * ncand / t,
               "lane_instructions_per_s": 9.0 * n * ncand / t, "hbm_gbs": 4.0 * n / t / 1e9,
               "selected": {"encoding": f"E{encs_cpu[b[0]].e}M{encs_cpu[b[0]].m}", "clip_index": int(b[1])}}
        out["rows"].append(row)
    clocks = sampler.stop()
    peak = props.multi_processor_count * 128 * (clocks["sm_mhz"] or 1965.0) * 1e6
    for row in out["rows"]:
        row["roofline"] = {"bound": "alu", "achieved": row["lane_instructions_per_s"] / 1e12, "peak": peak / 1e12,
                           "unit": "T lane-instructions/s", "frac": row["lane_instructions_per_s"] / peak,
                           "peak_source": "SM count x 128 lanes x sampled SM clock"}
    out["clocks"] = clocks
    if not args.skip_cpu:
        xs = x[: 1 << 16].cpu().numpy()
        t0 = time.perf_counter()
        O.search_mse(xs, O.FP8_ENCODINGS, clips.cpu().numpy())
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": xs.size * 444 / dt, "unit": "element-candidates/s", "cores": os.cpu_count(),
                               "kind": "oracle", "sample": "the first 2^16 elements, 4 x 111 candidates"}
    print(json.dumps(out), flush=True)


def run_round_learn(args):
    """One rounding-learning step (Sec. V-B objective + gradient + descent update) on the linear layers of
    the SD-v1-style transformer blocks, FP4 E2M1 weights, calibration rows = the tokens of one latent at
    that level.  Two FP32 contractions of 2 M N K flop each on the CUDA cores: the roofline is the FP32
    multiply-add rate, SMs x 128 lanes x 2 flop x sampled SM clock."""
    import numpy as np
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    from paper_2408_06995_b200 import build as fpq_build
    fpq_build.build()
    import paper_2408_06995_b200 as fpq
    import oracle as O
    shapes = [("qkv_320_960", 4096, 960, 320), ("attn_out_320_320", 4096, 320, 320),
              ("geglu_320_2560", 4096, 2560, 320), ("ffn_out_1280_320", 4096, 320, 1280),
              ("geglu_640_5120", 1024, 5120, 640), ("ffn_out_5120_1280", 256, 1280, 5120)]
    if args.only:
        shapes = [sh for sh in shapes if args.only in sh[0]]
        if not shapes:
            raise SystemExit(f"no shape of suite round_learn has {args.only!r} in its name")
    props = torch.cuda.get_device_properties(0)
    sampler = ClockSampler(physical_gpu_index(0))
    sampler.start()
    out = {"suite": "round_learn", "dtype": "f32", "rows": []}
    for name, M, N, K in shapes:
        w = torch.randn((N, K), device=dev) * 0.02
        scale = (w.abs().amax(dim=1) / 6.0).contiguous()
        a = torch.randn((M, K), device=dev)
        alpha = torch.randn((N, K), device=dev) * 2.0
        grad = torch.empty_like(alpha)
        loss = torch.empty(2, dtype=torch.float64, device=dev)
        wk = torch.empty(fpq.fpq_round_learn_workspace_size(M, N, K), dtype=torch.uint8, device=dev)
        fn = lambda: fpq.fpq_round_learn_step(w, scale, fpq.E2M1, alpha, a, 0.01, 1.0, grad, loss, wk)
        t = per_launch_us(torch, fn, 10) * 1e-6
        flop = 4.0 * M * N * K
        out["rows"].append({"name": name, "M": M, "N": N, "K": K, "us": t * 1e6, "tflops": flop / t / 1e12,
                            "steps_per_s": 1.0 / t})
    clocks = sampler.stop()
    # Rows of a multiple of 4 floats run on the tensor cores, every FP32 product as three TF32 products: the
    # tensor work is 3 x 4 M N K flop against the TF32 peak (the measured bf16 peak x the nominal 1.1 / 2.25).
    # `tflops` stays the FP32-equivalent figure; the CUDA cores' own FP32 multiply-add peak is given for scale.
    peaks = load_peaks()
    tf32_peak = peaks["bf16_tflops"] * (NOMINAL_TF32_TFLOPS / NOMINAL_BF16_TFLOPS)
    fma_peak = props.multi_processor_count * 128 * 2 * (clocks["sm_mhz"] or 1965.0) * 1e6 / 1e12
    for row in out["rows"]:
        on_tensor = row["K"] % 4 == 0
        if on_tensor:
            row["roofline"] = {"bound": "tensor", "achieved": 3.0 * row["tflops"], "peak": tf32_peak, "unit": "TFLOP/s",
                               "frac": 3.0 * row["tflops"] / tf32_peak,
                               "peak_source": peaks["source"] + " bf16 x 1.1/2.25 (TF32)", "traffic": None,
                               "fp32_fma_peak_tflops": fma_peak}
        else:
            row["roofline"] = {"bound": "alu", "achieved": row["tflops"], "peak": fma_peak, "unit": "TFLOP/s",
                               "frac": row["tflops"] / fma_peak,
                               "peak_source": "SM count x 128 FP32 lanes x 2 flop x sampled SM clock"}
    out["clocks"] = clocks
    if not args.skip_cpu:
        name, M, N, K = min(shapes, key=lambda sh: sh[1] * sh[2] * sh[3])
        rng = np.random.default_rng(0)
        w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
        sc = (np.abs(w).max(axis=1) / 6.0).astype(np.float32)
        al = (rng.standard_normal((N, K)) * 2).astype(np.float32)
        a = rng.standard_normal((M, K)).astype(np.float32)
        t0 = time.perf_counter()
        O.round_learn_step(w, sc, O.E2M1, al, a, 0.01)
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": 1.0 / dt, "unit": "steps/s", "cores": os.cpu_count(), "kind": "oracle",
                               "sample": f"one step of {name} (M={M})"}
    print(json.dumps(out), flush=True)


def run_formats(args):
    """The weight encodings the search can select, as the same linear layers (SD-v1-style transformer block,
    M = 8192): read by the tensor cores as they are (E4M3, E2M1), re-encoded exactly into E4M3 when the
    weights are prepared (E1M2), prepared as the sum of two E4M3 (E3M4, E2M5, E4M3 bias 8) or E5M2 (E5M2 bias 16)
    terms and contracted over twice the reduction length, or run on the CUDA cores with FP32 multiply-adds
    (E6M1, whose 64 binades no two tensor-core terms span: a stand-in for whatever the tensor cores cannot hold)."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    from paper_2408_06995_b200 import build as fpq_build
    fpq_build.build()
    import paper_2408_06995_b200 as fpq
    shapes = [("qkv_320_960", 8192, 960, 320), ("ffn_out_1280_320", 8192, 320, 1280)]
    formats = [("e4m3", fpq.E4M3, "tensor cores"), ("e2m1", fpq.E2M1, "tensor cores"),
               ("e5m2_ocp", fpq.E5M2, "tensor cores"),
               ("e1m2", fpq.E1M2, "tensor cores, weights re-encoded into E4M3"),
               ("e3m4", fpq.E3M4, "tensor cores, weights prepared as two E4M3 terms"),
               ("e2m5", fpq.E2M5, "tensor cores, weights prepared as two E4M3 terms"),
               ("e4m3_bias8", fpq.Format(4, 3, 8, fpq.SAT_PAPER), "tensor cores, weights prepared as two E4M3 terms"),
               ("e5m2_bias16", fpq.Format(5, 2, 16, fpq.SAT_PAPER), "tensor cores, weights prepared as two E5M2 terms"),
               ("e6m1", fpq.Format(6, 1, 31, fpq.SAT_PAPER), "FP32 grid values, one TF32 tensor-core product per term")]
    if args.only:
        formats = [f for f in formats if args.only in f[0]]
        if not formats:
            raise SystemExit(f"no weight format of suite formats has {args.only!r} in its name")
    props = torch.cuda.get_device_properties(0)
    sampler = ClockSampler(physical_gpu_index(0))
    sampler.start()
    rows = []
    for name, M, N, K in shapes:
        x = torch.randn((M, K), device=dev)
        xs = float(x.abs().max()) / 448.0
        w = torch.randn((N, K), device=dev) * 0.02
        bias = torch.randn(N, device=dev) * 0.01
        y = torch.empty((M, N), device=dev)
        for fname, f, route in formats:
            ws = (w.abs().amax(dim=1) / fpq.fpq_format_max(f)).contiguous()
            codes = fpq.fpq_quantize_weight(w, ws, f, None)
            prep = fpq.fpq_prepare_weight(codes, f, fpq.LINEAR, N, K)
            wk = torch.empty(max(256, fpq.fpq_linear_workspace_size(M, N, K, fpq.E4M3, f)), dtype=torch.uint8, device=dev)
            t = per_launch_us(torch, lambda: fpq.fpq_linear(x, prep, ws, xs, fpq.E4M3, f, bias, N, y, wk), 10) * 1e-6
            rows.append({"name": name, "weights": fname, "route": route, "M": M, "N": N, "K": K, "us": t * 1e6,
                         "tflops": 2.0 * M * N * K / t / 1e12, "weight_bytes": prep.numel()})
        if args.only:
            continue
        # the activation encodings of the search (Sec. V-A) against E4M3 / E2M1 weights
        for aname, fa, fwt, route in (("e4m3", fpq.E4M3, fpq.E2M1, "tensor cores"), ("e5m2_ocp", fpq.E5M2, fpq.E2M1, "tensor cores"),
                                      ("e3m4", fpq.E3M4, fpq.E4M3, "tensor cores, activations as two E4M3 terms"),
                                      ("e2m5", fpq.E2M5, fpq.E2M1, "tensor cores, activations as two E4M3 terms"),
                                      ("e4m3_all_finite", fpq.Format(4, 3, 7, fpq.SAT_PAPER), fpq.E2M1,
                                       "tensor cores, activations as two E4M3 terms"),
                                      ("e3m4", fpq.E3M4, fpq.E3M4, "FP32 grid values, one TF32 tensor-core product per term")):
            ws = (w.abs().amax(dim=1) / fpq.fpq_format_max(fwt)).contiguous()
            prep = fpq.fpq_prepare_weight(fpq.fpq_quantize_weight(w, ws, fwt, None), fwt, fpq.LINEAR, N, K)
            xsa = float(x.abs().max()) / fpq.fpq_format_max(fa)
            wk = torch.empty(max(256, fpq.fpq_linear_workspace_size(M, N, K, fa, fwt)), dtype=torch.uint8, device=dev)
            t = per_launch_us(torch, lambda: fpq.fpq_linear(x, prep, ws, xsa, fa, fwt, bias, N, y, wk), 10) * 1e-6
            rows.append({"name": name, "activations": aname, "weights": "e4m3" if fwt is fpq.E4M3 else ("e2m1" if fwt is fpq.E2M1 else "e3m4"),
                         "route": route, "M": M, "N": N, "K": K, "us": t * 1e6, "tflops": 2.0 * M * N * K / t / 1e12})
    clocks = sampler.stop()
    fp32_peak = props.multi_processor_count * 128 * 2 * (clocks["sm_mhz"] or 1965.0) * 1e6
    for r in rows:
        if r["route"].startswith("CUDA"):
            r["roofline"] = {"bound": "alu", "achieved": r["tflops"], "peak": fp32_peak / 1e12, "unit": "TFLOP/s",
                             "frac": r["tflops"] * 1e12 / fp32_peak,
                             "peak_source": "SM count x 128 FP32 lanes x 2 flop x sampled SM clock"}
    print(json.dumps({"suite": "formats", "rows": rows, "clocks": clocks}), flush=True)


def run_split(args):
    """The decoder convolutions of the SD-v1-style U-Net whose input is a concatenation (previous
    layer's output + skip connection), W4A8, batch 2: the two-scale call against the ordinary call
    on the already concatenated tensor."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    from paper_2408_06995_b200 import build as fpq_build
    fpq_build.build()
    import paper_2408_06995_b200 as fpq
    peaks = load_peaks()
    shapes = [("up3.res.conv1", 1280, 1280, 8, 1280, 3), ("up2.res0.conv1", 1280, 1280, 16, 1280, 3),
              ("up2.res2.conv1", 1280, 640, 16, 1280, 3), ("up1.res0.conv1", 1280, 640, 32, 640, 3),
              ("up1.res1.conv1", 640, 640, 32, 640, 3), ("up1.res2.conv1", 640, 320, 32, 640, 3),
              ("up0.res0.conv1", 640, 320, 64, 320, 3), ("up0.res1.conv1", 320, 320, 64, 320, 3),
              ("up0.res1.skip", 320, 320, 64, 320, 1)]
    B, fw = 2, fpq.E2M1
    rows = []
    for name, C1, C2, HW, Co, R in shapes:
        pad = R // 2
        nsets = max(2, int(3 * (128 << 20) / (B * (C1 + C2 + Co) * HW * HW * 4)) + 1)
        nsets = min(nsets, 64)
        x1 = [torch.randn(B, C1, HW, HW, device=dev) for _ in range(nsets)]
        x2 = [torch.randn(B, C2, HW, HW, device=dev) * 3 for _ in range(nsets)]
        xc = [torch.cat([a, b], dim=1).contiguous() for a, b in zip(x1, x2)]
        ys = [torch.empty(B, Co, HW, HW, device=dev) for _ in range(nsets)]
        w = torch.randn(Co, (C1 + C2) * R * R, device=dev) * 0.02
        ws = (w.abs().amax(dim=1) / 6.0).contiguous()
        codes = fpq.fpq_quantize_weight(w, ws, fw, None)
        prep_s = fpq.fpq_prepare_weight_split(codes, fw, Co, C1, C2, R, R)
        prep_c = fpq.fpq_prepare_weight(codes, fw, fpq.CONV2D, Co, C1 + C2, R, R)
        bias = torch.zeros(Co, device=dev)
        wk = torch.empty(fpq.fpq_conv2d_split_workspace_size(B, C1, C2, HW, HW, Co, R, R, pad, 1, fpq.E4M3, fw),
                         dtype=torch.uint8, device=dev)
        s1, s2, sc = float(x1[0].abs().max()) / 448, float(x2[0].abs().max()) / 448, float(xc[0].abs().max()) / 448
        k = [0]

        def split_call():
            i = k[0] = (k[0] + 1) % nsets
            fpq.fpq_conv2d_split(x1[i], s1, x2[i], s2, prep_s, ws, fpq.E4M3, fw, bias, ys[i], R, R, pad, 1, wk)

        def plain_call():
            i = k[0] = (k[0] + 1) % nsets
            fpq.fpq_conv2d(xc[i], prep_c, ws, sc, fpq.E4M3, fw, bias, Co, R, R, pad, 1, ys[i], wk)

        t_s = per_launch_us(torch, split_call, 4 * nsets)
        t_p = per_launch_us(torch, plain_call, 4 * nsets)
        flops = 2.0 * B * HW * HW * Co * (C1 + C2) * R * R
        by = 4.0 * B * (C1 + C2 + Co) * HW * HW + Co * (C1 + C2) * R * R / 2 + 8 * Co
        rows.append({"name": name, "C1": C1, "C2": C2, "HW": HW, "C_out": Co, "R": R, "us_split": t_s, "us_plain": t_p,
                     "tflops_split": flops / t_s / 1e6, "t_hbm_us": by / peaks["hbm_gbs"] / 1e3,
                     "t_tensor_us": flops / NOMINAL_FP8_TFLOPS / 1e6})
        del x1, x2, xc, ys
        torch.cuda.empty_cache()
    print(json.dumps({"suite": "sd_split", "batch": B, "rows": rows,
                      "sum_us": {"split": sum(r["us_split"] for r in rows), "plain": sum(r["us_plain"] for r in rows)}}),
          flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="own", choices=["own", "reference"])
    ap.add_argument("--skip-cpu", action="store_true", help="leave out the CPU-oracle baseline leg")
    ap.add_argument("--skip-w4", action="store_true", help="leave out the W4A8 side measurement")
    ap.add_argument("--suite", default=None, choices=["cifar", "ldm", "transformer", "sd", "sd_trace", "search", "sd_split", "round_learn", "formats"],
                    help="print a per-shape table of a whole workload instead of the headline line")
    ap.add_argument("--only", default=None, help="with --suite ldm|transformer|sd|round_learn: only the layers whose name contains this; "
                    "with --suite formats: only the weight formats whose name contains this")
    args = ap.parse_args()
    if args.suite == "sd_trace":
        run_trace(args)
    elif args.suite == "search":
        run_search(args)
    elif args.suite == "sd_split":
        run_split(args)
    elif args.suite == "round_learn":
        run_round_learn(args)
    elif args.suite == "formats":
        run_formats(args)
    elif args.suite:
        run_suite(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_own(args)


if __name__ == "__main__":
    main()
