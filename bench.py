#!/usr/bin/env python
"""Benchmark of the Bconv2D hot path on B200.

Workload ("config 2"): the ResNet-18-shaped 3x3 one-padded binarized convolutions
56x56x64->64, 28x28x128->128, 14x14x256->256, 7x7x512->512 at batch 64 per GPU, each once with
float output (per-channel multiply-add) and once with bit-packed output (per-channel thresholds),
on inputs bit-packed beforehand from seeded N(0,1) activations and uniform +-1 weights packed at
load time.  One step = those 8 LceBConv2d launches through the default dispatch (LCE_KERNEL_AUTO: the
tensor-core kernel at these sizes).  Metric: binary multiply-accumulates per second
(N*OH*OW*Cout*KH*KW*Cin per launch, summed) over all GPUs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl lce|reference] [--no-cpu-baseline]

Prints one JSON line.  With --impl reference the CPU oracle is timed instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import numpy as np  # noqa: E402

import lce_workloads as wl  # noqa: E402

CONFIG = 2
BATCH = 64
METRIC = "bconv2d_binary_macs_per_second"
UNIT = "binary-MAC/s"
WORKLOAD = ("config 2: 3x3 one-padded Bconv2D sweep 56x56x64, 28x28x128, 14x14x256, 7x7x512 at batch 64 per GPU, "
            "float and bit-packed output each (8 launches per step), pre-packed inputs, load-time packed weights")

# Derived compute ceiling of the integer pipes (logic + popcount), reported beside the measured one:
# 64 logic lanes/clk/SM, 16.75 logic instructions per nine 32-bit word operations, 32 binary MACs per word.
LOGIC_LANES_PER_CLK_PER_SM = 64
LOGIC_OPS_PER_9_WORDS = 16.75


def specs():
    return wl.config2_specs(BATCH)


def layer_inputs(spec, index):
    """Seeded host tensors of one launch: fp32 activations and +-1 weights plus per-channel arrays."""
    x = wl.activations(CONFIG, 10 * index, (spec.batch, spec.in_h, spec.in_w, spec.in_c))
    t = wl.conv_tensors(CONFIG, 10 * index + 1, spec)
    return x, t


def shard_index(layer: int, rank: int) -> int:
    """RNG index offset of one launch's tensors on one rank: every rank draws its own 64-image shard."""
    return layer + 100 * rank


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Slowest rank's time (the job is as slow as its slowest GPU); identity on one rank."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    tt = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_value(units_per_rank: float, world: int, ms: float) -> float:
    """Weak scaling: every rank processes units_per_rank in the (max-over-ranks) time."""
    return world * units_per_rank / (ms * 1e-3)


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.001)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_items(batch: int, rank: int = 0):
    """Seeded inputs of the 8 launches as the oracle takes them: +-1 activations and the layer parameters."""
    import oracle
    items = []
    for i, spec in enumerate(wl.config2_specs(batch)):
        x, t = layer_inputs(spec, shard_index(i, rank))
        items.append((spec, oracle.sign(x), t))
    return items


def oracle_pass(items):
    """One pass of the CPU oracle, as it stands, over the 8 launches; returns its outputs."""
    import oracle
    outs = []
    for spec, a, t in items:
        acc = oracle.bconv2d_acc(a, t.w_pm1, (1, 1), spec.padding)
        if spec.out_type == wl.OUT_FLOAT32:
            outs.append(oracle.transform_float(acc, t.multiplier, t.bias))
        else:
            outs.append(oracle.transform_bits(acc, t.thresholds))
    return outs


def time_oracle(items, passes: int = 1, min_seconds: float = 0.0):
    """Times the oracle on all 8 launches: `passes` passes, then more until `min_seconds` of CPU work
    are done (at most 16).  Returns (binary MACs per second, seconds per pass, passes, outputs of the first pass)."""
    import oracle
    oracle.bconv2d_acc(items[0][1][:1], items[0][2].w_pm1)  # load the library, warm the threads
    macs = sum(s.binary_macs for s, _, _ in items)
    t0 = time.perf_counter()
    done, first = 0, None
    while done < passes or (time.perf_counter() - t0 < min_seconds and done < 16):
        outs = oracle_pass(items)
        if first is None:
            first = outs
        done += 1
    dt = (time.perf_counter() - t0) / done
    return macs / dt, dt, done, first


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the same config at the same batch (every step
    = all 8 launches at batch 64 on the host cores)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    items = oracle_items(BATCH)
    for _ in range(min(args.warmup, 2)):
        oracle_pass(items)
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        oracle_pass(items)
        times.append(time.perf_counter() - t0)
    macs = sum(s.binary_macs for s, _, _ in items)
    ms = 1e3 * float(np.mean(times))
    value = macs / (ms * 1e-3)
    sample = f"each step = all 8 launches of config 2 at batch {BATCH} (the whole workload of one GPU), {args.steps} steps"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": min(args.warmup, 2), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": BATCH, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "images_per_second": 8 * BATCH / (ms * 1e-3),
    }
    print(json.dumps(line))


def load_probe():
    """liblce_probe.so: the measurement-only companion library (pipe micro-benchmarks)."""
    import ctypes

    from paper_2011_09398_b200 import build as lce_build
    lib = ctypes.CDLL(str(lce_build.PROBE_LIB))
    lib.lce_probe_pipe.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                   ctypes.c_void_p]
    lib.lce_probe_pipe.restype = ctypes.c_int

    lib.lce_probe_stage.argtypes = [ctypes.c_int32] * 7 + [ctypes.POINTER(ctypes.c_double)] * 2 + [ctypes.c_void_p]
    lib.lce_probe_stage.restype = ctypes.c_int

    def probe(mix: int, iterations: int = 2000):
        import torch
        a, b = ctypes.c_double(), ctypes.c_double()
        st = lib.lce_probe_pipe(mix, iterations, ctypes.byref(a), ctypes.byref(b), torch.cuda.current_stream().cuda_stream)
        if st != 0:
            raise RuntimeError(f"lce_probe_pipe: status {st}")
        return a.value, b.value

    def stage(mode: int, batch: int, h: int, w: int, words: int, rows: int, passes: int = 20):
        import torch
        a, b = ctypes.c_double(), ctypes.c_double()
        st = lib.lce_probe_stage(mode, batch, h, w, words, rows, passes, ctypes.byref(a), ctypes.byref(b),
                                 torch.cuda.current_stream().cuda_stream)
        if st != 0:
            raise RuntimeError(f"lce_probe_stage: status {st}")
        return a.value, b.value
    probe.stage = stage
    return probe


def staging_probe(probe, batch: int) -> dict:
    """The three ways of staging activation tiles (4-byte async copies into word planes, 16-byte async
    copies, one tensor-map bulk copy per tile), timed with nothing behind them on the 28x28x128 layer."""
    names = ("cp_async_4B_word_planes", "cp_async_16B", "tensor_map_bulk_copy")
    res = [probe.stage(mode, batch, 28, 28, 4, 7) for mode in range(3)]
    return {"workload": f"input of the 28x28x128 layer at batch {batch} (0.8 MB), tiles of 7 + 2 rows, 2 CTAs of 256 threads per SM",
            "whole_tensor_us": {n: r[0] for n, r in zip(names, res)},
            "first_tile_us": {n: r[1] for n, r in zip(names, res)}}


def measured_peaks() -> dict:
    try:
        return json.loads((ROOT / "MEASURED_PEAKS.json").read_text())
    except Exception:
        return {}


def profiled_traffic(kernel: str):
    """DRAM bytes per launch of the named kernel on this workload, from the ncu capture summarised under
    profiles/ (one value per layer; the mean is reported).  None if there is no such summary."""
    path = ROOT / "profiles" / f"{kernel}_config2_dram.json"
    try:
        rows = json.loads(path.read_text())["layers"]
        return float(np.mean([r["dram_bytes_read"] + r["dram_bytes_write"] for r in rows.values()]))
    except Exception:
        return None


def run_lce(args):
    import torch
    import torch.distributed as dist

    import paper_2011_09398_b200 as lce

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # ---- inputs: every rank draws its own batch shard (weak scaling: 64 images per GPU) ------
    layers = []
    h2d = d2h = 0
    for i, spec in enumerate(specs()):
        x, t = layer_inputs(spec, shard_index(i, rank))
        xd = torch.from_numpy(x).to(dev)
        a = lce.lce_bitpack(xd)                                   # pre-packed input (outside the timed region)
        wplain = lce.pack_weights(torch.from_numpy(t.w_pm1).to(dev))
        mk = lambda kernel, packed: lce.make_desc(spec.batch, spec.in_h, spec.in_w, spec.in_c, spec.out_c, (3, 3), (1, 1), spec.padding,
                                                   spec.out_type, lce.ACT_NONE, kernel, packed)
        desc = mk(lce.KERNEL_AUTO, 1)
        wpacked = lce.lce_bconv2d_pack_weights(desc, wplain)       # load-time weight packing
        mult = torch.from_numpy(t.multiplier).to(dev)
        bias = torch.from_numpy(t.bias).to(dev)
        thr = torch.from_numpy(t.thresholds).to(dev)
        if spec.out_type == wl.OUT_FLOAT32:
            out = torch.empty((spec.batch, spec.out_h, spec.out_w, spec.out_c), dtype=torch.float32, device=dev)
        else:
            out = torch.empty((spec.batch, spec.out_h, spec.out_w, (spec.out_c + 31) // 32), dtype=torch.int32, device=dev)
        # host side of the end-to-end leg: pinned buffers, plain weights
        desc_host = mk(lce.KERNEL_AUTO, 0)
        host = dict(
            a=a.cpu().pin_memory(), w=wplain.cpu().pin_memory(),
            mult=torch.from_numpy(t.multiplier).pin_memory() if spec.out_type == wl.OUT_FLOAT32 else None,
            bias=torch.from_numpy(t.bias).pin_memory() if spec.out_type == wl.OUT_FLOAT32 else None,
            thr=torch.from_numpy(t.thresholds).pin_memory() if spec.out_type == wl.OUT_BITPACKED else None,
            out=torch.empty(out.shape, dtype=out.dtype).pin_memory(),
            ws=torch.empty(lce.lce_bconv2d_host_workspace_bytes(desc_host), dtype=torch.uint8, device=dev),
            desc=desc_host)
        h2d += host["a"].numel() * 4 + host["w"].numel() * 4 + 4 * spec.out_c * (2 if spec.out_type == wl.OUT_FLOAT32 else 1)
        d2h += host["out"].numel() * 4
        layers.append(dict(spec=spec, desc=desc, desc_tiled=mk(lce.KERNEL_TILED, 1), kernel=lce.lce_bconv2d_plan(desc)["kernel"],
                           a=a, w=wpacked, mult=mult, bias=bias, thr=thr, out=out, host=host))
        del xd
    torch.cuda.synchronize()

    flush = torch.empty(256 * 1024 * 1024 // 4, dtype=torch.int32, device=dev)  # > 126 MB L2

    def launch(layer, which="desc"):
        s = layer["spec"]
        if s.out_type == wl.OUT_FLOAT32:
            lce.lce_bconv2d(layer[which], layer["a"], layer["w"], layer["mult"], layer["bias"], None, layer["out"])
        else:
            lce.lce_bconv2d(layer[which], layer["a"], layer["w"], None, None, layer["thr"], layer["out"])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.Stream(device=dev)

    def capture(fn):
        """fn() enqueued once for real, then captured into a CUDA graph (replays run without host gaps)."""
        fn()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            fn()
        return g

    def timed_steps(graph, steps, sample_clocks):
        """`steps` replays, the L2 flushed before each by a 256 MiB write, one CUDA-event pair per replay on
        the launching stream."""
        sampler = ClockSampler(local_rank) if sample_clocks else None
        if sampler:
            sampler.start()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        wall0 = time.perf_counter()
        for k in range(steps):
            flush.fill_(k)
            ev[k][0].record(stream)
            graph.replay()
            ev[k][1].record(stream)
        barrier()
        wall = time.perf_counter() - wall0
        clocks = sampler.stop() if sampler else None
        return [a.elapsed_time(b) for a, b in ev], clocks, wall

    with torch.cuda.stream(stream):
        # One step = the 8 launches replayed as one CUDA graph, through the default dispatch (AUTO).
        graph = capture(lambda: [launch(l) for l in layers])
        for _ in range(max(args.warmup, 3)):
            flush.fill_(1)
            graph.replay()
        barrier()
        # ---- timed region: exactly K steps -----------------------------------------------------------
        step_ms, clocks, wall = timed_steps(graph, args.steps, True)
        outputs_of_timed_launches = [l["out"].clone() for l in layers]

        # ---- the same step for about a second more, so that the clock record has hundreds of samples ----
        sustained = None
        if world == 1 and not args.profile:
            n_more = int(min(4000, max(50, 1.0 / max(1e-6, (np.mean(step_ms) + 0.12) * 1e-3))))
            more_ms, more_clocks, more_wall = timed_steps(graph, n_more, True)
            sustained = {"steps": n_more, "ms_per_step": float(np.mean(more_ms)), "wall_s": more_wall, "clocks": more_clocks,
                         "ms_per_step_x_median_sm_mhz": float(np.mean(more_ms)) * (more_clocks["sm_mhz"] or 0)}

        # ---- the benchmark spec's pipe: the integer XOR/POPC kernel forced, timed the same way ------------
        graph_int = capture(lambda: [launch(l, "desc_tiled") for l in layers])
        for _ in range(3):
            flush.fill_(1)
            graph_int.replay()
        int_ms, _, _ = timed_steps(graph_int, args.steps, False)

        # ---- per-launch durations: each layer alone as a graph of 10 launches, L2 warm ----------------
        def per_layer_us(which):
            res = []
            for l in layers:
                g = capture(lambda: [launch(l, which) for _ in range(10)])
                g.replay()
                stream.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(3):
                    g.replay()
                e1.record(stream)
                stream.synchronize()
                res.append(e0.elapsed_time(e1) * 1e3 / 30)
            return res
        us_auto, us_int = per_layer_us("desc"), per_layer_us("desc_tiled")
        for l, o in zip(layers, outputs_of_timed_launches):   # the timing loops above rewrote the buffers with equal values
            l["timed_out"] = o
    total_ms = max_over_ranks(float(np.sum(step_ms)), world, dev)
    ms_per_step = total_ms / args.steps
    macs_per_step = sum(l["spec"].binary_macs for l in layers)
    value = whole_job_value(macs_per_step, world, ms_per_step)
    images_per_s = world * len(layers) * BATCH / (ms_per_step * 1e-3)

    # ---- end-to-end leg: the host-buffer C-ABI entry point, copies inside the timed region ---------
    # Every step copies each layer's inputs in from pinned host memory, runs the kernel and copies the
    # result back, through lce_bconv2d_host_async on two streams (layers alternate, each with its own
    # workspace), so that one layer's copy back overlaps the next layer's copies in and kernel; the
    # step ends when both streams are synchronised, i.e. when all eight results are in host memory.
    host_streams = [torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)]

    def step_host():
        for j, layer in enumerate(layers):
            h = layer["host"]
            with torch.cuda.stream(host_streams[j % 2]):
                lce.lce_bconv2d_host_async(h["desc"], h["a"], h["w"], h["mult"], h["bias"], h["thr"], h["out"], h["ws"])
        for st in host_streams:
            st.synchronize()

    for _ in range(2):
        step_host()
    barrier()
    e2e_steps = max(3, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step_host()
    barrier()
    e2e_wall = time.perf_counter() - t0
    e2e_ms = 1e3 * e2e_wall / e2e_steps  # every step ends with a host synchronisation: wall clock is the honest one
    e2e_ms = max_over_ranks(e2e_ms, world, dev)
    e2e_value = whole_job_value(macs_per_step, world, e2e_ms)

    # ---- rooflines ------------------------------------------------------------------------------------
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    max_mhz = clocks["sm_max_mhz"] or 1965
    peaks = measured_peaks()
    n_launch = len(layers)
    avg_launch_ms = float(np.mean(step_ms)) / n_launch           # the step holds nothing but the 8 launches
    achieved = (macs_per_step / n_launch) / (avg_launch_ms * 1e-3)
    bit = [j for j, l in enumerate(layers) if l["spec"].out_type == wl.OUT_BITPACKED]
    flt = [j for j, l in enumerate(layers) if l["spec"].out_type == wl.OUT_FLOAT32]
    rate = lambda us, idx: sum(layers[j]["spec"].binary_macs for j in idx) / (sum(us[j] for j in idx) * 1e-6)
    hbm_bound_us = float(np.mean([l["spec"].algorithmic_bytes for l in layers])) / peak_hbm_bytes_per_s() * 1e6
    all_tensor = all(l["kernel"] == lce.KERNEL_TENSOR for l in layers)
    # tensor-core path: the contraction runs on e2m1 (fp4) operands; its peak is the measured bf16 burst
    # rate x the nominal fp4 : bf16 ratio (4), in MACs (2 FLOP each)
    bf16 = float(peaks.get("bf16_tflops", 1590.0))
    tensor_peak = bf16 * 1e12 * 4 / 2
    roofline = {
        "bound": "tensor", "kernel": "bconv_mx_kernel (tcgen05 kind::mxf4, all 8 launches)" if all_tensor else "mixed",
        "achieved": achieved / 1e12, "peak": tensor_peak / 1e12, "unit": "T binary-MAC/s (x2 = TFLOP/s)", "frac": achieved / tensor_peak,
        "peak_source": ("MEASURED_PEAKS.json bf16_tflops (burst) x 4 (nominal fp4 : bf16) / 2 FLOP per MAC, of measured" if peaks
                        else "fallback 1590 TFLOP/s bf16 x 4 / 2, of fallback"),
        "frac_of_int8_peak": achieved / (bf16 * 1e12),  # the same work on 8-bit operands would have this ceiling
        "avg_launch_us": avg_launch_ms * 1e3,
        "frac_bitpacked_launches": rate(us_auto, bit) / tensor_peak, "frac_float_launches": rate(us_auto, flt) / tensor_peak,
        "traffic": profiled_traffic("bconv_mx_kernel"),
        "hbm_bound_us": hbm_bound_us,
        # the float launches alone (their outputs are what moves): per launch, and as a fraction of their measured time
        "hbm_bound_us_float_launches": [layers[j]["spec"].algorithmic_bytes / peak_hbm_bytes_per_s() * 1e6 for j in flt],
        "hbm_frac_float_launches": sum(layers[j]["spec"].algorithmic_bytes for j in flt) / peak_hbm_bytes_per_s() * 1e6 / sum(us_auto[j] for j in flt),
    }
    # integer path (the pipe the benchmark spec names): ceiling = the best measured register-resident
    # instruction mix (probe run in this process), the derived figure beside it
    probe = load_probe()
    probe_ops, _ = probe(3, 2000)
    probe_naive, _ = probe(0, 2000)
    int_launch_ms = float(np.mean(int_ms)) / n_launch
    int_achieved = (macs_per_step / n_launch) / (int_launch_ms * 1e-3)
    derived = sms * max_mhz * 1e6 * LOGIC_LANES_PER_CLK_PER_SM * 9.0 / LOGIC_OPS_PER_9_WORDS * 32
    roofline_integer = {
        "bound": "alu", "kernel": "bconv3x3_kernel (LCE_KERNEL_TILED forced, all 8 launches)",
        "achieved": int_achieved / 1e12, "peak": probe_ops * 32 / 1e12, "unit": "T binary-MAC/s", "frac": int_achieved / (probe_ops * 32),
        "peak_source": "measured in this process: best register-resident instruction mix (nine-word carry-save tree, weighted sum on the FMA pipe)",
        "peak_naive_mix": probe_naive * 32 / 1e12,
        "peak_derived": derived / 1e12, "frac_of_derived": int_achieved / derived,
        "peak_derived_source": "SMs x max SM clock x 64 logic lanes/clk/SM x 9/16.75 word-ops per logic op x 32",
        "ms_per_step": float(np.mean(int_ms)), "avg_launch_us": int_launch_ms * 1e3,
        "frac_bitpacked_launches": rate(us_int, bit) / (probe_ops * 32), "frac_float_launches": rate(us_int, flt) / (probe_ops * 32),
        "frac_of_derived_bitpacked_launches": rate(us_int, bit) / derived,
        "traffic": profiled_traffic("bconv3x3_kernel"),
        "staging_probe": staging_probe(probe, BATCH),
    }
    per_layer = {
        l["spec"].name: {"kernel": "tensor" if l["kernel"] == lce.KERNEL_TENSOR else "integer", "us": us_auto[j],
                         "T_bmac_per_s": l["spec"].binary_macs / (us_auto[j] * 1e-6) / 1e12,
                         "integer_kernel_us": us_int[j], "integer_kernel_T_bmac_per_s": l["spec"].binary_macs / (us_int[j] * 1e-6) / 1e12}
        for j, l in enumerate(layers)
    }

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "e2m1 operands, fp32 accumulate (exact integers)" if all_tensor else "int32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": BATCH, "parallelism": f"batch-split x{world}, no collective",
                   "l2": "flushed between steps by a 256 MiB write", "launch": "one CUDA graph replay per step",
                   "dispatch": "LCE_KERNEL_AUTO on load-time packed weights"},
        "images_per_second": images_per_s,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms, "api": "lce_bconv2d_host_async on two streams, synchronised every step (pinned host buffers, plain weights)"},
        "gpu_launches": args.steps * len(layers),
        "clocks": clocks, "sustained": sustained, "roofline": roofline, "roofline_integer": roofline_integer, "per_layer": per_layer,
        "wall_s_timed_region": wall,
    }
    if world == 1 and not args.no_chains:
        line["chains"] = time_chains(dev)
        line["e2e_chain_config5"] = time_chain_e2e(dev)
        if not args.no_sweep:
            line["paper_sweep"] = time_paper_sweep(dev)
        line["streaming_kernels"] = time_streaming_kernels(dev)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cores = len(os.sched_getaffinity(0))
        items = oracle_items(BATCH, rank)
        v, dt, passes, ref = time_oracle(items, passes=2, min_seconds=10.0)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"all 8 launches of config 2 at batch {BATCH}, {passes} passes of {dt:.1f} s"}
        # the oracle's first pass doubles as the parity run of the timed launches: every output element
        checked = mismatches = 0
        for l, want in zip(layers, ref):
            got = l["timed_out"].cpu().numpy()
            got = got.view(np.uint32) if want.dtype == np.uint32 else got
            checked += int(want.size)
            mismatches += int((got != want).sum())
        line["parity"] = {"checked_elements": checked, "mismatches": mismatches,
                          "what": "outputs of the timed launches against the CPU oracle, element by element (floats compared for equality)"}
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


def time_chain_e2e(dev, reps: int = 3):
    """Config 5 end to end for a caller whose tensors live in host memory: every repetition copies the
    fp32 input batch in from pinned host memory (154 MB), runs the 18 kernels of the chain and copies
    only the final float tensor back (25.7 MB); wall clock around a synchronised repetition."""
    import torch

    from chains import Chain
    steps = wl.config5_steps()
    chain = Chain(steps, 5, str(dev))
    x_host = torch.randn((256, 224, 224, 3), dtype=torch.float32).pin_memory()
    y_host = torch.empty((256, 7, 7, 512), dtype=torch.float32).pin_memory()
    macs = sum(s.conv.binary_macs for s in steps if s.kind.startswith("bconv"))

    def once():
        chain.buffers["X"].copy_(x_host, non_blocking=True)
        chain.run()
        y_host.copy_(chain.buffers["T17"], non_blocking=True)
        torch.cuda.synchronize(dev)
    once()
    t0 = time.perf_counter()
    for _ in range(reps):
        once()
    ms = 1e3 * (time.perf_counter() - t0) / reps
    out = {"batch": 256, "ms": ms, "images_per_second": 256 / (ms * 1e-3), "binary_macs_per_second": macs / (ms * 1e-3),
           "h2d_bytes": x_host.numel() * 4, "d2h_bytes": y_host.numel() * 4}
    del chain
    torch.cuda.empty_cache()
    return out


def time_streaming_kernels(dev, reps: int = 20):
    """The HBM-bound kernels around the convolution (LceQuantize, LceBMaxPool2d, the shortcut add) on
    tensors larger than the L2, each against the measured copy bandwidth: bytes moved / time."""
    import torch

    import paper_2011_09398_b200 as lce
    peak = peak_hbm_bytes_per_s()
    out = {}

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) * 1e-3 / reps

    def entry(name, seconds, nbytes):
        out[name] = {"us": seconds * 1e6, "GB_per_s": nbytes / seconds / 1e9, "frac_of_measured_hbm": nbytes / seconds / peak}

    x = torch.randn((256, 112, 112, 64), device=dev)                       # 822 MB of fp32
    words = lce.lce_bitpack(x)
    entry("bitpack_256x112x112x64", timed(lambda: lce.lce_bitpack(x, words)), x.numel() * 4 + words.numel() * 4)
    rgb = torch.randn((256, 224, 224, 3), device=dev)                      # 154 MB: the config 5 input
    w3 = lce.lce_bitpack(rgb)
    entry("bitpack_256x224x224x3", timed(lambda: lce.lce_bitpack(rgb, w3)), rgb.numel() * 4 + w3.numel() * 4)
    back = torch.empty_like(x)
    entry("unpack_256x112x112x64", timed(lambda: lce.lce_unpack(words, 64, back)), x.numel() * 4 + words.numel() * 4)
    del back
    y = torch.randn_like(x)
    z = torch.empty_like(x)
    entry("add_f32_256x112x112x64", timed(lambda: lce.lce_add_f32(x, y, z)), 3 * x.numel() * 4)
    big = torch.randint(-2**31, 2**31 - 1, (256, 224, 224, 8), dtype=torch.int32, device=dev)   # 411 MB of packed words
    pooled = lce.lce_bmaxpool(big, 256)
    entry("bmaxpool2x2_256x224x224x256", timed(lambda: lce.lce_bmaxpool(big, 256, out=pooled)), big.numel() * 4 + pooled.numel() * 4)
    return out


def time_paper_sweep(dev, reps: int = 3):
    """The paper's convolution sweep (Section 5.1: Cin = Cout in {32..256}, 8..64 pixels square, 3x3 and
    5x5, stride 1, same padding, float output) through the default integer path: 48 layers, each timed
    alone as a CUDA-graph replay of 10 launches, at the headline batch and one image at a time (the
    paper's setting).  Reported beside the headline, outside its timed region."""
    import torch

    import paper_2011_09398_b200 as lce
    stream = torch.cuda.Stream(device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.SEED0 % (2**31))
    out = {}
    for batch in (BATCH, 1):
        rows, total_s, total_macs = {}, 0.0, 0
        for s in wl.sweep_specs(batch):
            a = torch.randint(-2**31, 2**31 - 1, (s.batch, s.in_h, s.in_w, s.in_words), dtype=torch.int32, device=dev, generator=gen)
            w = torch.randint(-2**31, 2**31 - 1, (s.out_c, s.kernel, s.kernel, s.in_words), dtype=torch.int32, device=dev, generator=gen)
            mult = torch.rand(s.out_c, device=dev, generator=gen) + 0.5
            bias = torch.randn(s.out_c, device=dev, generator=gen) * 0.1
            desc = lce.make_desc(s.batch, s.in_h, s.in_w, s.in_c, s.out_c, (s.kernel, s.kernel), (1, 1), s.padding,
                                 s.out_type, lce.ACT_NONE, lce.KERNEL_AUTO, 1)
            wp = lce.lce_bconv2d_pack_weights(desc, w)
            o = lce.lce_bconv2d(desc, a, wp, mult, bias, None)
            with torch.cuda.stream(stream):
                stream.wait_stream(torch.cuda.current_stream(dev))
                for _ in range(3):
                    lce.lce_bconv2d(desc, a, wp, mult, bias, None, o)
                stream.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    for _ in range(10):
                        lce.lce_bconv2d(desc, a, wp, mult, bias, None, o)
                g.replay()
                stream.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(reps):
                    g.replay()
                e1.record(stream)
                stream.synchronize()
            sec = e0.elapsed_time(e1) * 1e-3 / (10 * reps)
            rows[s.name] = {"us": round(sec * 1e6, 2), "T_bmac_per_s": round(s.binary_macs / sec / 1e12, 2)}
            total_s += sec
            total_macs += s.binary_macs
            del g, a, w, wp, o
        rates = [r["T_bmac_per_s"] for r in rows.values()]
        out[f"batch_{batch}"] = {"layers": len(rows), "sum_us": total_s * 1e6, "T_bmac_per_s_whole_sweep": total_macs / total_s / 1e12,
                                 "T_bmac_per_s_min": min(rates), "T_bmac_per_s_max": max(rates), "per_layer": rows}
    return out


def time_chains(dev, reps: int = 5):
    """Configs 4 and 5 end to end (every kernel of the chain on one stream), inputs resident on the
    device; reported beside the headline number, outside its timed region."""
    import torch

    import paper_2011_09398_b200 as lce

    from chains import Chain
    out = {}
    for key, cfg, steps, name, batch in (("config4", 4, wl.config4_steps(), "X0", 128),
                                         ("config4_fused", 4, wl.config4_fused_steps(), "X0", 128),
                                         ("config5", 5, wl.config5_steps(), "X", 256)):
        chain = Chain(steps, cfg, str(dev))
        chain.buffers[name].normal_()
        for _ in range(3):
            chain.run()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        for r in range(reps):
            ev[r].record()
            chain.run()
        ev[reps].record()
        torch.cuda.synchronize()
        ms = ev[0].elapsed_time(ev[reps]) / reps
        macs = sum(s.conv.binary_macs for s in steps if s.kind.startswith("bconv"))
        out[key] = {"batch": batch, "launches": chain.launches, "ms": ms, "images_per_second": batch / (ms * 1e-3),
                               "binary_macs_per_second": macs / (ms * 1e-3)}
        del chain
        torch.cuda.empty_cache()
    return out


def peak_hbm_bytes_per_s() -> float:
    p = ROOT / "MEASURED_PEAKS.json"
    try:
        return float(json.loads(p.read_text())["hbm_gbs"]) * 1e9
    except Exception:
        return 6650e9  # fallback figure of this pool


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="lce", choices=["lce", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-chains", action="store_true", help="skip the config 4 / config 5 chain timings")
    ap.add_argument("--no-sweep", action="store_true", help="skip the paper's 48-layer convolution sweep")
    ap.add_argument("--profile", action="store_true",
                    help="short form for runs under ncu: the timed steps of the default and the integer path only (no one-second "
                         "clock loop, chains, sweep or CPU baseline)")
    args = ap.parse_args()
    if args.profile:
        args.no_chains = args.no_cpu_baseline = True
    if args.impl == "reference":
        run_reference(args)
    else:
        run_lce(args)


if __name__ == "__main__":
    main()
