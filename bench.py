#!/usr/bin/env python
"""Benchmark of the sdwino hot path on the Stable Diffusion 3x3-convolution sweeps.

A step is one pass over the stride-1 pad-1 3x3 convolutions of a workload, each run through the C ABI
(activation transform -> batched tcgen05 GEMM -> output transform + bias, or one of the single-kernel
paths).  The filter transform is the once-per-weight preprocess and runs before the timed region; its
time is reported separately.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

By default all five workloads are measured (single layer, SD v1.5 UNet, SD VAE decoder, SD v2.1 UNet,
SDXL at 1024x1024) and the headline `value` sits on the largest one, `sdxl_1024`; the others are in
`workloads`.  Prints ONE JSON line (rank 0).  With --gpus N > 1 (under torchrun) every rank runs an
independent replica of the sweep on its own GPU (the path has no exchange step); the time is the max
over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "direct-conv-equivalent TFLOP/s over {sweep} (2*N*K*C*H*W*9 / time)"
_SWEEP_NAMES = {"single": "the single 320->320 at 32x32 layer", "sd15_unet": "the SD v1.5 UNet 3x3 conv sweep",
                "sd_vae_512": "the SD VAE decoder (512x512) 3x3 conv sweep", "sd21_unet": "the SD v2.1 UNet 3x3 conv sweep",
                "sdxl_1024": "the SDXL (1024x1024) UNet + VAE decoder 3x3 conv sweep"}
ALL_WORKLOADS = ["single", "sd15_unet", "sd_vae_512", "sd21_unet", "sdxl_1024"]
HEADLINE = "sdxl_1024"      # the largest single-GPU configuration


def metric_name(workload: str) -> str:
    return METRIC.format(sweep=_SWEEP_NAMES[workload])


UNIT = "TFLOP/s"
TILE = "auto"   # per layer: what sdwino_choose_algorithm returns; --tile 1 / 2 / 4 force one algorithm
L2_BYTES = 126e6
SUSTAINED_SECONDS = 2.2
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
PAPER_CONTEXT = {"per_layer_speedup_vs_sdcpp_m1pro": 2.76, "end_to_end_speedup_vs_sdcpp_m1pro": 4.79}

# DRAM traffic of the GEMM launches of one step (ncu: dram__bytes_read.sum + dram__bytes_write.sum, summed over the
# GEMM launches of a step and divided by their number), per workload with the per-layer tile choice.  Each entry
# records the capture it came from and the hash of the kernel sources it was taken with; `roofline.traffic` is null,
# with the reason, when the sources have changed since.
GEMM_DRAM_TRAFFIC = {
    "single": {"bytes_per_launch": 2134272, "launches": 1, "source_hash": "efa84ef76a2a",
                  "capture": "ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum --cache-control none "
                             "--clock-control none -k regex:wino_gemm -s 3 -c 1 python bench.py --workload single --no-cpu-baseline "
                             "--no-yardstick --no-e2e --no-sustained --no-graph --steps 2 --warmup 3 (one pass per launch; the fourth step)"},
    "sd15_unet": {"bytes_per_launch": 45421380, "launches": 15, "source_hash": "efa84ef76a2a",
                  "capture": "ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum --cache-control none "
                             "--clock-control none -k regex:wino_gemm -s 45 -c 15 python bench.py --workload sd15_unet --no-cpu-baseline "
                             "--no-yardstick --no-e2e --no-sustained --no-graph --steps 2 --warmup 3 (one pass per launch; the fourth step)"},
    "sd_vae_512": {"bytes_per_launch": 270605760, "launches": 8, "source_hash": "efa84ef76a2a",
                  "capture": "ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum --cache-control none "
                             "--clock-control none -k regex:wino_gemm -s 24 -c 8 python bench.py --workload sd_vae_512 --no-cpu-baseline "
                             "--no-yardstick --no-e2e --no-sustained --no-graph --steps 2 --warmup 3 (one pass per launch; the fourth step)"},
    "sd21_unet": {"bytes_per_launch": 51061486, "launches": 15, "source_hash": "efa84ef76a2a",
                  "capture": "ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum --cache-control none "
                             "--clock-control none -k regex:wino_gemm -s 45 -c 15 python bench.py --workload sd21_unet --no-cpu-baseline "
                             "--no-yardstick --no-e2e --no-sustained --no-graph --steps 2 --warmup 3 (one pass per launch; the fourth step)"},
    "sdxl_1024": {"bytes_per_launch": 473147325, "launches": 23, "source_hash": "efa84ef76a2a",
                  "capture": "ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum --cache-control none "
                             "--clock-control none -k regex:wino_gemm -s 69 -c 23 python bench.py --workload sdxl_1024 --no-cpu-baseline "
                             "--no-yardstick --no-e2e --no-sustained --no-graph --steps 2 --warmup 3 (one pass per launch; the fourth step)"},
}


def kernel_source_hash() -> str:
    """Hash of the CUDA sources: ties a stored ncu figure to the build it was captured on."""
    csrc = os.path.join(ROOT, "paper_2412_05781_b200", "csrc")
    h = hashlib.sha256()
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh")):
            with open(os.path.join(csrc, name), "rb") as f:
                h.update(name.encode())
                h.update(f.read())
    return h.hexdigest()[:12]


def stored_traffic(workload: str, tile: str, layer_subset: str):
    entry = GEMM_DRAM_TRAFFIC.get(workload)
    if entry is None or tile != "auto" or layer_subset:
        return None, "no ncu capture stored for this workload / tile / layer subset"
    if entry["source_hash"] != kernel_source_hash():
        return None, f"stale: the kernel sources changed since the capture ({entry['capture']})"
    return entry["bytes_per_launch"], entry["capture"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"]))}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML (read-only) while the GPU works."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake", 0x2: "applications_clocks_setting"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                util = nv.nvmlDeviceGetUtilizationRates(self.h).gpu
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((int(mhz), int(util)))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        loaded = [m for m, u in self.samples if u > 0] or [m for m, _ in self.samples]
        return {"sm_mhz": int(statistics.median(loaded)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The slowest rank's figure: every multi-GPU number is the max over ranks of a device-side time."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(flops_per_replica: float, world: int, ms_per_step: float) -> float:
    """Whole-job throughput in TFLOP/s of `world` independent replicas that each do
    `flops_per_replica` per step, the step taking `ms_per_step` on the slowest rank."""
    return world * flops_per_replica / (ms_per_step * 1e-3) / 1e12


def visible_to_nvml_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------------
# reference arm: the fp64 oracle on the host cores
# ------------------------------------------------------------------------------------------
def oracle_sample(layers, inputs, channels_per_layer, seed=0):
    """Direct fp64 convolution of `channels_per_layer` seeded output channels of every layer.
    Returns (seconds, direct flops computed)."""
    import numpy as np
    import oracle
    flops, t = 0, 0.0
    for li, (L, (x, w, b)) in enumerate(zip(layers, inputs)):
        rng = np.random.default_rng(seed + li)
        ks = np.sort(rng.choice(L.K, size=min(channels_per_layer, L.K), replace=False)).tolist()
        t0 = time.perf_counter()
        oracle.direct_conv3x3(x, w, b, channels=ks)
        t += time.perf_counter() - t0
        flops += 2 * L.N * len(ks) * L.C * L.H * L.W * 9
    return t, flops


def oracle_budgeted_sample(layers, inputs, seconds: float, order_seed: int = 0, start: int = 0, max_layers=None):
    """The oracle as it stands, on a bounded sample: it parallelises over output channels, so a sample is one seeded
    output channel per host thread of one layer; layers are taken in a seeded order, beginning at position `start`
    of that order, until `seconds` have been used (a layer is skipped when the rate seen so far says that it alone
    would overrun the rest of the budget by half).  Returns (seconds, flops, names of the sampled layers)."""
    import numpy as np
    import oracle
    nthreads = oracle.threads()
    order = np.random.default_rng(order_seed).permutation(len(layers)).tolist()
    order = order[start % len(order):] + order[:start % len(order)]
    t_tot, f_tot, names = 0.0, 0, []
    for li in order:
        L = layers[li]
        nch = min(L.K, nthreads)
        flops = 2 * L.N * nch * L.C * L.H * L.W * 9
        if names and f_tot > 0 and flops / (f_tot / t_tot) > 1.5 * (seconds - t_tot):
            continue
        t, f = oracle_sample([L], [inputs[li]], nch, seed=li)
        t_tot += t
        f_tot += f
        names.append(L.name)
        if t_tot >= seconds or (max_layers is not None and len(names) >= max_layers):
            break
    return t_tot, f_tot, names


def select_layers(workload: str, layer_subset: str):
    """A workload, optionally cut down to some of its layers (profiling runs)."""
    from paper_2412_05781_b200 import workloads
    layers = workloads.WORKLOADS[workload]()
    if layer_subset:
        layers = [layers[int(i)] for i in layer_subset.split(",")]
    return layers


def host_inputs(layers):
    from paper_2412_05781_b200 import workloads
    out = []
    for li, L in enumerate(layers):
        x, w, b = workloads.make_inputs(L, seed=li)
        out.append((x.numpy(), w.numpy(), b.numpy()))
    return out


def headline_of(args) -> str:
    return HEADLINE if args.workload == "all" else args.workload


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    workload = headline_of(args)
    layers = select_layers(workload, args.layers)
    inputs = host_inputs(layers)
    # A bounded sample per step: one layer (the steps walk the layers in a seeded order), one seeded output channel
    # per host thread, which is how the oracle's loops use the cores.
    for i in range(args.warmup):
        oracle_budgeted_sample(layers, inputs, 1e9, start=i, max_layers=1)
    t_tot, f_tot, seen = 0.0, 0, []
    for i in range(args.steps):
        t, f, names = oracle_budgeted_sample(layers, inputs, 1e9, start=args.warmup + i, max_layers=1)
        t_tot += t
        f_tot += f
        seen += names
    val = f_tot / t_tot / 1e12
    sample = (f"per step one layer of the {len(layers)} (seeded order, {len(set(seen))} distinct layers over the run), "
              f"min(K, {oracle.threads()}) seeded output channels of it (fp64 direct conv)")
    line = {
        "impl": "reference", "metric": metric_name(workload), "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_tot / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload, "layers": len(layers), "batch": layers[0].N, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------
class Ctx:
    """What every workload measurement shares: the binding, the device, the timing stream, the peaks."""
    pass


def bench_workload(ctx, args, workload: str, headline: bool):
    """Measures one workload; returns its record (see the keys at the end)."""
    import torch
    from paper_2412_05781_b200 import workloads
    B, dev, stream, dist, world, rank = ctx.B, ctx.dev, ctx.stream, ctx.dist, ctx.world, ctx.rank
    peaks, peak_kind = ctx.peaks, ctx.peak_kind
    steps, warmup = args.steps, max(args.warmup, 3)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    layers = select_layers(workload, args.layers)
    tiles = [B.sdwino_choose_algorithm(L.N, L.C, L.H, L.W, L.K) if args.tile == "auto" else int(args.tile) for L in layers]
    io32 = args.io == "f32"       # the fp32 interface: x, w, bias, y in fp32
    if io32 or args.weights == "q8":   # those interfaces have no direct form
        tiles = [B.sdwino_choose_tile(L.N, L.C, L.H, L.W, L.K) if t == 1 else t for L, t in zip(layers, tiles)]
    io_bytes = 4.0 if io32 else 2.0
    io_t = torch.float32 if io32 else torch.float16

    # ---- inputs: pinned host copies (for the end-to-end pass) and resident device copies ----
    host, devt = [], []
    ws_bytes = 0
    for li, L in enumerate(layers):
        x, w, b = workloads.make_inputs(L, seed=li, pin=not args.no_e2e)
        y_h = torch.empty(L.N, L.K, L.H, L.W, dtype=torch.float16)
        if not args.no_e2e:
            y_h = y_h.pin_memory()
        host.append((x, w, b, y_h))
        ws_bytes = max(ws_bytes, B.sdwino_workspace_bytes(L.N, L.C, L.H, L.W, L.K, tiles[li]))
    ws = B.alloc_workspace(ws_bytes, dev)

    # filter transform: once per weight, outside the timed step; timed on its own
    B.sdwino_profile_enable(1)
    w_dev = [h[1].to(dev).float() if io32 else h[1].to(dev) for h in host]
    for _ in range(3):
        wTs = [(B.sdwino_filter_transform_f32 if io32 else B.sdwino_filter_transform)(wd, t) for wd, t in zip(w_dev, tiles)]
        prof = B.sdwino_profile_collect()
    ft_ms = prof["filter_transform"][0]
    ft_bytes = sum(L.K * L.C * 9 * io_bytes + B.sdwino_filter_bytes(L.K, L.C, t) for L, t in zip(layers, tiles))
    B.sdwino_profile_enable(0)
    del w_dev
    q8 = [args.weights == "q8" and not io32 and min(L.C, L.K) > 8 for L in layers]
    wTs = [B.sdwino_filter_quantize(wT, L.K, L.C, t) if q else wT for wT, L, t, q in zip(wTs, layers, tiles, q8)]
    for (x, w, b, y_h), wT in zip(host, wTs):
        devt.append((x.to(dev).to(io_t), wT, b.to(dev).to(io_t), torch.empty(y_h.shape, dtype=io_t, device=dev)))
    if args.epilogue != "none":
        gres = torch.Generator().manual_seed(1234)
        res_dev = [torch.randn(y_h.shape, generator=gres).to(io_t).to(dev) for (_, _, _, y_h) in host]
        act = B.ACT_SILU if args.epilogue == "residual_silu" else B.ACT_NONE

    def run_layer(li, strm):
        L, t, (xd, wT, bd, yd) = layers[li], tiles[li], devt[li]
        if q8[li]:
            B.sdwino_conv3x3_q8(xd, wT, bd, L.K, t, ws, y=yd, stream=strm)
        elif io32 and (args.epilogue == "none" or min(L.C, L.K) <= 8):
            B.sdwino_conv3x3_f32(xd, wT, bd, L.K, t, ws, y=yd, stream=strm)
        elif io32:
            B.sdwino_conv3x3_f32_ex(xd, wT, bd, res_dev[li], L.K, t, act, ws, y=yd, stream=strm)
        elif args.epilogue == "none" or min(L.C, L.K) <= 8:     # the first and last convolution of a network have neither
            B.sdwino_conv3x3(xd, wT, bd, L.K, t, y=yd, workspace=ws, stream=strm)
        else:
            B.sdwino_conv3x3_ex(xd, wT, bd, res_dev[li], L.K, t, act, ws, y=yd, stream=strm)

    # --sequence: the whole step is ONE call of the multi-layer entry (same kernels in the same order; with
    # --prefetch-mb > 0 each layer's filters are sent towards L2 while the layer before it computes)
    use_sequence = args.sequence and not io32 and args.epilogue == "none" and not any(q8)
    if use_sequence:
        seq = B.make_sequence([(xd, wT, bd, yd, L.K, t) for L, t, (xd, wT, bd, yd) in zip(layers, tiles, devt)])

    def step():
        if use_sequence:
            B.sdwino_conv3x3_sequence(seq, ws, args.prefetch_mb << 20, stream=torch.cuda.current_stream())
            return
        for li in range(len(layers)):
            run_layer(li, torch.cuda.current_stream())

    # The timed step is replayed from a CUDA graph captured from the same C-ABI calls, so that host launch latency
    # (about three launches per layer) does not enter the device-resident number; --no-graph launches directly.
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            step()
    stream.synchronize()
    l0 = B.sdwino_launch_count()
    graph = None
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step()
        launches_per_step = B.sdwino_launch_count() - l0
        with torch.cuda.stream(stream):
            for _ in range(3):
                graph.replay()
    else:
        with torch.cuda.stream(stream):
            step()
        launches_per_step = B.sdwino_launch_count() - l0
    stream.synchronize()

    def one_step():
        if graph is not None:
            graph.replay()
        else:
            step()

    # ---- timed region: resident inputs, exactly `steps` steps, an event after every step ----
    flops_step = sum(L.direct_flops for L in layers)
    def filt_bytes(L, t, q):
        return B.sdwino_filter_q8_bytes(L.K, L.C, t) if q else B.sdwino_filter_bytes(L.K, L.C, t)
    step_bytes = sum(io_bytes * L.N * (L.C + L.K) * L.H * L.W + filt_bytes(L, t, q) for L, t, q in zip(layers, tiles, q8))
    # A step that touches less than twice the L2 would find its operands cached by the previous step: then
    # the L2 is flushed (a 256 MB buffer is written) before every step and only the steps are timed.
    flush_l2 = step_bytes < 2 * L2_BYTES
    sampler = ClockSampler(visible_to_nvml_index(ctx.local_rank)).start() if headline else None
    barrier()
    if not flush_l2:
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        with torch.cuda.stream(stream):
            ev[0].record(stream)
            for i in range(steps):
                one_step()
                ev[i + 1].record(stream)
        stream.synchronize()
        ms_total = ev[0].elapsed_time(ev[steps])
        per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    else:
        flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        with torch.cuda.stream(stream):
            for a, b_ in pairs:
                flush_buf.fill_(1)
                a.record(stream)
                one_step()
                b_.record(stream)
        stream.synchronize()
        per_step = [a.elapsed_time(b_) for a, b_ in pairs]
        ms_total = sum(per_step)
        del flush_buf
    barrier()
    clocks = sampler.stop() if sampler is not None else None
    ms_step = max_over_ranks(ms_total, dist, dev) / steps
    assert B.sdwino_last_device_status(stream) == B.OK, "a device-side wait timed out"
    value = aggregate_value(flops_step, world, ms_step)

    # ---- sustained leg: back-to-back replays for at least two seconds, with the clocks that were seen.  For a
    #      workload whose timed steps flush the L2 this leg does not: it is the L2-warm figure. ----
    sustained = None
    if not args.no_sustained:
        n_sus = max(steps, min(200000, int(math.ceil(SUSTAINED_SECONDS * 1e3 / max(min(per_step), 1e-3)))))
        sus_sampler = ClockSampler(visible_to_nvml_index(ctx.local_rank)).start()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            s0.record(stream)
            for _ in range(n_sus):
                one_step()
            s1.record(stream)
        stream.synchronize()
        sus_clocks = sus_sampler.stop()
        sus_ms = max_over_ranks(s0.elapsed_time(s1), dist, dev) / n_sus
        sustained = {"steps": n_sus, "seconds": round(sus_ms * n_sus * 1e-3, 3), "ms_per_step": round(sus_ms, 4),
                     "value": round(aggregate_value(flops_step, world, sus_ms), 2), "unit": UNIT,
                     "l2": "warm (no flush between steps)" if flush_l2 else "as in the timed steps",
                     "clocks": sus_clocks,
                     "ms_x_mhz": round(sus_ms * sus_clocks["sm_mhz"], 1) if sus_clocks.get("sm_mhz") else None}

    # ---- the same step launched directly (no graph): what a caller without graphs sees ----
    direct_ms = None
    if graph is not None:
        nd = min(steps, 20)
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            step()
            d0.record(stream)
            for _ in range(nd):
                step()
            d1.record(stream)
        stream.synchronize()
        direct_ms = d0.elapsed_time(d1) / nd

    # ---- per-layer times: the step replayed from a graph in which every convolution call (not every kernel) is
    #      bracketed by event nodes, so the kernels of a layer keep their programmatic overlap and the layer times
    #      add up to the step; then per-kernel times (events around every launch), used for the split of a
    #      layer's time over its kernels. ----
    prof_steps = max(3, min(steps, 20))
    layer_ms = [0.0] * len(layers)
    per_layer = [dict(input_transform=0.0, wino_gemm=0.0, output_transform=0.0, fused=0.0, launches=0) for _ in layers]

    def profiled_pass(mode, account):
        B.sdwino_profile_enable(mode)
        if not args.no_graph:
            pgraph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(pgraph, stream=stream):
                step()
            for _ in range(prof_steps):
                with torch.cuda.stream(stream):
                    pgraph.replay()
                stream.synchronize()
                account(B.sdwino_profile_records(keep=True))
            B.sdwino_profile_records()
            del pgraph
        else:
            for _ in range(prof_steps):
                with torch.cuda.stream(stream):
                    step()
                stream.synchronize()
                account(B.sdwino_profile_records())
        B.sdwino_profile_enable(0)

    def account_layers(recs):
        assert len(recs) == len(layers) and all(k == "layer" and ms >= 0 for k, ms in recs)
        for li, (_, ms) in enumerate(recs):
            layer_ms[li] += ms / prof_steps

    profiled_pass(2, account_layers)
    B.sdwino_profile_enable(1)
    records_per_layer = []
    with torch.cuda.stream(stream):
        for li in range(len(layers)):     # learn how many launches each layer makes
            run_layer(li, stream)
            records_per_layer.append(len(B.sdwino_profile_records()))
    B.sdwino_profile_enable(0)

    def account_kernels(recs):
        assert len(recs) == sum(records_per_layer) and all(ms >= 0 for _, ms in recs)
        it = iter(recs)
        for li, nrec in enumerate(records_per_layer):
            for _ in range(nrec):
                kind, ms = next(it)
                per_layer[li][kind] += ms / prof_steps
                if kind == "wino_gemm":
                    per_layer[li]["launches"] += 1

    profiled_pass(1, account_kernels)

    tpeak = peaks["bf16_tflops"]          # burst figure (the larger denominator); the sustained one is given beside it
    tpeak_sus = peaks["bf16_tflops_sustained"]
    hpeak = peaks["hbm_gbs"]

    def gbs(nbytes, ms):
        return nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0

    layer_rows = []
    gemm_flops = gemm_ms = gemm_u_bytes = gemm_io_bytes = 0.0
    in_ms = out_ms = in_bytes = out_bytes = fused_ms = 0.0
    for L, t, pl, lms, q in zip(layers, tiles, per_layer, layer_ms, q8):
        a2 = (t + 2) ** 2
        P = L.tiles(t)
        wino_flops = 2.0 * a2 * L.K * L.C * P
        u_bytes = filt_bytes(L, t, q)
        xb, yb = io_bytes * L.N * L.C * L.H * L.W, io_bytes * L.N * L.K * L.H * L.W
        t_tensor = wino_flops / (tpeak * 1e12) * 1e6
        t_hbm = (xb + (1.0 if q else 2.0) * a2 * L.K * L.C + yb + 2 * L.K) / (hpeak * 1e9) * 1e6
        ksum = pl["input_transform"] + pl["wino_gemm"] + pl["output_transform"] + pl["fused"]
        scale = lms / ksum if ksum > 0 else 0.0     # the kernels' event-bracketed times, scaled to the layer's time
        k_in, k_gemm, k_out, k_fused = (pl[k] * scale for k in ("input_transform", "wino_gemm", "output_transform", "fused"))
        total_us = lms * 1e3
        layer_rows.append({
            "layer": L.name, "tile": t, "us": round(total_us, 2),
            "us_input": round(k_in * 1e3, 2), "us_gemm": round(k_gemm * 1e3, 2),
            "us_output": round(k_out * 1e3, 2), "us_fused": round(k_fused * 1e3, 2),
            "eq_tflops": round(L.direct_flops / (total_us * 1e-6) / 1e12, 1) if total_us > 0 else None,
            "bound": "tensor" if t_tensor >= t_hbm else "hbm",
            "roof_us": round(max(t_tensor, t_hbm), 2),
            "frac_of_roof": round(max(t_tensor, t_hbm) / total_us, 3) if total_us > 0 else None,
            "gemm_tensor_frac": (round(wino_flops / (k_gemm * 1e-3) / 1e12 / tpeak, 3) if k_gemm > 0 else None),
        })
        if pl["wino_gemm"] > 0:                  # layers on a single-kernel path have no GEMM launch
            gemm_flops += wino_flops
            gemm_u_bytes += u_bytes
            gemm_io_bytes += u_bytes + 2.0 * a2 * (L.C + L.K) * P      # what the unfused GEMM must move: U, V in, M out
            gemm_ms += k_gemm
            in_ms += k_in
            out_ms += k_out
            in_bytes += xb + 2.0 * a2 * L.C * P      # read x, write V
            out_bytes += 2.0 * a2 * L.K * P + yb     # read M, write y
        fused_ms += k_fused
    gemm_launches = sum(pl["launches"] for pl in per_layer) / prof_steps
    achieved = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    traffic, traffic_note = stored_traffic(workload, args.tile, args.layers)
    sum_layers_ms = sum(layer_ms)
    roofline = {
        "kernel": "wino_gemm_kernel", "bound": "tensor", "achieved": round(achieved, 1), "peak": tpeak,
        "unit": "TFLOP/s", "frac": round(achieved / tpeak, 4),
        "frac_of_sustained_peak": round(achieved / tpeak_sus, 4),
        "traffic": traffic, "traffic_unit": "bytes per launch (ncu dram read + write, L2 left warm)",
        "traffic_source": traffic_note,
        "peak_source": f"{peak_kind} (cuBLAS bf16 burst {tpeak}, sustained {tpeak_sus}; fp16 has the same nominal rate)",
        "launches_per_step": gemm_launches,
        "avg_launch_us": round(gemm_ms * 1e3 / gemm_launches, 2) if gemm_launches else None,
        "algorithmic_flops_per_step": gemm_flops,
        "share_of_step": round(gemm_ms / sum_layers_ms, 3) if sum_layers_ms > 0 else None,
        "sum_of_layer_times_over_step": round(sum_layers_ms / ms_step, 3),
    }
    # the same launches against the other roof: the GEMM is the kernel that streams the transformed weights, and
    # on the small-image layers that stream, not the tensor pipe, is what bounds it
    roofline["weight_stream_view"] = {
        "bound": "hbm", "algorithmic_bytes_per_step": gemm_u_bytes,
        "achieved": round(gbs(gemm_u_bytes, gemm_ms), 1), "peak": hpeak, "unit": "GB/s",
        "frac": round(gbs(gemm_u_bytes, gemm_ms) / hpeak, 4)}
    # ... and against the bytes the GEMM kernel itself must move in the three-kernel design (U, V in, M out): on the
    # large layers this, not the tensor pipe, is what bounds the launch (V and M do not fit in L2)
    roofline["operand_stream_view"] = {
        "bound": "hbm", "bytes_per_step": gemm_io_bytes, "achieved": round(gbs(gemm_io_bytes, gemm_ms), 1), "peak": hpeak,
        "unit": "GB/s", "frac": round(gbs(gemm_io_bytes, gemm_ms) / hpeak, 4),
        "note": "U + V + M of the GEMM launches over their time; an L2 hit counts like a DRAM access, so small layers can exceed 1"}
    # the whole step against the per-layer roofline max(tensor time, mandatory HBM bytes / bandwidth), both at
    # the measured peaks: what an ideal implementation of each layer would need, summed over the sweep
    roof_us_sum = sum(r["roof_us"] for r in layer_rows)
    roofline["step_vs_layer_rooflines"] = {
        "sum_of_layer_rooflines_us": round(roof_us_sum, 1), "step_us": round(ms_step * 1e3, 1),
        "frac": round(roof_us_sum / (ms_step * 1e3), 3),
        "hbm_bound_layers": sum(1 for r in layer_rows if r["bound"] == "hbm"), "layers": len(layer_rows)}
    transforms = {
        "input_transform": {"gbs": round(gbs(in_bytes, in_ms), 1), "frac_of_hbm_peak": round(gbs(in_bytes, in_ms) / hpeak, 3),
                            "ms_per_step": round(in_ms, 4)},
        "output_transform": {"gbs": round(gbs(out_bytes, out_ms), 1), "frac_of_hbm_peak": round(gbs(out_bytes, out_ms) / hpeak, 3),
                             "ms_per_step": round(out_ms, 4)},
        "single_kernel_layers_ms_per_step": round(fused_ms, 4),
        "filter_transform_once_per_weight": {"ms": round(ft_ms, 4), "gbs": round(gbs(ft_bytes, ft_ms), 1),
                                             "frac_of_hbm_peak": round(gbs(ft_bytes, ft_ms) / hpeak, 3)},
        "hbm_peak_gbs": hpeak, "peak_source": peak_kind,
    }

    # ---- end to end: host buffers in, host buffers out, through the host entry of the C ABI (fp16 or fp32) ----
    e2e = None
    if not args.no_e2e and args.weights == "f16":
        host_call = B.sdwino_conv3x3_host_f32 if io32 else B.sdwino_conv3x3_host
        staging = B.sdwino_host_staging_bytes_f32 if io32 else B.sdwino_host_staging_bytes
        e2e_bytes = [staging(L.N, L.C, L.H, L.W, L.K, t) + B.sdwino_workspace_bytes(L.N, L.C, L.H, L.W, L.K, t)
                     for L, t in zip(layers, tiles)]
        per_layer_ws = sum(e2e_bytes) <= (48 << 30)
        # a workspace (staging + scratch) per layer, so that the copies of neighbouring layers may overlap; layers
        # that share one are ordered copy after copy by the library
        shared = None if per_layer_ws else B.alloc_workspace(max(e2e_bytes), dev)
        ws_e2e = [B.alloc_workspace(nb, dev) for nb in e2e_bytes] if per_layer_ws else [shared] * len(layers)
        if io32:
            host_io = [(x.float().pin_memory(), w, b.float().pin_memory(), torch.empty(y.shape, dtype=torch.float32).pin_memory())
                       for (x, w, b, y) in host]
        else:
            host_io = host
        e2e_steps = max(3, min(steps, 30 if flops_step < 2e12 else 10))

        def e2e_step():
            for t, (x, w, b, y_h), (_, wT, _, _), wsl in zip(tiles, host_io, devt, ws_e2e):
                host_call(x, wT, b, y_h, t, wsl, stream=stream, wait=False)
            B.sdwino_host_join(stream)
            stream.synchronize()                  # y of every layer is complete in host memory

        for _ in range(3):
            e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        e2e_value = aggregate_value(flops_step, world, max_over_ranks(e2e_s, dist, dev) / e2e_steps * 1e3)
        h2d = sum(x.numel() * x.element_size() + b.numel() * b.element_size() for (x, w, b, y) in host_io)
        d2h = sum(y.numel() * y.element_size() for (x, w, b, y) in host_io)
        # what came back through the host path is what the device-resident step computed (same kernels: same bits)
        e2e_matches = args.epilogue != "none" or all(
            torch.equal(y_h, yd.cpu()) for (_, _, _, y_h), (_, _, _, yd) in zip(host_io, devt))
        assert e2e_matches, "the host path returned something else than the device path"
        e2e = {"value": round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": e2e_steps, "ms_per_step": round(e2e_s / e2e_steps * 1e3, 3), "matches_device_path": bool(e2e_matches),
               "api": ("sdwino_conv3x3_host_f32_async" if io32 else "sdwino_conv3x3_host_async") +
                      " per layer (pinned host x, bias, y; " +
                      ("a workspace per layer: uploads and downloads overlap the neighbouring layers" if per_layer_ws
                       else "one shared workspace: the copies of differently sized layers are ordered one after the other") +
                      "), one join + stream synchronisation per step"}
        del ws_e2e, shared, host_io

    # ---- cuDNN yardstick (not the target) ----
    cudnn = None
    if rank == 0 and not args.no_yardstick:
        try:
            import torch.nn.functional as F
            torch.backends.cudnn.benchmark = True
            wd = [h[1].to(dev).to(io_t) for h in host]
            for _ in range(3):
                for (xd, _, bd, _), w_ in zip(devt, wd):
                    F.conv2d(xd, w_, bd, padding=1)
            torch.cuda.synchronize()
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record()
            for _ in range(prof_steps):
                for (xd, _, bd, _), w_ in zip(devt, wd):
                    F.conv2d(xd, w_, bd, padding=1)
            c1.record()
            torch.cuda.synchronize()
            cms = c0.elapsed_time(c1) / prof_steps
            cudnn = {"value": round(flops_step / (cms * 1e-3) / 1e12, 1), "unit": UNIT, "ms_per_step": round(cms, 4),
                     "what": "torch.nn.functional.conv2d NCHW, cudnn.benchmark=True (yardstick only)"}
            del wd
        except Exception as e:  # pragma: no cover
            cudnn = {"error": repr(e)}

    # ---- oracle on the host cores (reported baseline): the headline workload at one GPU only ----
    cpu_baseline = None
    if headline and rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        inputs = [(x.numpy(), w.numpy(), b.numpy()) for (x, w, b, _) in host]
        sec, fl, names = oracle_budgeted_sample(layers, inputs, 12.0)
        cpu_baseline = {"value": fl / sec / 1e12, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                        "sample": f"fp64 direct conv of min(K, {oracle.threads()}) seeded output channels of {len(names)} of the "
                                  f"{len(layers)} layers, taken in a seeded order until 12 s were used "
                                  f"({fl / 1e9:.1f} GFLOP in {sec:.1f} s): " + ", ".join(names)}

    rec = {
        "workload": workload, "value": round(value, 2), "unit": UNIT, "ms_per_step": round(ms_step, 4),
        "ms_per_step_min": round(min(per_step), 4), "ms_per_step_median": round(statistics.median(per_step), 4),
        "steps": steps, "direct_launch_ms_per_step": round(direct_ms, 4) if direct_ms is not None else None,
        "sustained": sustained, "layers_n": len(layers), "batch": layers[0].N, "tile_per_layer": tiles,
        "launches_per_step": int(launches_per_step), "flops_per_step": flops_step,
        "l2": ((f"flushed before every timed step (256 MB written): one step touches only {step_bytes / 1e6:.0f} MB")
               if flush_l2 else
               (f"no flush: one step touches {step_bytes / 1e6:.0f} MB of distinct inputs, transformed weights and outputs "
                f"({step_bytes / L2_BYTES:.1f}x the 126 MB L2), so a layer starts with its operands cold")),
        "e2e": e2e, "roofline": roofline, "transforms": transforms, "cudnn_yardstick": cudnn, "layers": layer_rows,
        "clocks": clocks, "cpu_baseline": cpu_baseline,
    }
    del devt, host, ws, wTs, graph
    torch.cuda.empty_cache()
    return rec


def run_ours(args):
    import torch
    from paper_2412_05781_b200 import build_library
    build_library()
    from paper_2412_05781_b200 import binding as B

    ctx = Ctx()
    ctx.B = B
    ctx.world = int(os.environ.get("WORLD_SIZE", "1"))
    ctx.rank = int(os.environ.get("RANK", "0"))
    ctx.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the sdwino path has no CPU fallback")
    torch.cuda.set_device(ctx.local_rank)
    ctx.dev = torch.device("cuda", ctx.local_rank)
    ctx.dist = None
    if ctx.world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=ctx.dev)
        ctx.dist = dist_mod
    ctx.peaks, ctx.peak_kind = load_peaks()
    ctx.stream = torch.cuda.Stream()
    B.sdwino_set_pipeline(args.pipeline, args.pipe_ring, args.pipe_lead)

    head = headline_of(args)
    names = ALL_WORKLOADS if args.workload == "all" else [args.workload]
    records = {}
    for name in names:
        if name == head:
            continue
        records[name] = bench_workload(ctx, args, name, headline=False)
    records[head] = bench_workload(ctx, args, head, headline=True)   # last: its clocks and CPU baseline are the line's
    h = records[head]
    io32 = args.io == "f32"

    if ctx.rank == 0:
        def brief(r):
            return {k: r[k] for k in ("value", "unit", "ms_per_step", "ms_per_step_min", "ms_per_step_median", "steps",
                                      "direct_launch_ms_per_step", "sustained", "layers_n", "batch", "tile_per_layer",
                                      "launches_per_step", "l2", "e2e", "roofline", "transforms", "cudnn_yardstick", "layers")}
        e2e = h["e2e"] or {"value": None, "unit": UNIT, "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
                           "skipped": "--no-e2e"}
        line = {
            "metric": metric_name(head), "value": h["value"], "unit": UNIT, "n_gpus": ctx.world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": h["ms_per_step"], "ms_per_step_min": h["ms_per_step_min"],
            "ms_per_step_median": h["ms_per_step_median"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32 in/out, f16 operands, f32 accumulate" if io32 else "f16",
            "data": "synthetic",
            "config": {"workload": head, "io": args.io, "layers": h["layers_n"], "layer_subset": args.layers or "all",
                       "batch": h["batch"], "tile": args.tile, "tile_per_layer": h["tile_per_layer"],
                       "algorithm": ("Winograd F(2x2,3x3) or F(4x4,3x3), or the direct form F(1x1,3x3), per layer (sdwino_choose_algorithm)"
                                     if args.tile == "auto" else f"Winograd F({args.tile}x{args.tile},3x3)") +
                                    (", fp32 x / w / bias / y, fp16 transformed operands, fp32 accumulate"
                                     if io32 else ", fp16 storage, fp32 accumulate"),
                       "parallelism": f"replicas x{ctx.world} (no exchange step)",
                       "launch": "direct" if args.no_graph else "CUDA graph of one step, replayed",
                       "weights": args.weights,
                       "pipeline": {0: "off", 1: "where the library takes it", 2: "wherever possible"}[args.pipeline],
                       "step_call": (f"one sdwino_conv3x3_sequence call per step, {args.prefetch_mb} MB of filters prefetched per layer"
                                     if args.sequence else "one sdwino_conv3x3 call per layer"),
                       "l2": h["l2"],
                       "filter_transform": "once per weight, before the timed region (reported separately)",
                       "epilogue": {"none": "bias", "residual": "bias + residual, fused, on the layers with more than 8 input and output channels (e2e runs the plain convolution)",
                                    "residual_silu": "SiLU(bias + residual), fused, on the layers with more than 8 input and output channels (e2e runs the plain convolution)"}[args.epilogue],
                       "other_workloads_in_this_line": [n for n in names if n != head]},
            "e2e": e2e,
            "gpu_launches": int(h["launches_per_step"] * args.steps),
            "clocks": h["clocks"],
            "sustained": h["sustained"],
            "direct_launch_ms_per_step": h["direct_launch_ms_per_step"],
            "roofline": h["roofline"],
            "transforms": h["transforms"],
            "cpu_baseline": h["cpu_baseline"],
            "cudnn_yardstick": h["cudnn_yardstick"],
            "layers": h["layers"],
            "workloads": {n: brief(records[n]) for n in names},
            "kernel_source_hash": kernel_source_hash(),
            "paper_context": PAPER_CONTEXT,
        }
        print(json.dumps(line), flush=True)
    if ctx.dist is not None:
        ctx.dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=["all"] + ALL_WORKLOADS,
                    help="all: every workload, the headline on sdxl_1024; a name: that workload alone")
    ap.add_argument("--layers", default="", help="comma-separated layer indices of the workload (default: all)")
    ap.add_argument("--tile", default=TILE, choices=["auto", "1", "2", "4"])
    ap.add_argument("--io", default="f16", choices=["f16", "f32"],
                    help="element type of x, w, bias and y: f32 runs the fp32 interface (fp16 operands, fp32 accumulation)")
    ap.add_argument("--epilogue", default="none", choices=["none", "residual", "residual_silu"],
                    help="fuse y = act(conv + bias + residual) into the output transform of the timed step (sdwino_conv3x3_ex)")
    ap.add_argument("--weights", default="f16", choices=["f16", "q8"],
                    help="q8: 8-bit transformed filters (sdwino_conv3x3_q8) on every layer with more than 8 input and output channels")
    ap.add_argument("--pipeline", type=int, default=1, choices=[0, 1, 2],
                    help="the pipelined single-launch path of F(4x4): 0 never, 1 where the library takes it, 2 wherever possible")
    ap.add_argument("--pipe-ring", type=int, default=0, help="ring length of the pipelined path in blocks of 128 tiles (0: library's choice)")
    ap.add_argument("--pipe-lead", type=int, default=0, help="lag of its output transform in blocks (0: library's choice)")
    ap.add_argument("--sequence", action="store_true",
                    help="run the step as one sdwino_conv3x3_sequence call (fp16 interface, no epilogue, fp16 filters)")
    ap.add_argument("--prefetch-mb", type=int, default=0,
                    help="with --sequence: MB of the next layer's filters prefetched into L2 per layer (0: none)")
    ap.add_argument("--no-graph", action="store_true", help="launch every step directly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-yardstick", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer pass (profiling runs)")
    ap.add_argument("--no-sustained", action="store_true", help="skip the two-second back-to-back leg (profiling runs)")
    args = ap.parse_args()
    if args.layers and args.workload == "all":
        ap.error("--layers needs a --workload")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
