#!/usr/bin/env python
"""Benchmark of the sdwino hot path on the SD v1.5 UNet 3x3-convolution sweep.

A step is one pass over the 16 stride-1 pad-1 3x3 convolutions of the SD v1.5 UNet at 512x512
(latent 64x64, batch 2), each run as activation transform -> batched tcgen05 GEMM -> output
transform + bias through the C ABI.  The filter transform is the once-per-weight preprocess and
runs before the timed region; its time is reported separately.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  With --gpus N > 1 (under torchrun) every rank runs an independent
replica of the sweep on its own GPU (the path has no exchange step); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "direct-conv-equivalent TFLOP/s over the SD v1.5 UNet 3x3 conv sweep (2*N*K*C*H*W*9 / time)"
_SWEEP_NAMES = {"single": "the single 320->320 at 32x32 layer", "sd15_unet": "the SD v1.5 UNet 3x3 conv sweep",
                "sd_vae_512": "the SD VAE decoder (512x512) 3x3 conv sweep", "sd21_unet": "the SD v2.1 UNet 3x3 conv sweep",
                "sdxl_1024": "the SDXL (1024x1024) UNet + VAE decoder 3x3 conv sweep"}


def metric_name(workload: str) -> str:
    """The headline metric, named for the workload that was run (the default is the SD v1.5 sweep)."""
    return METRIC.replace("the SD v1.5 UNet 3x3 conv sweep", _SWEEP_NAMES[workload])
UNIT = "TFLOP/s"
WORKLOAD = "sd15_unet"
TILE = "auto"   # per layer: what sdwino_choose_tile returns; --tile 2 / --tile 4 force one algorithm
L2_BYTES = 126e6
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per GEMM launch of one SD v1.5 step, from ncu captures
# (profiles/launch_list_sd15_unet_sweep.md), by --tile.  Only valid for the default workload with all layers.
GEMM_DRAM_BYTES_PER_LAUNCH_SD15 = {"auto": 49.89e6, "2": 40.66e6}
PAPER_CONTEXT = {"per_layer_speedup_vs_sdcpp_m1pro": 2.76, "end_to_end_speedup_vs_sdcpp_m1pro": 4.79}


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


def select_layers(args):
    """The benchmarked workload, optionally cut down to some of its layers (profiling runs)."""
    from paper_2412_05781_b200 import workloads
    layers = workloads.WORKLOADS[args.workload]()
    if args.layers:
        layers = [layers[int(i)] for i in args.layers.split(",")]
    return layers


def host_inputs(layers):
    from paper_2412_05781_b200 import workloads
    out = []
    for li, L in enumerate(layers):
        x, w, b = workloads.make_inputs(L, seed=li)
        out.append((x.numpy(), w.numpy(), b.numpy()))
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2412_05781_b200 import workloads
    oracle.build()
    layers = select_layers(args)
    inputs = host_inputs(layers)
    nch = 2
    for _ in range(args.warmup):
        oracle_sample(layers, inputs, nch)
    t_tot, f_tot = 0.0, 0
    for _ in range(args.steps):
        t, f = oracle_sample(layers, inputs, nch)
        t_tot += t
        f_tot += f
    val = f_tot / t_tot / 1e12
    sample = f"{nch} seeded output channels of each of the {len(layers)} layers per step (fp64 direct conv)"
    line = {
        "impl": "reference", "metric": metric_name(args.workload), "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_tot / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "layers": len(layers), "batch": layers[0].N, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    from paper_2412_05781_b200 import build_library, workloads
    build_library()
    from paper_2412_05781_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the sdwino path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    peaks, peak_kind = load_peaks()
    layers = select_layers(args)
    tiles = [B.sdwino_choose_tile(L.N, L.C, L.H, L.W, L.K) if args.tile == "auto" else int(args.tile) for L in layers]

    # ---- inputs: pinned host copies (for the end-to-end pass) and resident device copies ----
    host, devt = [], []
    ws_bytes, hws_bytes = 0, 0
    for li, L in enumerate(layers):
        x, w, b = workloads.make_inputs(L, seed=li, pin=True)
        y_h = torch.empty(L.N, L.K, L.H, L.W, dtype=torch.float16).pin_memory()
        host.append((x, w, b, y_h))
        dims = (L.N, L.C, L.H, L.W, L.K, tiles[li])
        ws_bytes = max(ws_bytes, B.sdwino_workspace_bytes(*dims))
        hws_bytes = max(hws_bytes, B.sdwino_host_staging_bytes(*dims) + B.sdwino_workspace_bytes(*dims))
    ws = B.alloc_workspace(max(ws_bytes, hws_bytes), dev)
    # end-to-end pass: a workspace (staging + scratch) per layer, so that the copies of neighbouring layers may
    # overlap; layers that share one are ordered copy after copy by the library
    e2e_bytes = [B.sdwino_host_staging_bytes(L.N, L.C, L.H, L.W, L.K, t) + B.sdwino_workspace_bytes(L.N, L.C, L.H, L.W, L.K, t)
                 for L, t in zip(layers, tiles)]
    per_layer_ws = sum(e2e_bytes) <= (48 << 30)
    ws_e2e = [B.alloc_workspace(nb, dev) for nb in e2e_bytes] if per_layer_ws else [ws] * len(layers)

    # filter transform: once per weight, outside the timed step; timed on its own
    B.sdwino_profile_enable(True)
    io32 = args.io == "f32"       # the fp32 interface: x, w, bias, y in fp32 (the host arm below stays fp16)
    io_bytes = 4.0 if io32 else 2.0
    w_dev = [h[1].to(dev).float() if io32 else h[1].to(dev) for h in host]
    for _ in range(3):
        wTs = [(B.sdwino_filter_transform_f32 if io32 else B.sdwino_filter_transform)(wd, t) for wd, t in zip(w_dev, tiles)]
        prof = B.sdwino_profile_collect()
    ft_ms = prof["filter_transform"][0]
    ft_bytes = sum(L.K * L.C * 9 * io_bytes + B.sdwino_filter_bytes(L.K, L.C, t) for L, t in zip(layers, tiles))
    B.sdwino_profile_enable(False)
    del w_dev
    for (x, w, b, y_h), wT in zip(host, wTs):
        io_t = torch.float32 if io32 else torch.float16
        devt.append((x.to(dev).to(io_t), wT, b.to(dev).to(io_t), torch.empty(y_h.shape, dtype=io_t, device=dev)))
    if args.epilogue != "none":
        gres = torch.Generator().manual_seed(1234)
        res_dev = [torch.randn(y_h.shape, generator=gres).to(torch.float32 if io32 else torch.float16).to(dev)
                   for (_, _, _, y_h) in host]
        act = B.ACT_SILU if args.epilogue == "residual_silu" else B.ACT_NONE

    def run_layer(li, strm):
        L, t, (xd, wT, bd, yd) = layers[li], tiles[li], devt[li]
        if io32 and (args.epilogue == "none" or min(L.C, L.K) <= 8):
            B.sdwino_conv3x3_f32(xd, wT, bd, L.K, t, ws, y=yd, stream=strm)
        elif io32:
            B.sdwino_conv3x3_f32_ex(xd, wT, bd, res_dev[li], L.K, t, act, ws, y=yd, stream=strm)
        elif args.epilogue == "none" or min(L.C, L.K) <= 8:     # the first and last convolution of a network have neither
            B.sdwino_conv3x3(xd, wT, bd, L.K, t, y=yd, workspace=ws, stream=strm)
        else:
            B.sdwino_conv3x3_ex(xd, wT, bd, res_dev[li], L.K, t, act, ws, y=yd, stream=strm)

    def step():
        for li in range(len(layers)):
            run_layer(li, torch.cuda.current_stream())

    sampler = ClockSampler(visible_to_nvml_index(local_rank))
    # the timed step is replayed from a CUDA graph captured from the same C-ABI calls, so that host launch
    # latency (48+ launches per step) does not enter the device-resident number; --no-graph launches directly
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
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
    barrier()
    sampler.start()

    # ---- timed region: resident inputs ----
    flops_step = sum(L.direct_flops for L in layers)
    step_bytes = sum(io_bytes * L.N * (L.C + L.K) * L.H * L.W + B.sdwino_filter_bytes(L.K, L.C, t) for L, t in zip(layers, tiles))
    # A step that touches less than twice the L2 would find its operands cached by the previous step: then
    # the L2 is flushed (a 256 MB buffer is written) before every step and only the steps are timed.
    flush_l2 = step_bytes < 2 * L2_BYTES
    barrier()
    if not flush_l2:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(args.steps):
                if graph is not None:
                    graph.replay()
                else:
                    step()
            e1.record(stream)
        stream.synchronize()
        ms_total = e0.elapsed_time(e1)
    else:
        flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        with torch.cuda.stream(stream):
            for a, b_ in pairs:
                flush_buf.fill_(1)
                a.record(stream)
                if graph is not None:
                    graph.replay()
                else:
                    step()
                b_.record(stream)
        stream.synchronize()
        ms_total = sum(a.elapsed_time(b_) for a, b_ in pairs)
        del flush_buf
    barrier()
    launches = launches_per_step * args.steps
    ms_step = max_over_ranks(ms_total, dist, dev) / args.steps
    assert B.sdwino_last_device_status(stream) == B.OK, "a device-side wait timed out"

    value = aggregate_value(flops_step, world, ms_step)

    # ---- end to end: host buffers in, host buffers out, through sdwino_conv3x3_host ----
    e2e_steps = max(3, min(args.steps, 30))

    def e2e_step():
        for t, (x, w, b, y_h), (_, wT, _, _), wsl in zip(tiles, host, devt, ws_e2e):
            B.sdwino_conv3x3_host(x, wT, b, y_h, t, wsl, stream=stream, wait=False)
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
    h2d = sum(x.numel() * 2 + b.numel() * 2 for (x, w, b, y) in host)
    d2h = sum(y.numel() * 2 for (x, w, b, y) in host)
    # what came back through the host path is what the device-resident step computed (same kernels: same bits)
    e2e_matches = args.epilogue != "none" or io32 or all(torch.equal(y_h, yd.cpu()) for (_, _, _, y_h), (_, _, _, yd) in zip(host, devt))
    assert e2e_matches, "the host path returned something else than the device path"

    # ---- per-kernel and per-layer times: a second timed pass with CUDA events around every launch (recorded
    #      by the library on the launch stream).  The sweeps run back to back without host syncs, so the device
    #      stays busy and an event pair measures its kernel; the event gaps keep this pass out of `value`. ----
    B.sdwino_profile_enable(True)
    records_per_layer = []
    with torch.cuda.stream(stream):
        for li in range(len(layers)):     # learn how many launches each layer makes
            run_layer(li, stream)
            records_per_layer.append(len(B.sdwino_profile_records()))
    prof_steps = max(3, min(args.steps, 20))
    per_layer = [dict(input_transform=0.0, wino_gemm=0.0, output_transform=0.0, fused=0.0, launches=0)
                 for _ in layers]

    def account(recs):
        assert len(recs) == sum(records_per_layer) and all(ms >= 0 for _, ms in recs)
        it = iter(recs)
        for li, nrec in enumerate(records_per_layer):
            for _ in range(nrec):
                kind, ms = next(it)
                per_layer[li][kind] += ms / prof_steps
                if kind == "wino_gemm":
                    per_layer[li]["launches"] += 1

    if graph is not None:
        # the event records become nodes of a second graph: replaying it keeps the device busy, so an event
        # pair measures its kernel and not the host's launch latency
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
    B.sdwino_profile_enable(False)
    clocks = sampler.stop()

    def gbs_safe(nbytes, ms):
        return nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0

    tpeak = peaks["bf16_tflops"]          # burst figure: each kernel is microseconds long and timed alone
    hpeak = peaks["hbm_gbs"]
    layer_rows = []
    gemm_flops = gemm_ms = gemm_u_bytes = 0.0
    in_ms = out_ms = 0.0
    in_bytes = out_bytes = 0.0
    fused_ms = 0.0
    for L, t, pl in zip(layers, tiles, per_layer):
        a2 = (t + 2) ** 2
        P = L.tiles(t)
        wino_flops = 2.0 * a2 * L.K * L.C * P
        u_bytes = B.sdwino_filter_bytes(L.K, L.C, t)
        xb, yb = io_bytes * L.N * L.C * L.H * L.W, io_bytes * L.N * L.K * L.H * L.W
        t_tensor = wino_flops / (tpeak * 1e12) * 1e6
        t_hbm = (xb + 2.0 * a2 * L.K * L.C + yb + 2 * L.K) / (hpeak * 1e9) * 1e6
        total_us = (pl["input_transform"] + pl["wino_gemm"] + pl["output_transform"] + pl["fused"]) * 1e3
        layer_rows.append({
            "layer": L.name, "tile": t, "us": round(total_us, 2),
            "us_input": round(pl["input_transform"] * 1e3, 2), "us_gemm": round(pl["wino_gemm"] * 1e3, 2),
            "us_output": round(pl["output_transform"] * 1e3, 2), "us_fused": round(pl["fused"] * 1e3, 2),
            "eq_tflops": round(L.direct_flops / (total_us * 1e-6) / 1e12, 1),
            "bound": "tensor" if t_tensor >= t_hbm else "hbm",
            "roof_us": round(max(t_tensor, t_hbm), 2),
            "frac_of_roof": round(max(t_tensor, t_hbm) / total_us, 3),
            "gemm_tensor_frac": (round(wino_flops / (pl["wino_gemm"] * 1e-3) / 1e12 / tpeak, 3)
                                 if pl["wino_gemm"] > 0 else None),
        })
        if pl["wino_gemm"] > 0:                  # layers on the fused few-channel kernel have no GEMM launch
            gemm_flops += wino_flops
            gemm_u_bytes += u_bytes
            gemm_ms += pl["wino_gemm"]
            in_ms += pl["input_transform"]
            out_ms += pl["output_transform"]
            in_bytes += xb + 2.0 * a2 * L.C * P      # read x, write V
            out_bytes += 2.0 * a2 * L.K * P + yb     # read M, write y
        fused_ms += pl["fused"]
    gemm_launches = sum(pl["launches"] for pl in per_layer) / prof_steps
    achieved = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0   # a subset of fused-kernel layers
    roofline = {
        "kernel": "wino_gemm_kernel", "bound": "tensor", "achieved": round(achieved, 1), "peak": tpeak,
        "unit": "TFLOP/s", "frac": round(achieved / tpeak, 4),
        "traffic": (GEMM_DRAM_BYTES_PER_LAUNCH_SD15.get(str(args.tile))
                    if (args.workload == WORKLOAD and not args.layers) else None),
        "traffic_unit": "bytes per launch (ncu dram read + write, L2 left warm)",
        "peak_source": f"{peak_kind} (cuBLAS bf16 burst; fp16 has the same nominal rate)",
        "launches_per_step": gemm_launches,
        "avg_launch_us": round(gemm_ms * 1e3 / gemm_launches, 2) if gemm_launches else None,
        "algorithmic_flops_per_step": gemm_flops,
        "share_of_step": round(gemm_ms / max(gemm_ms + in_ms + out_ms + fused_ms, 1e-12), 3),
    }
    def gbs(nbytes, ms):
        return nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0

    # the same launches against the other roof: the GEMM is the kernel that streams the transformed weights, and
    # on the small-image layers that stream, not the tensor pipe, is what bounds it
    roofline["weight_stream_view"] = {
        "bound": "hbm", "algorithmic_bytes_per_step": gemm_u_bytes,
        "achieved": round(gbs_safe(gemm_u_bytes, gemm_ms), 1), "peak": hpeak, "unit": "GB/s",
        "frac": round(gbs_safe(gemm_u_bytes, gemm_ms) / hpeak, 4)}
    # the whole step against the per-layer roofline max(tensor time, mandatory HBM bytes / bandwidth), both at
    # the measured peaks: what an ideal implementation of each layer would need, summed over the sweep
    roof_us_sum = sum(r["roof_us"] for r in layer_rows)
    roofline["step_vs_layer_rooflines"] = {
        "sum_of_layer_rooflines_us": round(roof_us_sum, 1), "step_us": round(ms_step * 1e3, 1),
        "frac": round(roof_us_sum / (ms_step * 1e3), 3),
        "hbm_bound_layers": sum(1 for r in layer_rows if r["bound"] == "hbm"), "layers": len(layer_rows)}

    transforms = {
        "input_transform": {"gbs": round(gbs(in_bytes, in_ms), 1), "frac_of_hbm_peak":
                            round(gbs(in_bytes, in_ms) / hpeak, 3), "ms_per_step": round(in_ms, 4)},
        "output_transform": {"gbs": round(gbs(out_bytes, out_ms), 1), "frac_of_hbm_peak":
                             round(gbs(out_bytes, out_ms) / hpeak, 3), "ms_per_step": round(out_ms, 4)},
        "filter_transform_once_per_weight": {"ms": round(ft_ms, 4), "gbs": round(ft_bytes / (ft_ms * 1e-3) / 1e9, 1),
                                             "frac_of_hbm_peak": round(ft_bytes / (ft_ms * 1e-3) / 1e9 / hpeak, 3)},
        "hbm_peak_gbs": hpeak, "peak_source": peak_kind,
    }

    # ---- cuDNN yardstick (not the target) ----
    cudnn = None
    if rank == 0 and not args.no_yardstick:
        try:
            import torch.nn.functional as F
            torch.backends.cudnn.benchmark = True
            wd = [h[1].to(dev) for h in host]
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
                     "what": "torch.nn.functional.conv2d fp16 NCHW, cudnn.benchmark=True (yardstick only)"}
        except Exception as e:  # pragma: no cover
            cudnn = {"error": repr(e)}

    # ---- oracle on the host cores (reported baseline) ----
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        inputs = [(x.numpy(), w.numpy(), b.numpy()) for (x, w, b, _) in host]
        nch = 160   # about 10-15 s of host work on the default workload
        sec, fl = oracle_sample(layers, inputs, nch)
        cpu_baseline = {"value": fl / sec / 1e12, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                        "sample": f"fp64 direct conv of min(K, {nch}) seeded output channels of each of the {len(layers)} "
                                  f"layers ({fl / 1e9:.1f} GFLOP in {sec:.1f} s)"}

    if rank == 0:
        line = {
            "metric": metric_name(args.workload), "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32 in/out, f16 operands, f32 accumulate" if io32 else "f16",
            "data": "synthetic",
            "config": {"workload": args.workload, "io": args.io, "layers": len(layers), "layer_subset": args.layers or "all",
                       "batch": layers[0].N, "tile": args.tile,
                       "tile_per_layer": tiles,
                       "algorithm": ("Winograd F(2x2,3x3) or F(4x4,3x3) per layer (sdwino_choose_tile)"
                                     if args.tile == "auto" else f"Winograd F({args.tile}x{args.tile},3x3)") +
                                    (", fp32 x / w / bias / y, fp16 transformed operands, fp32 accumulate (e2e runs the fp16 interface)"
                                     if io32 else ", fp16 storage, fp32 accumulate"),
                       "parallelism": f"replicas x{world} (no exchange step)",
                       "launch": "direct" if args.no_graph else "CUDA graph of one step, replayed",
                       "l2": ((f"flushed before every timed step (256 MB written): one step touches only {step_bytes / 1e6:.0f} MB")
                              if flush_l2 else
                              (f"no flush: one step touches {step_bytes / 1e6:.0f} MB of distinct inputs, transformed weights "
                               f"and outputs ({step_bytes / L2_BYTES:.1f}x the 126 MB L2), so a layer starts with its operands "
                               "cold")),
                       "filter_transform": "once per weight, before the timed region (reported separately)",
                       "epilogue": {"none": "bias", "residual": "bias + residual, fused, on the layers with more than 8 input and output channels (e2e runs the plain convolution)",
                                    "residual_silu": "SiLU(bias + residual), fused, on the layers with more than 8 input and output channels (e2e runs the plain convolution)"}[args.epilogue]},
            "e2e": {"value": round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "matches_device_path": bool(e2e_matches), "api": "sdwino_conv3x3_host_async per layer (pinned host x, bias, y; " +
                           ("a workspace per layer: uploads and downloads overlap the neighbouring layers" if per_layer_ws
                            else "one shared workspace: the copies of differently sized layers are ordered one after the other") +
                           "), one join + stream synchronisation per step"},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roofline,
            "transforms": transforms,
            "cpu_baseline": cpu_baseline,
            "cudnn_yardstick": cudnn,
            "layers": layer_rows,
            "paper_context": PAPER_CONTEXT,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD, choices=["single", "sd15_unet", "sd_vae_512", "sd21_unet", "sdxl_1024"])
    ap.add_argument("--layers", default="", help="comma-separated layer indices of the workload (default: all)")
    ap.add_argument("--tile", default=TILE, choices=["auto", "2", "4"])
    ap.add_argument("--io", default="f16", choices=["f16", "f32"],
                    help="element type of x, w, bias and y in the timed step: f32 runs sdwino_conv3x3_f32 (fp16 operands, "
                         "fp32 accumulation); the end-to-end arm stays fp16")
    ap.add_argument("--epilogue", default="none", choices=["none", "residual", "residual_silu"],
                    help="fuse y = act(conv + bias + residual) into the output transform of the timed step (sdwino_conv3x3_ex)")
    ap.add_argument("--no-graph", action="store_true", help="launch every step directly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-yardstick", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
