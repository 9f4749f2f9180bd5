#!/usr/bin/env python
"""Benchmark of the cached causal Conv3D hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one ccv3d_forward call (channels-last staging + cache update and the tcgen05 implicit GEMM; in the
default schedule one kernel does all three, its stager warps running a band ahead of its MMA tiles, after a small
staging launch for the first two bands of rows) on one synthetic decoder-shaped layer.  The default workload is the 192->192, T=4 + 2-frame cache,
352x640, 3x3x3 BF16 layer (the large-spatial configuration the >= 60 %-of-tensor-peak target is quoted on);
inputs are seeded, synthetic, resident in HBM when the timed region starts, and larger than L2 (no flush
needed).  One JSON line on stdout.

--impl reference times the CPU oracle (the plain FP64 definition) on a bounded spatial crop of the same
workload on the host's cores.  With N > 1 every rank runs an independent replica (no collective on the data
path): weak scaling.  Started without torchrun, `--gpus N` with N > 1 starts its own N ranks (one per GPU).

Besides the K timed steps the line carries a `sustained` leg (at least two seconds of back-to-back calls
whatever --steps says, per-call times from events, clocks sampled throughout), the other benchmark
configurations each with its own roofline, clock record and CPU-oracle baseline, cold-L2 figures for the
HBM-bound kernels, and the first-chunk (NULL cache) form with its useful FLOP count.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import synth_inputs as si  # noqa: E402

METRIC = "causal Conv3D BF16 TFLOP/s"
DEFAULT_WORKLOAD = "cfg3_bf16_192"

NOMINAL_BF16_TFLOPS = 2250.0     # B200 dense BF16, the datasheet figure the 60 % target is stated on

# DRAM bytes (read + write) of one launch of a kernel, from ncu captures of quarter-size cases scaled by the pixel
# count (activation reads and output writes grow with it; the weights are 2 MB).  Keyed by workload AND by the kernel
# variant that ran, so that a changed schedule cannot inherit another variant's figure (it reports null instead).
#   cooperative = cooperative staging on CTA pairs (staging + cache update + convolution in one launch, after a staging
#                 kernel for the first two bands of rows):
#                 profiles/conv3d_tcgen05_coop_192ch_176x320.md, 229.8 MB read + 192.4 MB written at 176x320
#   ring        = the same kernel on frame rings: profiles/conv3d_tcgen05_ring_192ch_176x320.md, 132.0 MB read +
#                 53.6 MB written during the kernel (the rest of the 86.5 MB output still in L2 when it ends)
#   two_kernels = the convolution kernel of the two-kernel schedule: profiles/conv3d_tcgen05_192ch_176x320.md
TRAFFIC_BYTES_PER_LAUNCH = {
    ("cfg3_bf16_192", "cooperative"): 4 * (229.8e6 + 192.4e6),
    ("cfg3_bf16_192", "ring"): 4 * (132.0e6 + 53.6e6),
    ("cfg3_bf16_192", "two_kernels"): 4 * (133.2e6 + 53.0e6),
    ("cfg4a_bf16_96", "cooperative"): 4 * (471.2e6 + 452.1e6),   # profiles/conv3d_tcgen05_coop_96out_352x640.md
    ("cfg4a_bf16_96", "ring"): 4 * (260.4e6 + 143.4e6),         # profiles/conv3d_tcgen05_96out_352x640.md
    ("cfg4b_bf16_192_96", "cooperative"): 4 * (1044.0e6 + 783.0e6),
    ("cfg4b_bf16_192_96", "ring"): 4 * (524.3e6 + 155.5e6),
    # profiles/conv1x1_tcgen05_192to96_352x640.md: x read once, 137 of the 173 MB of output written during the kernel
    ("cfg4c_bf16_pw_192_96", "pointwise"): 4 * (346.1e6 + 137.0e6),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(tflops=float(p["bf16_tflops"]), tflops_sustained=float(p.get("bf16_tflops_sustained", 0.0)),
                    hbm_gbs=float(p["hbm_gbs"]), source="measured")
    return dict(tflops=1590.0, tflops_sustained=1400.0, hbm_gbs=6650.0, source="fallback")


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
                 getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
                 getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                 getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                 getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown"}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2.0)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": int(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def cfg_of(name):
    cfg = dict(si.CONFIGS[name])
    dims = dict(N=cfg["N"], Cin=cfg["Cin"], Cout=cfg["Cout"], T=cfg["T"], H=cfg["H"], W=cfg["W"], k=cfg["k"])
    return cfg, dims


# ---------------------------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(name, target_s=12.0):
    """Picks a spatial crop (all channels, all frames, the cache included) of the workload on which one pass of
    the oracle, as it stands, takes about target_s seconds on this host: a small calibration pass (run twice, the
    second timed, so that thread start-up is not counted) gives the rate."""
    import oracle
    cfg, d = cfg_of(name)
    crop = dict(cfg, H=min(d["H"], 32), W=min(d["W"], 32))
    c = si.conv_case(**crop)
    oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    t0 = time.perf_counter()
    oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    t_small = time.perf_counter() - t0
    px_small = crop["H"] * crop["W"]
    px = target_s / max(t_small, 1e-6) * px_small        # pixels per frame the oracle covers in target_s seconds
    W = int(min(d["W"], 80))
    H = int(min(d["H"], max(8, px // W)))
    if H == d["H"]:
        W = int(min(d["W"], max(W, px // H)))
    return dict(cfg, H=H, W=W)


def run_oracle_once(crop):
    import oracle
    c = si.conv_case(**crop)
    t0 = time.perf_counter()
    oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    dt = time.perf_counter() - t0
    fl = si.conv_flops(crop["N"], crop["Cin"], crop["Cout"], crop["T"], crop["H"], crop["W"], crop["k"])
    return dt, fl


def cpu_baseline(name, target_s=12.0):
    import oracle
    crop = oracle_sample(name, target_s)
    dt, fl = run_oracle_once(crop)
    return {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"one pass over a {crop['H']}x{crop['W']} spatial crop (all {crop['Cin']}->{crop['Cout']} "
                      f"channels, T={crop['T']} + {crop['k'][0] - 1}-frame cache) of {name}: {dt:.2f} s"}


def main_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    name = args.workload
    cfg, d = cfg_of(name)
    crop = oracle_sample(name, target_s=6.0)
    for _ in range(min(args.warmup, 1)):
        run_oracle_once(crop)
    steps = max(1, min(args.steps, 5))
    t_tot, fl_tot = 0.0, 0.0
    for _ in range(steps):
        dt, fl = run_oracle_once(crop)
        t_tot += dt
        fl_tot += fl
    val = fl_tot / t_tot / 1e12
    sample = (f"each step = the oracle over a {crop['H']}x{crop['W']} spatial crop (all channels and frames) "
              f"of {name}; {steps} steps timed")
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * t_tot / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": name, **{k: (list(v) if isinstance(v, tuple) else v) for k, v in d.items()},
                       "sample": sample},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------------------------- multi-rank plumbing
def init_ranks(backend, device=None):
    """(world, rank, local_rank, dist or None) from the torchrun environment; one process per GPU, replicas only."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group(backend)
    return world, rank, local, dist


def max_over_ranks(ms_local, dist, device=None):
    """The slowest rank's time: the job is done when the last replica is."""
    if dist is None:
        return float(ms_local)
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def weak_scaling_value(world, flops_per_step, ms_per_step):
    """Whole-job TFLOP/s of `world` independent replicas that each run the full workload."""
    return world * flops_per_step / (ms_per_step * 1e-3) / 1e12


def main_selftest_dist(args):
    """Host-side check of the multi-rank path without GPUs (gloo): every rank pretends to have measured a
    rank-dependent step time; rank 0 prints the aggregated line.  Used by tests/test_bench_ranks.py."""
    world, rank, local, dist = init_ranks("gloo")
    if dist is not None:
        dist.barrier()
    cfg, d = cfg_of(args.workload)
    flops = si.conv_flops(**d)
    ms_local = 1.0 + 0.25 * rank                     # the last rank is the slowest
    ms = max_over_ranks(ms_local * args.steps, dist) / args.steps
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": weak_scaling_value(world, flops, ms), "unit": "TFLOP/s",
                          "n_gpus": world, "steps": args.steps, "ms_per_step": ms, "scaling": "weak",
                          "selftest": "gloo ranks with fabricated step times"}))
    return 0


# ---------------------------------------------------------------------------------------------- CUDA leg
def chain_leg(dev):
    """Streamed synthetic decoder chain (configuration 5): 21 one-latent-frame chunks through six cached 3x3x3
    convolutions (384 ch @ 44x80 T=1, 192 ch @ 88x160 T=4, 96 ch @ 176x320 T=4), two 1x1x1 transitions, residual
    adds and upsampling, caches carried per layer.  Returns ms per output frame (84 frames)."""
    import math
    import torch
    from paper_2609_31938_b200.chain import DecoderChain, LAYERS, ResidentDecoderChain
    shapes = {"A1": (384, 384, 3), "A2": (384, 384, 3), "PA": (192, 384, 1), "B1": (192, 192, 3), "B2": (192, 192, 3),
              "PB": (96, 192, 1), "C1": (96, 96, 3), "C2": (96, 96, 3)}
    up = lambda a: torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
    w, b = {}, {}
    for i, n in enumerate(LAYERS):
        co, ci, k = shapes[n]
        w[n] = up(si.normal((co, ci, k, k, k), 1.0 / math.sqrt(ci * k ** 3), si.BF16, 0, si.TID_W + 16 * (i + 1)))
        b[n] = up(si.normal((co,), math.sqrt(0.1), si.BF16, 0, si.TID_B + 16 * (i + 1)))
    u = up(si.normal((1, 384, 21, 44, 80), 1.0, si.BF16, 0, si.TID_X))
    chunks = [u[:, :, i:i + 1].contiguous() for i in range(21)]
    flops = 21 * (2 * si.conv_flops(1, 384, 384, 1, 44, 80, (3, 3, 3)) + si.conv_flops(1, 384, 192, 1, 44, 80, (1, 1, 1))
                  + 2 * si.conv_flops(1, 192, 192, 4, 88, 160, (3, 3, 3)) + si.conv_flops(1, 192, 96, 4, 88, 160, (1, 1, 1))
                  + 2 * si.conv_flops(1, 96, 96, 4, 176, 320, (3, 3, 3)))

    def run(ch):
        for c in chunks[:3]:
            ch.step(c)
        ch.reset()
        torch.cuda.synchronize()
        base = sum(l.counters()["kernel_launches"] for l in ch.layers.values())
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for c in chunks:
            ch.step(c)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        launches = sum(l.counters()["kernel_launches"] for l in ch.layers.values()) - base
        ch.close()
        return {"ms_total": ms, "ms_per_chunk": ms / 21, "ms_per_output_frame": ms / 84,
                "tflops": flops / (ms * 1e-3) / 1e12, "conv_kernel_launches": int(launches)}

    # activations resident in frame rings between the layers (the default way to run a chain), and the same chain
    # returning to NCTHW after every layer (cache tensors, separate residual adds)
    res = run(ResidentDecoderChain(w, b))
    res["workload"] = "cfg5 streamed decoder chain, 21 chunks -> 84 frames of 96x176x320"
    res["activations"] = "resident frame rings between layers, residual adds in the epilogues"
    res["ncthw_between_layers"] = run(DecoderChain(w, b))
    return res


class L2Flusher:
    """Evicts the L2 between timed calls by writing a buffer twice its size (cold-L2 figures of the HBM-bound kernels)."""

    def __init__(self, dev, nbytes=320 << 20):
        import torch
        self.buf = torch.empty(nbytes, dtype=torch.uint8, device=dev)

    def __call__(self):
        self.buf.add_(1)


def timed_calls(fn, iters, warmup=3, flush=None):
    """Per-call device times in ms (CUDA events on the current stream).  Without `flush` the calls run back to back
    and call i is the time between the events before it and after it (launch gaps included); with `flush` every
    call is timed on its own after the flush."""
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * iters if flush else iters + 1)]
    if flush:
        for i in range(iters):
            flush()
            ev[2 * i].record()
            fn()
            ev[2 * i + 1].record()
        torch.cuda.synchronize()
        return [ev[2 * i].elapsed_time(ev[2 * i + 1]) for i in range(iters)]
    ev[0].record()
    for i in range(iters):
        fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    return [ev[i].elapsed_time(ev[i + 1]) for i in range(iters)]


def graph_replay_ms(fn, calls=20, replays=10):
    """Per-call device time of `fn` captured `calls` times in a CUDA graph and replayed: what a launch-bound layer
    costs when the host's enqueue time is out of the way.  `fn` must allocate nothing (lent workspace, rings)."""
    import torch
    fn()
    torch.cuda.synchronize()
    g, st = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(st):
        g.capture_begin()
        for _ in range(calls):
            fn()
        g.capture_end()
    torch.cuda.synchronize()
    ms = timed_calls(g.replay, replays, warmup=2)
    return float(np.median(ms)) / calls


def stats(ms_list):
    a = np.asarray(ms_list, dtype=np.float64)
    return {"ms_mean": float(a.mean()), "ms_median": float(np.median(a)), "ms_min": float(a.min()), "samples": int(a.size)}


def roofline_of(flops, abytes, ms, peaks):
    """The slower of FLOPs at the measured tensor peak and algorithmic bytes at the measured HBM bandwidth, against
    the measured time; `bound` names which of the two it is."""
    t_tensor = flops / (peaks["tflops"] * 1e12) * 1e3
    t_hbm = abytes / (peaks["hbm_gbs"] * 1e9) * 1e3
    if t_tensor >= t_hbm:
        ach = flops / (ms * 1e-3) / 1e12
        return {"bound": "tensor", "achieved": ach, "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": ach / peaks["tflops"],
                "frac_of_nominal_2250": ach / NOMINAL_BF16_TFLOPS, "peak_source": f"{peaks['source']} (burst cuBLAS bf16)"}
    ach = abytes / (ms * 1e6)
    return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
            "peak_source": f"{peaks['source']} (device copy)"}


def kernel_variant(ccv, layer, fn):
    """Which kernels served `fn` (two profiled calls): the 1x1x1 streaming kernel, one launch that stages and
    convolves, or a staging kernel followed by the convolution kernel."""
    import torch
    p0 = layer.counters()["pointwise"]
    ccv.ccv3d_profile_enable(layer.h, True)
    fn()
    fn()
    torch.cuda.synchronize()
    _, stage_ms, _, ncalls = ccv.ccv3d_profile_read(layer.h)
    ccv.ccv3d_profile_enable(layer.h, False)
    if layer.counters()["pointwise"] > p0:
        return "pointwise"
    return "cooperative" if stage_ms / max(ncalls, 1) < 0.02 else "two_kernels"


def useful_tap_fraction(T, kt, cache_frames):
    """Share of the (output frame, temporal tap) pairs whose source frame exists (Eq. (4)): with no history the
    taps that would read it are skipped - 1/3, 3/6, 9/12 of them remain at T = 1, 2, 4 with kt = 3."""
    p_l = (kt - 1) - cache_frames
    return sum(1 for t in range(T) for k in range(kt) if t + k - p_l >= 0) / float(T * kt)


def other_configs_leg(dev, local):
    """The remaining benchmark configurations, each in a burst of 20 calls after 3 warm-ups, through ccv3d_forward
    (NCTHW boundary) and, for the cached layers, through ccv3d_forward_ring; the first-chunk (NULL cache) form of
    the headline layer; the staging + cache-update kernel alone; cold-L2 repeats of the HBM-bound ones.  Inputs come
    from the seeded host generator (the tensors the parity tests use); every entry carries its own roofline, clock
    record and CPU-oracle baseline (a bounded spatial crop, stated)."""
    import torch
    import paper_2609_31938_b200 as ccv
    peaks = measured_peaks()
    out = {}
    flush = L2Flusher(dev)

    def up(a):
        if a is None:
            return None
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
        return torch.from_numpy(a).to(dev)

    def clocked(fn, iters=20, flush_fn=None):
        smp = ClockSampler(local, period_s=0.002)
        smp.start()
        ms = timed_calls(fn, iters, flush=flush_fn)
        smp.stop()
        return ms, smp.summary()

    # the HBM-bound 1x1x1 layer first, after a pause: right after a long tensor-bound run the part is still in its
    # power-capped state and the same kernel measures 20 % slower (the clock record of the entry shows which state
    # it ran in)
    time.sleep(1.0)
    for name in ("cfg4c_bf16_pw_192_96", "cfg2_bf16_384", "cfg4a_bf16_96", "cfg4b_bf16_192_96", "cfg1_f32_16"):
        cfg, d = cfg_of(name)
        N, Cin, Cout, T, H, W, k = d["N"], d["Cin"], d["Cout"], d["T"], d["H"], d["W"], d["k"]
        f32 = cfg["dtype"] == si.F32
        c = si.conv_case(**cfg)
        x, cache = up(c["x"]), up(c["cache"])
        layer = ccv.CausalConv3d(up(c["w"]), up(c["b"]))
        y = torch.empty((N, Cout, T, H, W), dtype=torch.float32 if f32 else torch.bfloat16, device=dev)
        nc = torch.empty_like(cache) if cache is not None else None
        es = 4 if f32 else 2
        flops, abytes = si.conv_flops(**d), si.conv_bytes(**d, elem=es, out_elem=es)
        ms, clk = clocked(lambda: layer(x, cache, out=y, new_cache=nc))
        st = stats(ms)
        row = {"ms_per_call": st["ms_median"], **st, "tflops": flops / (st["ms_median"] * 1e-3) / 1e12,
               "gbs": abytes / (st["ms_median"] * 1e6), "clocks": clk, "data": "seeded synthetic (host generator)"}
        if f32:
            row["dtype"] = "f32"
            row["note"] = "3xTF32 route (staging + convolution, two short launches); latency-bound: no roofline claim"
        else:
            row["roofline"] = roofline_of(flops, abytes, st["ms_median"], peaks)
            variant = kernel_variant(ccv, layer, lambda: layer(x, cache, out=y, new_cache=nc))
            row["roofline"]["kernel_variant"] = variant
            row["roofline"]["traffic"] = TRAFFIC_BYTES_PER_LAUNCH.get((name, variant))
        if name == "cfg4c_bf16_pw_192_96":
            cms, cclk = clocked(lambda: layer(x, cache, out=y, new_cache=nc), flush_fn=flush)
            cst = stats(cms)
            row["cold_l2"] = {**cst, "gbs": abytes / (cst["ms_median"] * 1e6),
                              "frac_of_measured_hbm": abytes / (cst["ms_median"] * 1e6) / peaks["hbm_gbs"], "clocks": cclk,
                              "note": "every call timed on its own after a 320 MB write that evicts the L2"}
        if cache is not None and not f32:
            F = T + k[0] - 1
            rin, rout = ccv.FrameRing(N, Cin, F, H, W), ccv.FrameRing(N, Cout, T, H, W)
            rin.load(0, cache)
            rin.load(k[0] - 1, x)
            slot = [k[0] - 1]

            def ring_step():
                layer.forward_ring(rin, slot[0], k[0] - 1, T, out_ring=rout)
                slot[0] = (slot[0] + T) % F

            rms, rclk = clocked(ring_step)
            rst = stats(rms)
            r_bytes = 2 * N * H * W * T * (Cin + Cout) + c["w"].nbytes
            row["resident"] = {**rst, "tflops": flops / (rst["ms_median"] * 1e-3) / 1e12, "clocks": rclk,
                               "roofline": roofline_of(flops, r_bytes, rst["ms_median"], peaks)}
            row["resident"]["roofline"]["traffic"] = TRAFFIC_BYTES_PER_LAUNCH.get((name, "ring"))
            row["resident_ms_per_call"] = rst["ms_median"]
            row["resident_tflops"] = row["resident"]["tflops"]
            del rin, rout
        assert layer.device_status()[0] == ccv.OK
        layer.close()
        if name in ("cfg2_bf16_384", "cfg1_f32_16"):
            # launch-bound layers: the same calls captured in a CUDA graph (the staging copy in a lent workspace, so
            # that nothing is allocated inside the capture)
            lay2 = ccv.CausalConv3d(up(c["w"]), up(c["b"]))
            _, need = ccv.ccv3d_workspace_bytes(lay2.h, N, T, H, W)
            wsb = torch.empty(max(int(need), 256) + 256, dtype=torch.uint8, device=dev)
            if need:
                assert ccv.ccv3d_set_workspace(lay2.h, (wsb.data_ptr() + 255) // 256 * 256, int(need)) == ccv.OK
            gms = graph_replay_ms(lambda: lay2(x, cache, out=y, new_cache=nc))
            row["graph_replay"] = {"ms_per_call": gms, "tflops": flops / (gms * 1e-3) / 1e12,
                                   "note": "20 calls captured in a CUDA graph, replayed; lent workspace"}
            if not f32:
                row["graph_replay"]["frac_of_measured_bf16_peak"] = flops / (gms * 1e-3) / 1e12 / peaks["tflops"]
                F = T + k[0] - 1
                rin, rout = ccv.FrameRing(N, Cin, F, H, W), ccv.FrameRing(N, Cout, T, H, W)
                rin.load(0, cache)
                rin.load(k[0] - 1, x)
                rg = graph_replay_ms(lambda: lay2.forward_ring(rin, k[0] - 1, k[0] - 1, T, out_ring=rout))
                row["graph_replay"]["resident_ms_per_call"] = rg
                row["graph_replay"]["resident_frac_of_measured_bf16_peak"] = flops / (rg * 1e-3) / 1e12 / peaks["tflops"]
                del rin, rout
            assert lay2.device_status()[0] == ccv.OK
            lay2.close()
            del wsb
        if not f32:
            row["cpu_baseline"] = cpu_baseline(name, target_s=3.0)
        out[name] = row
        del x, cache, y, nc, c
        torch.cuda.empty_cache()

    # ---- the paper's wider contract at speed (Eq. (2) passes the layer's stride and dilation to every tap): a
    # downsampling layer at two widths (spatial stride 2: phase-decomposed staging inside the kernel on CTA pairs) and a
    # dilated one (straight-line taps two pixels apart)
    for label, (Cin, Cout, T, H, W), stride, dil in (
            ("general_96to192_stride2_704x1280", (96, 192, 4, 704, 1280), (1, 2, 2), (1, 1, 1)),
            ("general_192to384_stride2_352x640", (192, 384, 4, 352, 640), (1, 2, 2), (1, 1, 1)),
            ("general_192_dilation2_352x640", (192, 192, 4, 352, 640), (1, 1, 1), (1, 2, 2))):
        c = si.conv_case(1, Cin, Cout, T, H, W, dtype=si.BF16, seed=0)
        x, cache = up(c["x"]), up(c["cache"])
        layer = ccv.CausalConv3d(up(c["w"]), up(c["b"]), stride=stride, dilation=dil)
        _, To, Ho, Wo, _ = ccv.ccv3d_out_dims(layer.h, T, H, W)
        y = torch.empty((1, Cout, To, Ho, Wo), dtype=torch.bfloat16, device=dev)
        nc = torch.empty_like(cache)
        ms, clk = clocked(lambda: layer(x, cache, out=y, new_cache=nc))
        st = stats(ms)
        flops = 2.0 * Cout * Cin * 27 * To * Ho * Wo
        abytes = c["x"].nbytes + 2 * c["cache"].nbytes + c["w"].nbytes + 2 * Cout * To * Ho * Wo
        out[label] = {"ms_per_call": st["ms_median"], **st, "tflops": flops / (st["ms_median"] * 1e-3) / 1e12, "clocks": clk,
                      "stride": list(stride), "dilation": list(dil), "out_hw": [Ho, Wo],
                      "roofline": roofline_of(flops, abytes, st["ms_median"], peaks),
                      "kernel_variant": kernel_variant(ccv, layer, lambda: layer(x, cache, out=y, new_cache=nc))}
        assert layer.device_status()[0] == ccv.OK
        layer.close()
        del x, cache, y, nc, c
        torch.cuda.empty_cache()

    # ---- a one-frame streaming call at the headline layer's size (T = 1 on a two-frame history: the short temporal
    # extents on large feature maps that the paper's profile concentrates on).  Through the NCTHW boundary the call
    # has to stage three frames to produce one; on frame rings the history is simply there.
    cfg, d = cfg_of(DEFAULT_WORKLOAD)
    c = si.conv_case(**{**cfg, "T": 1})
    x, cache = up(c["x"]), up(c["cache"])
    N, Cin, Cout, H, W, k = d["N"], d["Cin"], d["Cout"], d["H"], d["W"], d["k"]
    layer = ccv.CausalConv3d(up(c["w"]), up(c["b"]))
    y = torch.empty((N, Cout, 1, H, W), dtype=torch.bfloat16, device=dev)
    nc = torch.empty_like(cache)
    ms, clk = clocked(lambda: layer(x, cache, out=y, new_cache=nc))
    st = stats(ms)
    d1 = {**d, "T": 1}
    flops, abytes = si.conv_flops(**d1), si.conv_bytes(**d1)
    F = 1 + k[0] - 1
    rin, rout = ccv.FrameRing(N, Cin, F, H, W), ccv.FrameRing(N, Cout, 1, H, W)
    rin.load(0, cache)
    rin.load(k[0] - 1, x)
    slot = [k[0] - 1]

    def ring_step1():
        layer.forward_ring(rin, slot[0], k[0] - 1, 1, out_ring=rout)
        slot[0] = (slot[0] + 1) % F

    rms, rclk = clocked(ring_step1)
    rst = stats(rms)
    out[DEFAULT_WORKLOAD + "_one_frame"] = {
        **st, "ms_per_call": st["ms_median"], "tflops": flops / (st["ms_median"] * 1e-3) / 1e12, "clocks": clk,
        "roofline": roofline_of(flops, abytes, st["ms_median"], peaks),
        "kernel_variant": kernel_variant(ccv, layer, lambda: layer(x, cache, out=y, new_cache=nc)),
        "resident": {**rst, "tflops": flops / (rst["ms_median"] * 1e-3) / 1e12, "clocks": rclk,
                     "roofline": roofline_of(flops, 2 * N * H * W * (Cin + Cout) + c["w"].nbytes, rst["ms_median"], peaks)},
        "note": "T = 1 with a two-frame cache: three staged frames per output frame through ccv3d_forward, none on frame rings"}
    assert layer.device_status()[0] == ccv.OK
    layer.close()
    del x, cache, y, nc, c, rin, rout
    torch.cuda.empty_cache()

    # ---- the headline layer's first-chunk form (NULL cache: the taps of absent history are skipped) and its
    # staging + cache-update kernel alone (two-kernel schedule), warm and with a cold L2
    name = DEFAULT_WORKLOAD
    cfg, d = cfg_of(name)
    c = si.conv_case(**cfg)
    x, cache = up(c["x"]), up(c["cache"])
    y = torch.empty((d["N"], d["Cout"], d["T"], d["H"], d["W"]), dtype=torch.bfloat16, device=dev)
    nc = torch.empty_like(cache)
    layer = ccv.CausalConv3d(up(c["w"]), up(c["b"]))
    ms, clk = clocked(lambda: layer(x, None, out=y, new_cache=nc))
    st = stats(ms)
    flops = si.conv_flops(**d)
    useful = useful_tap_fraction(d["T"], d["k"][0], 0)
    out[name + "_null_cache"] = {
        **st, "ms_per_call": st["ms_median"], "tflops_conventional": flops / (st["ms_median"] * 1e-3) / 1e12,
        "useful_tap_fraction": useful, "tflops_useful": useful * flops / (st["ms_median"] * 1e-3) / 1e12, "clocks": clk,
        "roofline": roofline_of(useful * flops, si.conv_bytes(**d) - c["cache"].nbytes, st["ms_median"], peaks),
        "note": "first chunk: no cache is read, the new cache is still written; FLOPs counted with the skipped "
                "(frame, tap) pairs removed (9 of 12 remain at T = 4, kt = 3), and by the usual convention"}
    layer.close()
    two = ccv.CausalConv3d(up(c["w"]), up(c["b"]), flags=ccv.FLAG_TWO_KERNELS)
    stage_bytes = 2 * c["x"].nbytes + 2 * c["cache"].nbytes + c["cache"].nbytes   # read x, cache; write the copy, new cache
    k4 = {}
    for label, fl in (("warm", None), ("cold_l2", flush)):
        ccv.ccv3d_profile_enable(two.h, True)
        timed_calls(lambda: two(x, cache, out=y, new_cache=nc), 10, flush=fl)
        _, stage_ms, conv_ms, ncalls = ccv.ccv3d_profile_read(two.h)
        ccv.ccv3d_profile_enable(two.h, False)
        sms = stage_ms / max(ncalls, 1)
        k4[label] = {"ms": sms, "gbs": stage_bytes / (sms * 1e6), "frac_of_measured_hbm": stage_bytes / (sms * 1e6) / peaks["hbm_gbs"],
                     "conv_kernel_ms": conv_ms / max(ncalls, 1), "calls": int(ncalls)}
    k4["bytes"] = int(stage_bytes)
    k4["note"] = ("stage_frames_kernel of the two-kernel schedule (CCV3D_FLAG_TWO_KERNELS): reads x and the cache once, "
                  "writes the channels-last copy and the new cache; mean over the calls, events recorded by the library "
                  "between its kernels (with the flush the convolution kernel finds the copy in DRAM)")
    out[name + "_staging_and_cache_update"] = k4
    assert two.device_status()[0] == ccv.OK
    two.close()
    return out


def hsplit_leg(dev):
    """Per-rank work of the height-split headline layer on this one GPU: rank 1 at world sizes
    2, 4 and 8 packs its halo rows, assembles its slab and runs the layer on it (10 calls after 3 warm-ups).  The
    neighbour exchange itself needs more than one GPU and is not in these times; its size is reported."""
    import math
    import torch
    import paper_2609_31938_b200 as ccv
    from paper_2609_31938_b200.hsplit import HSplitCausalConv3d, HSplitRingConv3d
    name = "cfg3_bf16_192"
    d = {k: v for k, v in si.CONFIGS[name].items() if k not in ("dtype", "x_dist")}
    N, Cin, Cout, T, H, W, k = d["N"], d["Cin"], d["Cout"], d["T"], d["H"], d["W"], d["k"]
    # the seeded tensors of the headline workload; a rank's band, halo rows and slabs are row slices of them (one zero
    # row above and below the image stands for the layer's zero padding at the image edge)
    c = si.conv_case(**si.CONFIGS[name])
    up = lambda a: torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
    pad_rows = lambda t: torch.nn.functional.pad(t, (0, 0, 1, 1))
    xp, cp = pad_rows(up(c["x"])), pad_rows(up(c["cache"]))          # row r of the image is row r + 1 here
    w, b = up(c["w"]), up(c["b"])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    out = {"workload": name, "data": "seeded synthetic (row slices of the headline tensors)",
           "note": "rank 1 of the world (halo rows on both sides of its slab). NCTHW: pack + slab assembly + layer "
                   "on the slab; resident: the ring call on the slab + pack and unpack of the output's halo "
                   "rows. Neighbour exchange (NCCL send/recv) not included"}
    for world in (2, 4, 8):
        layer = HSplitCausalConv3d(w, b, H, min(1, world - 1), world, transport=None)
        p = layer.plan
        xb = xp[:, :, :, p.r0 + 1:p.r1 + 1].contiguous()
        cache = cp[:, :, :, p.r0 + 1 - p.top:p.r1 + 1 + p.bot].contiguous()
        halo_up = xp[:, :, :, p.r0 + 1 - p.top:p.r0 + 1].contiguous()
        halo_down = xp[:, :, :, p.r1 + 1:p.r1 + 1 + p.bot].contiguous()

        def rank_step():
            layer.pack(xb)
            return layer.conv(layer.assemble(xb, halo_up, halo_down), cache)

        for _ in range(3):
            rank_step()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(10):
            rank_step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 10
        flops = si.conv_flops(**d) * p.rows / H
        # the same rank on frame rings: the ring call on the slab, then pack + unpack of the output's halo rows
        rl = HSplitRingConv3d(w, b, H, min(1, world - 1), world, transport=None)
        F = T + k[0] - 1
        rin, rout = rl.ring(N, Cin, F, W), rl.ring(N, Cout, T, W)
        rin.load(0, cache)
        rin.load(k[0] - 1, xp[:, :, :, p.r0 + 1 - p.top:p.r1 + 1 + p.bot].contiguous())
        slot = [k[0] - 1]

        def ring_rank_step():
            rl.conv.forward_ring(rin, slot[0], k[0] - 1, T, out_ring=rout)
            to_up, to_down = rl.pack(rout, 0, T)
            rl.unpack(rout, 0, T, to_down if to_down is not None else to_up, to_up if to_up is not None else to_down)
            slot[0] = (slot[0] + T) % F

        for _ in range(3):
            ring_rank_step()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(10):
            ring_rank_step()
        e1.record()
        torch.cuda.synchronize()
        rms = e0.elapsed_time(e1) / 10
        out[f"world{world}"] = {"rows": p.rows, "slab_rows": p.slab_rows, "ms_per_rank_step": ms,
                                "tflops_per_rank": flops / (ms * 1e-3) / 1e12,
                                "resident_ms_per_rank_step": rms, "resident_tflops_per_rank": flops / (rms * 1e-3) / 1e12,
                                "halo_bytes_sent_per_step": int(2 * N * Cin * T * (p.top + p.bot) * W)}
        assert layer.conv.device_status()[0] == ccv.OK and rl.conv.device_status()[0] == ccv.OK
        layer.close()
        rl.close()
        del xb, cache, halo_up, halo_down, rin, rout
        torch.cuda.empty_cache()
    return out


def hsplit_exchange_leg(dev, dist, world, rank):
    """World >= 2 only: the headline layer split by image rows over the ranks, on frame rings, with the real
    neighbour exchange (NCCL send/recv into this GPU's own buffers; no kernel reads a peer's memory).  Per rank:
    ms of the ring call on its slab and of the exchange of the output's halo rows; the slowest rank counts."""
    import torch
    import paper_2609_31938_b200 as ccv
    from paper_2609_31938_b200.hsplit import HSplitRingConv3d
    cfg, d = cfg_of(DEFAULT_WORKLOAD)
    N, Cin, Cout, T, H, W, k = d["N"], d["Cin"], d["Cout"], d["T"], d["H"], d["W"], d["k"]
    c = si.conv_case(**dict(cfg, H=8, W=8))                 # seeded weights and bias of the layer
    up = lambda a: torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
    rl = HSplitRingConv3d(up(c["w"]), up(c["b"]), H, rank, world)
    F = T + k[0] - 1
    rin, rout = rl.ring(N, Cin, F, W), rl.ring(N, Cout, T, W)
    rin.buf.normal_()
    slot = [k[0] - 1]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    conv_ms, xch_ms = [], []
    for it in range(13):
        dist.barrier()
        ev[0].record()
        rl.conv.forward_ring(rin, slot[0], k[0] - 1, T, out_ring=rout)
        ev[1].record()
        rl.exchange(rout, 0, T)
        ev[2].record()
        torch.cuda.synchronize()
        slot[0] = (slot[0] + T) % F
        if it >= 3:
            conv_ms.append(ev[0].elapsed_time(ev[1]))
            xch_ms.append(ev[1].elapsed_time(ev[2]))
    t = torch.tensor([float(np.median(conv_ms)), float(np.median(xch_ms))], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    p = rl.plan
    ok = rl.conv.device_status()[0] == ccv.OK
    rl.close()
    return {"workload": DEFAULT_WORKLOAD, "world": world, "rows_per_rank": p.rows, "conv_ms_max_over_ranks": float(t[0]),
            "exchange_us_max_over_ranks": 1e3 * float(t[1]), "halo_bytes_sent_per_rank_step": int(2 * N * Cout * T * (p.top + p.bot) * W),
            "device_status_ok": bool(ok),
            "note": "HSplitRingConv3d with DistTransport: ring call on the slab, then pack + NCCL send/recv + unpack of "
                    "the output's halo rows; medians of 10 steps, the slowest rank"}


def main_ours(args):
    import torch
    import paper_2609_31938_b200 as ccv

    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    world, rank, local, dist = init_ranks("nccl", dev)

    name = args.workload
    cfg, d = cfg_of(name)
    c = si.conv_case(**cfg)
    kt = d["k"][0]

    def up(a):
        return None if a is None else torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

    x, cache = up(c["x"]), up(c["cache"])
    layer = ccv.CausalConv3d(up(c["w"]), up(c["b"]), flags=args.flags)
    out = torch.empty((d["N"], d["Cout"], d["T"], d["H"], d["W"]), dtype=torch.bfloat16, device=dev)
    nc = torch.empty_like(cache) if cache is not None else None
    stream = torch.cuda.current_stream()

    def step():
        layer(x, cache, out=out, new_cache=nc)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    assert layer.device_status()[0] == ccv.OK
    launches0 = layer.counters()["kernel_launches"]
    ccv.ccv3d_profile_enable(layer.h, True)

    # ---- the timed region: exactly K steps between two events, a barrier + synchronize on both sides; one more
    # event after every step gives the per-step times
    sampler = ClockSampler(local, period_s=0.002)
    sampler.start()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    evs[0].record(stream)
    for i in range(args.steps):
        step()
        evs[i + 1].record(stream)
    barrier()
    sampler.stop()
    ms_total = evs[0].elapsed_time(evs[args.steps])
    per_step = [evs[i].elapsed_time(evs[i + 1]) for i in range(args.steps)]
    clocks = sampler.summary()
    clocks["note"] = "NVML, sampled every 2 ms during the timed region" + (
        " (a short region: the `sustained` leg has the long record)" if clocks["samples"] < 20 else "")

    st, stage_ms, conv_ms, ncalls = ccv.ccv3d_profile_read(layer.h)
    ccv.ccv3d_profile_enable(layer.h, False)
    launches = layer.counters()["kernel_launches"] - launches0
    assert layer.device_status()[0] == ccv.OK

    ms_total = max_over_ranks(ms_total, dist, dev)

    flops = si.conv_flops(**d)
    abytes = si.conv_bytes(**d)
    ms_step = ms_total / args.steps
    value = weak_scaling_value(world, flops, ms_step)
    peaks = measured_peaks()

    # ---- sustained: at least two seconds of back-to-back steps whatever --steps says (the part settles under its
    # power cap within the first few hundred milliseconds), per-step times from events, clocks sampled throughout
    sus_sampler = ClockSampler(local, period_s=0.004)
    sus_ms = []
    barrier()
    sus_sampler.start()
    t_begin = time.perf_counter()
    while time.perf_counter() - t_begin < args.sustain_s or len(sus_ms) < 100:
        sus_ms += timed_calls(step, 200, warmup=0)
    sus_sampler.stop()
    barrier()
    assert layer.device_status()[0] == ccv.OK
    sus_clk = sus_sampler.summary()
    tail = np.asarray(sus_ms[len(sus_ms) // 4:])               # the first quarter is the ramp into the capped state
    sus_med = max_over_ranks(float(np.median(tail)), dist, dev)
    sustained = {"seconds": float(np.sum(sus_ms)) / 1e3, "samples": int(tail.size), "ms_per_step_median": sus_med,
                 "ms_per_step_min": float(tail.min()), "ms_per_step_mean": float(tail.mean()),
                 "tflops": world * flops / (sus_med * 1e-3) / 1e12,
                 "frac_of_sustained_peak": (flops / (sus_med * 1e-3) / 1e12) / peaks["tflops_sustained"] if peaks["tflops_sustained"] else None,
                 "frac_of_burst_peak": (flops / (sus_med * 1e-3) / 1e12) / peaks["tflops"],
                 "frac_of_nominal_2250": (flops / (sus_med * 1e-3) / 1e12) / NOMINAL_BF16_TFLOPS,
                 "sm_mhz_median": sus_clk["sm_mhz"], "clock_samples": sus_clk["samples"], "reasons": sus_clk["reasons"],
                 "ms_times_mhz": (sus_med * sus_clk["sm_mhz"]) if sus_clk["sm_mhz"] else None,
                 "note": "back-to-back ccv3d_forward calls; statistics over the last three quarters of the per-step "
                         "event times; the sustained peak is the measured seconds-long cuBLAS bf16 figure"}

    # ---- end to end through the host entry point: pinned host buffers, H2D and D2H inside the timed region
    e2e = None
    if rank == 0:
        hx = torch.from_numpy(c["x"].view(np.int16)).pin_memory()
        hc = torch.from_numpy(c["cache"].view(np.int16)).pin_memory() if c["cache"] is not None else None
        ho = torch.empty(out.shape, dtype=torch.int16).pin_memory()
        hn = torch.empty(hc.shape, dtype=torch.int16).pin_memory() if hc is not None else None
        e_steps = max(1, min(args.steps, 8))

        def host_step():
            s = ccv.ccv3d_forward_host(layer.h, hx.data_ptr(), None if hc is None else hc.data_ptr(), ho.data_ptr(),
                                       None if hn is None else hn.data_ptr(), d["N"], d["T"], d["H"], d["W"],
                                       stream.cuda_stream)
            assert s == ccv.OK, ccv.status_string(s)

        host_step()
        host_step()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(e_steps):
            host_step()
        torch.cuda.synchronize()
        e_ms = 1e3 * (time.perf_counter() - t0) / e_steps
        h2d = hx.numel() * 2 + (hc.numel() * 2 if hc is not None else 0)
        d2h = ho.numel() * 2 + (hn.numel() * 2 if hn is not None else 0)
        e2e = {"value": flops / (e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": e_ms, "steps": e_steps,
               "note": "ccv3d_forward_host: pinned host x, cache -> device, the layer, out, new_cache -> host; band of rows by "
                       "band, frame by frame on three streams (upload, compute on a frame ring, download overlap): bound by PCIe, whose two "
                       f"directions together moved {(h2d + d2h) / (e_ms * 1e6):.0f} GB/s here"}
        assert np.array_equal(ho.numpy().view(np.uint16), out.view(torch.int16).cpu().numpy().view(np.uint16))
        # the streaming form of the same call: the history stays in a frame ring on the device, so a step moves only
        # x up and out down (the steady state of a streamed decode; same arithmetic per step)
        def stream_step(reset=False):
            s = ccv.ccv3d_forward_host_stream(layer.h, hx.data_ptr(), ho.data_ptr(), reset, d["N"], d["T"], d["H"], d["W"],
                                              stream.cuda_stream)
            assert s == ccv.OK, ccv.status_string(s)

        stream_step(True)
        stream_step()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(e_steps):
            stream_step()
        torch.cuda.synchronize()
        s_ms = 1e3 * (time.perf_counter() - t0) / e_steps
        e2e["stream"] = {"value": flops / (s_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": s_ms,
                         "h2d_bytes_per_step": int(hx.numel() * 2), "d2h_bytes_per_step": int(ho.numel() * 2),
                         "note": "ccv3d_forward_host_stream: the temporal history stays on the device between calls; "
                                 "x up, out down"}
        del hx, hc, ho, hn

    hsplit_x = None
    if dist is not None and world >= 2 and not args.no_chain:
        try:
            hsplit_x = hsplit_exchange_leg(dev, dist, world, rank)
        except Exception as e:                                # a secondary leg must not take the line down
            hsplit_x = {"error": f"{type(e).__name__}: {e}"}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    conv_avg_ms = conv_ms / max(ncalls, 1)
    stage_avg_ms = stage_ms / max(ncalls, 1)
    variant = "cooperative" if stage_avg_ms < 0.02 else "two_kernels"
    achieved = flops / (conv_avg_ms * 1e-3) / 1e12 if conv_avg_ms > 0 else None
    roof_t_ms = 1e3 * max(flops / (peaks["tflops"] * 1e12), abytes / (peaks["hbm_gbs"] * 1e9))
    roofline = {"bound": "tensor", "kernel": "conv3d_tcgen05_kernel", "achieved": achieved, "peak": peaks["tflops"],
                "unit": "TFLOP/s", "frac": (achieved / peaks["tflops"]) if achieved else None,
                "frac_of_nominal_2250": (achieved / NOMINAL_BF16_TFLOPS) if achieved else None,
                "peak_source": f"{peaks['source']} (burst cuBLAS bf16: the timed region is a burst of {ms_total:.0f} ms)",
                "kernel_variant": variant, "traffic": TRAFFIC_BYTES_PER_LAUNCH.get((name, variant)),
                "kernel_ms": conv_avg_ms,
                "schedule": "cooperative: staging + cache update + convolution in one kernel (the first two bands of rows "
                            "through the staging kernel before it)" if variant == "cooperative" else
                            "two kernels: staging + cache update, then convolution",
                "staging_kernel_ms": stage_avg_ms if variant == "two_kernels" else None,
                "step_frac_of_roofline": roof_t_ms / ms_step}

    # ---- the same layer on resident activations (frame rings): history in place, no staging copy, no cache
    # update, output written channels-last for a following layer.  The streamed steady state: x advances by T
    # slots per call.  Reported beside the headline, which keeps the NCTHW boundary of ccv3d_forward.
    resident = None
    if world == 1 and kt > 1:
        F = d["T"] + kt - 1
        rin = ccv.FrameRing(d["N"], d["Cin"], F, d["H"], d["W"])
        rout = ccv.FrameRing(d["N"], d["Cout"], d["T"], d["H"], d["W"])
        rin.load(0, cache)
        rin.load(kt - 1, x)
        slot = [kt - 1]

        def ring_step():
            layer.forward_ring(rin, slot[0], kt - 1, d["T"], out_ring=rout)
            slot[0] = (slot[0] + d["T"]) % F

        time.sleep(0.5)
        rst = stats(timed_calls(ring_step, max(20, args.steps)))
        r_ms = rst["ms_median"]
        assert layer.device_status()[0] == ccv.OK
        r_bytes = 2 * d["N"] * d["H"] * d["W"] * d["T"] * (d["Cin"] + d["Cout"]) + c["w"].nbytes
        resident = {"value": flops / (r_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": r_ms, **rst,
                    "frac_of_measured_bf16_peak": flops / (r_ms * 1e-3) / 1e12 / peaks["tflops"],
                    "frac_of_nominal_2250": flops / (r_ms * 1e-3) / 1e12 / NOMINAL_BF16_TFLOPS,
                    "algorithmic_bytes_per_step": int(r_bytes), "gpu_launches_per_step": 1,
                    "traffic": TRAFFIC_BYTES_PER_LAUNCH.get((name, "ring")),
                    "note": "ccv3d_forward_ring: input and output in frame rings (channels-last blocks), temporal "
                            "history left in the ring by the previous call"}
        del rin, rout

    cpu = cpu_baseline(name) if world == 1 else None
    chain = chain_leg(dev) if (world == 1 and not args.no_chain) else None
    others = other_configs_leg(dev, local) if (world == 1 and not args.no_chain) else None
    hsplit = hsplit_leg(dev) if (world == 1 and not args.no_chain) else None
    a = np.asarray(per_step)
    line = {"metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "ms_per_step_median": float(np.median(a)),
            "ms_per_step_min": float(a.min()), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": name, **{k: (list(v) if isinstance(v, tuple) else v) for k, v in d.items()},
                       "cache_frames": kt - 1, "accumulate": "fp32", "l2": "inputs larger than L2 (x alone is "
                       f"{c['x'].nbytes / 1e6:.0f} MB); no flush", "parallelism": f"replicas x{world}",
                       "algorithmic_bytes_per_step": int(abytes), "flops_per_step": flops,
                       "pct_of_measured_bf16_peak": 100.0 * (value / world) / peaks["tflops"],
                       "pct_of_nominal_bf16_peak": 100.0 * (value / world) / NOMINAL_BF16_TFLOPS},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "sustained": sustained}
    if cpu is not None:
        line["cpu_baseline"] = cpu
    if resident is not None:
        line["resident"] = resident
    if chain is not None:
        line["decoder_chain"] = chain
    if others is not None:
        line["other_configs"] = others
    if hsplit is not None:
        line["height_split"] = hsplit
    if hsplit_x is not None:
        line["height_split_exchange"] = hsplit_x
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    layer.close()
    return 0


def spawn_ranks(n):
    """`--gpus N` without torchrun: start N ranks of this script (one per GPU) on 127.0.0.1 and wait for them.
    NCCL's start-up log is left on (stderr of the ranks) so that the number of ranks can be read off it."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-chain", action="store_true", help="skip the secondary legs (decoder chain, other configurations, height-split)")
    ap.add_argument("--sustain-s", type=float, default=2.0, help="seconds of back-to-back steps in the sustained leg")
    ap.add_argument("--selftest-dist", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--flags", type=int, default=0, help="CCV3D_FLAG_* bits for the layer (e.g. 8 = fused route without staging copy)")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(n for n in si.CONFIGS if "bf16" in n))
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args.gpus)
    if args.selftest_dist:
        return main_selftest_dist(args)
    if args.impl == "reference":
        return main_reference(args)
    return main_ours(args)


if __name__ == "__main__":
    sys.exit(main())
