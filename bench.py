#!/usr/bin/env python
"""Benchmark of the decode + fused-product hot path on synthetic layers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole hot path (stream w^c, XOR expand, patch, mask, rescale,
product) over one batch: ``sqnn_decode_matmul`` on the AlexNet-FC6-shaped layer
(4096 x 9216, 1 plane, M 100 x 10, 91 % pruned) at batch 1.  The metric is decoded
weights per second.  Inputs are resident in HBM for ``value``; ``e2e`` repeats the
measurement with host buffers and the copies inside the timed region.  L2 is flushed
between timed iterations: the K steps are timed as one CUDA-event interval over
K x (flush + step), and the same interval over K flushes alone is subtracted (one event
interval per step would be as coarse as the event timer's tick).  ``extra`` reports every
other configuration: the fused product on the four layer shapes at all their batch sizes
beside a dense bf16 product of the same layer and that layer's HBM floor, the decode-only
kernel on 2^30 weights at all 16 sweep points against the HBM roofline, the bf16-output
and checksum forms of the headline point, and a store-only kernel as the write ceiling.
``--impl reference`` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decoded_weights_per_s_fused_decode_gemv"
UNIT = "weights/s"
WORKLOAD = "alexnet-fc6 4096x9216, n_q=1, M 100x10, S=0.91, bf16 activations, batch 1"
# DRAM bytes (read + write) of one launch, from one ncu capture of each kernel as it stands now on exactly
# these workloads (summaries under profiles/).  An entry is None while its kernel has changed since the
# counters were taken.  k_decode_gemv: 5.654 MB read, nothing written.  k_decode_bits at 2^30 weights,
# 100x10, S = 0.90: 29.796 MB read + 74.684 MB written while the kernel ran; the other 59.5 MB of its
# 134.2 MB of output were still in L2 when it ended and reach DRAM afterwards.
NCU_DRAM_BYTES_PER_LAUNCH = {"k_decode_gemv": 5.654e6, "k_decode_bits": 104.48e6}
LANES_PER_SM = 128
SMS = 148


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "source": "fallback"}


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


class ClockSampler:
    """Samples SM clock and clock-event (throttle) reasons through NVML (read-only queries) from a
    thread while the timed region runs."""

    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
               "hw_thermal_slowdown": 0x40}

    def __init__(self, index: int, period_s: float = 0.002):
        self.index, self.period = index, period_s
        self.sm, self.bits, self.smax = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        self.error = None

    def _sample(self):
        self.sm.append(float(self._nvml.nvmlDeviceGetClockInfo(self._h, self._nvml.NVML_CLOCK_SM)))
        self.bits |= int(self._nvml.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))

    def _run(self):
        try:
            while not self._stop.is_set():
                self._sample()
                time.sleep(self.period)
        except Exception as e:                      # noqa: BLE001 - report, never fail the benchmark
            self.error = repr(e)

    def start(self):
        """Opens NVML and takes the first sample before returning, so that even a timed region of a few
        milliseconds has samples from inside it."""
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = self.index
            if visible:
                ids = [v.strip() for v in visible.split(",") if v.strip()]
                if self.index < len(ids) and ids[self.index].isdigit():
                    phys = int(ids[self.index])
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.smax = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:                      # noqa: BLE001
            self.error = repr(e)
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2.0)
            try:
                self._sample()                      # one more, taken as the region ends
                self._nvml.nvmlShutdown()
            except Exception as e:                  # noqa: BLE001
                self.error = self.error or repr(e)
        reasons = sorted(k for k, bit in self.REASONS.items() if self.bits & bit)
        if self.error:
            reasons.append("nvml: " + self.error)
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.smax,
                "samples": len(self.sm), "reasons": reasons}


def encode_layer(layer):
    from paper_1905_10138_b200 import sqnn
    from paper_1905_10138_b200 import workloads as wl
    planes_words = np.concatenate([wl.pack_bits(layer.planes[i]) for i in range(layer.n_q)])
    mask_words = wl.pack_bits(layer.mask)
    blob, stats = sqnn.sqnn_encode_host(wl.network_rows(layer.M), layer.n_in, layer.m, layer.n, layer.n_q,
                                        planes_words, mask_words)
    return blob, mask_words, stats


class Flusher:
    """Evicts L2 by writing a buffer larger than it (126 MB)."""

    def __init__(self, torch, nbytes=256 << 20):
        self.buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        self.v = 0

    def __call__(self):
        self.v = (self.v + 1) & 0x7F
        self.buf.fill_(self.v)


def gpu_spin(torch, cycles=400_000):
    """Keeps the GPU busy for ~0.2 ms so that the host has queued the timed call before the GPU
    reaches it (otherwise the event interval would include host launch latency)."""
    try:
        torch.cuda._sleep(cycles)
    except AttributeError:
        pass


def time_steps(torch, fn, steps, warmup, flush):
    """CUDA-event time of each of `steps` calls of fn on the current stream; L2 flushed before each."""
    for _ in range(warmup):
        flush()
        fn()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        flush()
        gpu_spin(torch)
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in ev]          # ms


def time_interval(torch, fn, reps, flush=None, rounds=3):
    """Mean device time of one call of fn in ms.  `reps` calls are timed inside ONE event interval; with a
    flush the interval holds reps x (flush + call) and the same interval over the flushes alone is
    subtracted.  Best of `rounds` (each round is already a mean over `reps`)."""
    def interval(body):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        gpu_spin(torch, 2_000_000)
        e0.record()
        for _ in range(reps):
            body()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)
    if flush is None:
        return min(interval(fn) for _ in range(rounds)) / reps
    both = min(interval(lambda: (flush(), fn())) for _ in range(rounds))
    alone = min(interval(flush) for _ in range(rounds))
    return (both - alone) / reps


def time_interval_graph(torch, fn, reps, flush=None, rounds=3):
    """As time_interval, but the reps x (flush + call) and the reps flushes are each captured into a CUDA
    graph once and replayed: consecutive kernels then start without the launch grid of about 2 us that
    separately launched kernels show on this system.  Returns None if the work cannot be captured."""
    try:
        side = torch.cuda.Stream()

        def graph_of(body):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                for _ in range(3):
                    body()
                side.synchronize()
                with torch.cuda.graph(g, stream=side):
                    for _ in range(reps):
                        body()
            return g

        def replay(g):
            best = None
            for _ in range(rounds):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record()
                g.replay()
                e1.record()
                torch.cuda.synchronize()
                t = e0.elapsed_time(e1)
                best = t if best is None else min(best, t)
            return best

        if flush is None:
            return replay(graph_of(fn)) / reps
        both = replay(graph_of(lambda: (flush(), fn())))
        alone = replay(graph_of(flush))
        return (both - alone) / reps
    except Exception as e:                          # noqa: BLE001 - fall back to separately launched calls
        print(f"graph timing unavailable: {e!r}", file=sys.stderr)
        try:
            torch.cuda.synchronize()
        except Exception:                           # noqa: BLE001
            pass
        return None


def max_over_ranks(dist, value: float, device) -> float:
    """Slowest rank's value (the job is as slow as its slowest replica); identity without a group."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world: int, units_per_rank: float, slowest_ms_per_step: float) -> float:
    """Replicas only: every rank processes `units_per_rank` per step, the job takes the slowest rank's time."""
    return world * units_per_rank / (slowest_ms_per_step * 1e-3)


def stream_bytes(stats, layer, with_mask):
    b = (stats["bits_wc"] + stats["bits_npatch"] + stats["bits_dpatch"] + stats["bits_index"]) / 8
    if with_mask:
        b += layer.mn / 8
    return b


def run_ours(args):
    import torch
    from paper_1905_10138_b200 import sqnn
    from paper_1905_10138_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = measured_peaks()
    sqnn.lib()                                           # fail loudly if the CUDA library is missing

    layer = wl.make_layer(2)
    blob, mask_words, stats = encode_layer(layer)
    desc = sqnn.sqnn_describe_host(blob)
    h_blob = torch.from_numpy(blob).pin_memory()
    h_mask = torch.from_numpy(mask_words.view(np.int64)).pin_memory()
    h_alpha = torch.from_numpy(layer.alpha).pin_memory()
    x1 = layer.activations(1)
    h_x = torch.from_numpy(x1).to(torch.bfloat16).pin_memory()
    d_blob, d_mask, d_alpha, d_x = h_blob.cuda(), h_mask.cuda(), h_alpha.cuda(), h_x.cuda()
    d_y = torch.zeros((1, layer.m), dtype=torch.float32, device="cuda")
    h_y = torch.zeros((1, layer.m), dtype=torch.float32).pin_memory()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flush = Flusher(torch)

    def step():
        sqnn.sqnn_decode_matmul(desc, d_blob, d_mask, d_alpha, d_x, d_y, None, status)

    # end to end: the step's inputs (blob, mask, scales, activations) sit in ONE pinned host buffer, each part
    # at a 256-byte boundary, and go to a preallocated device buffer in one copy per step; Y comes back
    parts = [h_blob.view(torch.uint8).reshape(-1), h_mask.view(torch.uint8).reshape(-1),
             h_alpha.view(torch.uint8).reshape(-1), h_x.view(torch.uint8).reshape(-1)]
    offs, total = [], 0
    for t in parts:
        offs.append(total)
        total += (t.numel() + 255) & ~255
    h_pack = torch.zeros(total, dtype=torch.uint8).pin_memory()
    for t, o in zip(parts, offs):
        h_pack[o:o + t.numel()] = t
    d_pack = torch.empty(total, dtype=torch.uint8, device="cuda")
    e_blob = d_pack[offs[0]:offs[0] + parts[0].numel()]
    e_mask = d_pack[offs[1]:offs[1] + parts[1].numel()].view(torch.int64)
    e_alpha = d_pack[offs[2]:offs[2] + parts[2].numel()].view(torch.float32).reshape(h_alpha.shape)
    e_x = d_pack[offs[3]:offs[3] + parts[3].numel()].view(torch.bfloat16).reshape(h_x.shape)

    def step_e2e():
        d_pack.copy_(h_pack, non_blocking=True)
        sqnn.sqnn_decode_matmul(desc, e_blob, e_mask, e_alpha, e_x, d_y, None, status)
        h_y.copy_(d_y, non_blocking=True)

    for _ in range(args.warmup):
        flush()
        step()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    # exactly K steps in one event interval over K x (flush + step), minus the K flushes alone, the kernels
    # launched one by one: this is the figure reported.  The same K x (flush + step) replayed from a CUDA graph
    # is reported beside it (separately launched kernels start on a grid of about 2 us on this system; in a
    # graph they do not, but there the flushes alone also pack tighter than flushes with a step between them,
    # so neither difference is the kernel's bare duration).
    ms_stream = time_interval(torch, step, args.steps, flush, rounds=1)
    ms_graph = time_interval_graph(torch, step, args.steps, flush, rounds=1)
    ms_per_step_local = ms_stream
    clocks = sampler.stop()
    if dist:
        dist.barrier()
    total_ms = max_over_ranks(dist, ms_per_step_local * args.steps, "cuda")
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status word set"
    units = layer.mn * layer.n_q
    ms_per_step = total_ms / args.steps
    value = whole_job_rate(world, units, ms_per_step)
    times = time_steps(torch, step, min(args.steps, 20), 0, flush)      # one event interval per step, for comparison

    for _ in range(args.warmup):
        flush()
        step_e2e()
    e2e_ms = max_over_ranks(dist, time_interval(torch, step_e2e, args.steps, flush, rounds=1) * args.steps, "cuda")
    h2d = int(h_pack.numel())
    d2h = int(h_y.numel() * 4)
    e2e = {"value": whole_job_rate(world, units, e2e_ms / args.steps), "unit": UNIT,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    # roofline of the dominant kernel (fused decode-GEMV).  It is bound by plain ALU work: one
    # table-driven expansion per weight bit plus one multiply-add per unpruned weight.
    alg_bytes = stream_bytes(stats, layer, True) + layer.alpha.nbytes + x1.size * 2 + layer.m * 4
    kern_s = ms_per_step_local * 1e-3
    alg_ops = layer.mn * layer.n_q + int(layer.mask.sum()) * layer.n_q
    alu_peak = SMS * LANES_PER_SM * peaks["sm_max_mhz"] * 1e6 / 1e12
    roofline = {"bound": "alu", "achieved": alg_ops / kern_s / 1e12, "peak": alu_peak, "unit": "Tlane-op/s",
                "frac": alg_ops / kern_s / 1e12 / alu_peak, "traffic": NCU_DRAM_BYTES_PER_LAUNCH["k_decode_gemv"],
                "kernel": "k_decode_gemv", "peak_source": f"148 SMs x 128 lanes x {peaks['sm_max_mhz']:.0f} MHz (max SM clock)",
                "per_step_event_intervals_ms_median": float(np.median(times)),
                "hbm_achieved_gbs": alg_bytes / kern_s / 1e9,
                "hbm_frac_of_measured": alg_bytes / kern_s / 1e9 / peaks["hbm_gbs"],
                "algorithmic_bytes": alg_bytes, "peaks": peaks["source"]}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": WORKLOAD, "l2": "flushed between timed iterations (256 MB write)",
                      "parallelism": "replicas only" if world > 1 else "single GPU",
                      "bits_per_weight_eq1": stats["bpw_eq1"], "bits_per_weight_stored": stats["bpw_actual"],
                      "patches": stats["patches"][0],
                      "timing": "K steps in one CUDA-event interval over K x (flush + step), minus K flushes; kernels launched one by one",
                      "ms_per_step_graph_replay": ms_graph},
           "clocks": clocks, "e2e": e2e,
           "gpu_launches": args.steps,          # per step: one launch of the fused decode-GEMV kernel
           "roofline": roofline}

    if rank == 0 and not args.quick:
        out["extra"] = extras(torch, sqnn, wl, layer, desc, d_blob, d_mask, d_alpha, status, flush, peaks, args)
    if rank == 0 and world == 1:
        out["cpu_baseline"] = cpu_baseline(layer)
        out["cpu_baseline"]["cpu_model"] = cpu_model()
    if rank == 0:
        print(json.dumps(out))
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def product_rows(torch, sqnn, layer, desc, d_blob, d_mask, d_alpha, status, flush, peaks, reps):
    """Fused product beside a dense bf16 product of the same layer, at every batch size of the configuration."""
    rows = {}
    w = torch.empty((layer.m, layer.n), dtype=torch.bfloat16, device="cuda")
    sqnn.sqnn_decode(desc, d_blob, d_mask, d_alpha, sqnn.OUT_BF16, w, status)   # dense weights by the library's own decode
    dense_floor_us = layer.mn * 2 / (peaks["hbm_gbs"] * 1e9) * 1e6
    for batch in layer.batches:
        x32 = torch.from_numpy(layer.activations(batch)).cuda()
        xb = x32.to(torch.bfloat16)
        x = x32 if layer.x_dtype == "f32" else xb
        y = torch.zeros((batch, layer.m), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(sqnn.sqnn_workspace_bytes(desc, batch), 256), dtype=torch.uint8, device="cuda")
        dense = lambda: torch.matmul(xb, w.t())
        fused = lambda: sqnn.sqnn_decode_matmul(desc, d_blob, d_mask, d_alpha, x, y, ws, status)
        for f in (dense, fused):
            for _ in range(3):
                f()
        rec = {"dense_bf16_us_cold_l2": 1e3 * time_interval(torch, dense, reps, flush),
               "dense_bf16_us_warm_l2": 1e3 * time_interval(torch, dense, reps),
               "dense_bf16_hbm_floor_us": dense_floor_us,
               "fused_us_cold_l2": 1e3 * time_interval(torch, fused, reps, flush),
               "fused_us_warm_l2": 1e3 * time_interval(torch, fused, reps),
               "path": "fp32 ALU (one kernel)" if batch <= 15 else "decode to packed bits + tcgen05 (two kernels)"}
        # the same four figures with the timed calls replayed from a CUDA graph (both sides alike)
        for key, f, fl in (("dense_bf16_us_cold_l2", dense, flush), ("dense_bf16_us_warm_l2", dense, None),
                           ("fused_us_cold_l2", fused, flush), ("fused_us_warm_l2", fused, None)):
            t = time_interval_graph(torch, f, reps, fl)
            rec[key + "_graph"] = None if t is None else 1e3 * t
        if rec["dense_bf16_us_cold_l2_graph"] and rec["fused_us_cold_l2_graph"]:
            rec["fused_vs_dense_cold_graph"] = rec["dense_bf16_us_cold_l2_graph"] / rec["fused_us_cold_l2_graph"]
        rec["fused_vs_dense_cold"] = rec["dense_bf16_us_cold_l2"] / rec["fused_us_cold_l2"]
        rec["dense_frac_of_hbm_peak_cold"] = dense_floor_us / rec["dense_bf16_us_cold_l2"]
        if batch >= 16:
            flops = 2.0 * layer.mn * batch
            rec["fused_tflops_cold"] = flops / (rec["fused_us_cold_l2"] * 1e-6) / 1e12
            rec["fused_frac_of_bf16_sustained"] = rec["fused_tflops_cold"] / peaks["bf16_tflops_sustained"]
        rows[f"batch{batch}"] = rec
    del w
    return rows


def extras(torch, sqnn, wl, layer2, desc2, d_blob2, d_mask2, d_alpha2, status, flush, peaks, args):
    """Reference points beside the headline: every configuration of the benchmark."""
    ex = {}
    reps = 20
    for cfg in (1, 2, 3, 4):
        if cfg == 2:
            layer, desc, d_blob, d_mask, d_alpha = layer2, desc2, d_blob2, d_mask2, d_alpha2
            stats = None
        else:
            layer = wl.make_layer(cfg)
            blob, mask_words, stats = encode_layer(layer)
            desc = sqnn.sqnn_describe_host(blob)
            d_blob = torch.from_numpy(blob).cuda()
            d_mask = torch.from_numpy(mask_words.view(np.int64)).cuda()
            d_alpha = torch.from_numpy(layer.alpha).cuda()
        rec = {"shape": f"{layer.m}x{layer.n}", "n_q": layer.n_q, "network": f"{layer.n_out}x{layer.n_in}",
               "prune_rate": layer.prune_rate,
               "batches": product_rows(torch, sqnn, layer, desc, d_blob, d_mask, d_alpha, status, flush, peaks, reps)}
        if stats is not None:
            rec["bits_per_weight_eq1"] = stats["bpw_eq1"]
            rec["bits_per_weight_stored"] = stats["bpw_actual"]
        ex[f"cfg{cfg}_{layer.name}"] = rec
        del layer
    if not args.skip_decode_sweep:
        ex["write_ceiling"] = write_ceiling(torch, sqnn, peaks)
        sweep = {}
        for i_s in range(len(wl.SWEEP_PRUNE)):
            for i_m in range(len(wl.SWEEP_NETS)):
                head = (i_s, i_m) == (2, 2)
                if args.sweep == "headline" and not head:
                    continue
                name = f"S{wl.SWEEP_PRUNE[i_s]:.2f}_{wl.SWEEP_NETS[i_m][0]}x{wl.SWEEP_NETS[i_m][1]}"
                sweep[name] = decode_point(torch, sqnn, wl, i_s, i_m, flush, peaks, 10, head)
        ex["decode_2p30"] = sweep
    return ex


def write_ceiling(torch, sqnn, peaks):
    """Store-only kernel of the library (the decode kernel's bulk-copy output path, nothing read)."""
    out = {}
    for label, nbytes in (("128MiB", 128 << 20), ("1GiB", 1 << 30)):
        buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        fn = lambda: sqnn.sqnn_store_probe(buf, 3200)
        for _ in range(3):
            fn()
        ms = time_interval(torch, fn, 10)
        out[label] = {"us": ms * 1e3, "gbs": nbytes / (ms * 1e-3) / 1e9,
                      "frac_of_copy_peak": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        del buf
    return out


def decode_point(torch, sqnn, wl, i_s, i_m, flush, peaks, reps, full, m=32768, n=32768):
    layer = wl.make_sweep_layer(i_s, i_m, m=m, n=n)
    blob, mask_words, stats = encode_layer(layer)
    desc = sqnn.sqnn_describe_host(blob)
    d_blob = torch.from_numpy(blob).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    words = (layer.mn + 63) // 64
    out = torch.empty(words, dtype=torch.int64, device="cuda")
    bits = lambda: sqnn.sqnn_decode(desc, d_blob, None, None, sqnn.OUT_BITS, out, status)
    for _ in range(3):
        bits()
    # stream + output (160 MB and more) exceed L2: timed back to back, no flush
    sec = time_interval(torch, bits, reps) * 1e-3
    in_bytes = stream_bytes(stats, layer, False)
    alg = in_bytes + layer.mn / 8
    # patch entries per tile of 256 slices (the unit a warp works on): how uneven the work is (Section 5.1)
    tiles = int(desc.slices_padded) // 256
    idx = blob[int(desc.off_idx[0]): int(desc.off_idx[0]) + 4 * (tiles + 1)].view(np.uint32).astype(np.int64)
    per_tile = np.diff(idx)[: (int(desc.slices) + 255) // 256]
    rec = {"weights": layer.mn, "us": sec * 1e6, "weights_per_s": layer.mn / sec,
           "compressed_stream_gbs": in_bytes / sec / 1e9,
           "roofline": {"bound": "hbm", "achieved": alg / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": alg / sec / 1e9 / peaks["hbm_gbs"],
                        "traffic": NCU_DRAM_BYTES_PER_LAUNCH["k_decode_bits"] if (full and (m, n) == (32768, 32768)) else None,
                        "kernel": "k_decode_bits", "algorithmic_bytes": alg, "peaks": peaks["source"]},
           "bits_per_weight_eq1": stats["bpw_eq1"], "bits_per_weight_stored": stats["bpw_actual"],
           "patches_per_slice": stats["patches"][0] / stats["slices"],
           "patches_per_tile_mean": float(per_tile.mean()), "patches_per_tile_max": int(per_tile.max()),
           "patch_hist": stats["patch_hist"]}
    if full:
        sink = torch.zeros(2, dtype=torch.int64, device="cuda")
        fs = lambda: sqnn.sqnn_decode(desc, d_blob, None, None, sqnn.OUT_SINK, sink, status)
        fs()
        ts = time_interval(torch, fs, reps) * 1e-3
        rec["sink_us"] = ts * 1e6
        rec["sink_stream_gbs"] = in_bytes / ts / 1e9
        d_mask = torch.from_numpy(mask_words.view(np.int64)).cuda()
        d_alpha = torch.from_numpy(layer.alpha).cuda()
        w = torch.empty((layer.m, layer.n), dtype=torch.bfloat16, device="cuda")
        fb = lambda: sqnn.sqnn_decode(desc, d_blob, d_mask, d_alpha, sqnn.OUT_BF16, w, status)
        fb()
        tb = time_interval(torch, fb, 5) * 1e-3
        alg_b = in_bytes + layer.mn / 8 + layer.mn * 2
        rec["bf16_out_us"] = tb * 1e6
        rec["bf16_out_gbs"] = alg_b / tb / 1e9
        rec["bf16_out_frac_of_copy_peak"] = alg_b / tb / 1e9 / peaks["hbm_gbs"]
        del w
    rec["status"] = int(status.item())
    return rec


def oracle_sample(layer, rows):
    """Inputs of the oracle's decode + product restricted to the first `rows` rows of the layer
    (the slices covering them), encoded by the oracle itself."""
    from oracle import oracle as orc
    sub_planes = np.ascontiguousarray(layer.planes[:, :rows, :])
    sub_mask = np.ascontiguousarray(layer.mask[:rows, :])
    arrays = [orc.encode_plane(layer.M, sub_planes[i].ravel(), sub_mask.ravel()) for i in range(layer.n_q)]
    return sub_planes, sub_mask, arrays


def oracle_step(layer, rows, sub_mask, arrays, x64):
    from oracle import oracle as orc
    bits = np.empty((layer.n_q, rows, layer.n), dtype=np.uint8)
    for i, (wc, np_, dp) in enumerate(arrays):
        bits[i] = orc.decode_plane(layer.M, rows * layer.n, wc, np_, dp).reshape(rows, layer.n)
    return orc.matmul(bits, sub_mask, layer.alpha[:rows], x64)


def cpu_baseline(layer, rows=4096):
    """The oracle as it stands (decode of every slice, then the fp64 product) on the host cores."""
    from oracle import oracle as orc
    rows = min(rows, layer.m)
    _, sub_mask, arrays = oracle_sample(layer, rows)
    x64 = layer.activations(1).astype(np.float64)
    oracle_step(layer, rows, sub_mask, arrays, x64)
    t0 = time.perf_counter()
    reps = 10
    for _ in range(reps):
        oracle_step(layer, rows, sub_mask, arrays, x64)
    dt = (time.perf_counter() - t0) / reps
    # the same passes on one thread, for the per-core figure
    threads = orc.num_threads()
    orc.set_num_threads(1)
    t0 = time.perf_counter()
    for _ in range(2):
        oracle_step(layer, rows, sub_mask, arrays, x64)
    dt1 = (time.perf_counter() - t0) / 2
    orc.set_num_threads(threads)
    return {"value": rows * layer.n * layer.n_q / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"first {rows} of {layer.m} rows of the same layer, decode + fp64 product, batch 1, "
                      f"{reps} repetitions", "seconds_per_pass": dt,
            "value_one_thread": rows * layer.n * layer.n_q / dt1}


def run_reference(args):
    """Times the CPU oracle (decode + fp64 product) on the host; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import oracle as orc
    from paper_1905_10138_b200 import workloads as wl
    layer = wl.make_layer(2)
    rows = 2048
    _, sub_mask, arrays = oracle_sample(layer, rows)
    x64 = layer.activations(1).astype(np.float64)
    for _ in range(args.warmup):
        oracle_step(layer, rows, sub_mask, arrays, x64)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(layer, rows, sub_mask, arrays, x64)
    dt = (time.perf_counter() - t0) / args.steps
    value = rows * layer.n * layer.n_q / dt
    sample = f"first {rows} of {layer.m} rows per step (bounded sample), decode + fp64 product, batch 1"
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
           "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
                            "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="headline line only (no extra reference points)")
    ap.add_argument("--skip-decode-sweep", action="store_true", help="skip the 2^30-weight decode-only points")
    ap.add_argument("--sweep", default="all", choices=["all", "headline"],
                    help="decode-only sweep: all 16 points (default) or only S=0.9, M 100x10")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
