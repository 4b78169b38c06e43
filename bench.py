#!/usr/bin/env python
"""Benchmark of the decode + fused-product hot path on synthetic layers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole hot path (stream w^c, XOR expand, patch, mask, rescale,
product) over one batch: ``sqnn_decode_matmul`` on the AlexNet-FC6-shaped layer
(4096 x 9216, 1 plane, M 100 x 10, 91 % pruned) at batch 1.  The metric is decoded
weights per second.  Inputs are resident in HBM for ``value``; ``e2e`` repeats the
measurement with host buffers and the copies inside the timed region.  L2 is flushed
between timed iterations.  Extra keys report the decode-only kernel on 2^30 weights
against the HBM roofline, the batch-64 tensor-core path and a dense bf16 product of the
same layer.  ``--impl reference`` times the CPU oracle on the host cores instead.
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
SM_CLOCK_HZ = 1.965e9
# DRAM bytes (read + write) of one launch, from one ncu capture of each kernel as it stands now on exactly
# these workloads (summaries under profiles/).  Set an entry to None when its kernel changes.
#   k_decode_gemv: 5 697 024 read + 0 written (Y stays in L2).
#   k_decode_bits: 27 243 264 read + 73 993 728 written while the kernel runs; it writes 134 217 728 bytes,
#   the rest is still dirty in L2 when the kernel ends and is written back during the next launch.
NCU_DRAM_BYTES_PER_LAUNCH = {"k_decode_gemv": 5697024, "k_decode_bits": 27243264 + 73993728}
LANES_PER_SM = 128


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


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

    def _run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = self.index
            if visible:
                ids = [v.strip() for v in visible.split(",") if v.strip()]
                if self.index < len(ids) and ids[self.index].isdigit():
                    phys = int(ids[self.index])
            h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.smax = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while not self._stop.is_set():
                self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                self.bits |= int(pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                time.sleep(self.period)
            pynvml.nvmlShutdown()
        except Exception as e:                      # noqa: BLE001 - report, never fail the benchmark
            self.error = repr(e)

    def start(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2.0)
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

    def step_e2e():
        b = h_blob.to("cuda", non_blocking=True)
        mk = h_mask.to("cuda", non_blocking=True)
        al = h_alpha.to("cuda", non_blocking=True)
        xx = h_x.to("cuda", non_blocking=True)
        sqnn.sqnn_decode_matmul(desc, b, mk, al, xx, d_y, None, status)
        h_y.copy_(d_y, non_blocking=True)

    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    times = time_steps(torch, step, args.steps, args.warmup, flush)
    clocks = sampler.stop()
    total_ms = float(sum(times))
    if dist:
        dist.barrier()
    total_ms = max_over_ranks(dist, total_ms, "cuda")
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status word set"
    units = layer.mn * layer.n_q
    ms_per_step = total_ms / args.steps
    value = whole_job_rate(world, units, ms_per_step)

    e2e_times = time_steps(torch, step_e2e, args.steps, args.warmup, flush)
    e2e_ms = max_over_ranks(dist, float(sum(e2e_times)), "cuda")
    h2d = int(h_blob.numel() + h_mask.numel() * 8 + h_alpha.numel() * 4 + h_x.numel() * 2)
    d2h = int(h_y.numel() * 4)
    e2e = {"value": whole_job_rate(world, units, e2e_ms / args.steps), "unit": UNIT,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    # roofline of the dominant kernel (fused decode-GEMV).  It is bound by plain ALU work: one
    # table-driven expansion per weight bit plus one multiply-add per unpruned weight.
    alg_bytes = stream_bytes(stats, layer, True) + layer.alpha.nbytes + x1.size * 2 + layer.m * 4
    kern_s = float(np.mean(times)) * 1e-3
    alg_ops = layer.mn * layer.n_q + int(layer.mask.sum()) * layer.n_q
    alu_peak = 148 * LANES_PER_SM * SM_CLOCK_HZ / 1e12
    roofline = {"bound": "alu", "achieved": alg_ops / kern_s / 1e12, "peak": alu_peak, "unit": "Tlane-op/s",
                "frac": alg_ops / kern_s / 1e12 / alu_peak, "traffic": NCU_DRAM_BYTES_PER_LAUNCH["k_decode_gemv"],
                "kernel": "k_decode_gemv", "peak_source": "148 SMs x 128 lanes x 1.965 GHz",
                "hbm_achieved_gbs": alg_bytes / kern_s / 1e9,
                "hbm_frac_of_measured": alg_bytes / kern_s / 1e9 / peaks["hbm_gbs"],
                "algorithmic_bytes": alg_bytes, "peaks": peaks["source"]}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": WORKLOAD, "l2": "flushed between timed iterations (256 MB write)",
                      "parallelism": "replicas only" if world > 1 else "single GPU",
                      "bits_per_weight_eq1": stats["bpw_eq1"], "bits_per_weight_stored": stats["bpw_actual"],
                      "patches": stats["patches"][0]},
           "clocks": clocks, "e2e": e2e,
           "gpu_launches": 2 * args.steps,      # per step: the kernel clearing Y and the fused decode-GEMV
           "roofline": roofline}

    if rank == 0 and not args.quick:
        out["extra"] = extras(torch, sqnn, wl, layer, desc, d_blob, d_mask, d_alpha, status, flush, peaks, args)
    if rank == 0 and world == 1:
        out["cpu_baseline"] = cpu_baseline(layer)
    if rank == 0:
        print(json.dumps(out))
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def extras(torch, sqnn, wl, layer, desc, d_blob, d_mask, d_alpha, status, flush, peaks, args):
    """Reference points beside the headline: dense bf16 product of the same layer, batch 64, and
    the decode-only kernel on 2^30 weights against the HBM roofline."""
    ex = {}
    steps, warm = max(args.steps, 10), max(args.warmup, 3)
    # dense bf16 weights of the same layer, produced by the library's own bf16 decode
    w = torch.empty((layer.m, layer.n), dtype=torch.bfloat16, device="cuda")
    sqnn.sqnn_decode(desc, d_blob, d_mask, d_alpha, sqnn.OUT_BF16, w, status)
    for batch in (1, 64):
        x = torch.from_numpy(layer.activations(batch)).cuda().to(torch.bfloat16)
        y = torch.zeros((batch, layer.m), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(sqnn.sqnn_workspace_bytes(desc, batch), 256), dtype=torch.uint8, device="cuda")
        dense_cold = time_steps(torch, lambda: torch.matmul(x, w.t()), steps, warm, flush)
        dense_warm = time_steps(torch, lambda: torch.matmul(x, w.t()), steps, warm, lambda: None)
        rec = {"dense_bf16_us_cold_l2": 1e3 * float(np.median(dense_cold)),
               "dense_bf16_us_warm_l2": 1e3 * float(np.median(dense_warm))}
        try:
            fn = lambda: sqnn.sqnn_decode_matmul(desc, d_blob, d_mask, d_alpha, x, y, ws, status)
            cold = time_steps(torch, fn, steps, warm, flush)
            warm_t = time_steps(torch, fn, steps, warm, lambda: None)
            rec["fused_us_cold_l2"] = 1e3 * float(np.median(cold))
            rec["fused_us_warm_l2"] = 1e3 * float(np.median(warm_t))
        except sqnn.SqnnError as e:
            rec["fused"] = str(e)
        ex[f"alexnet_fc6_batch{batch}"] = rec
    del w
    if not args.skip_decode_sweep:
        ex["decode_2p30_100x10_S0.90"] = decode_point(torch, sqnn, wl, 2, 2, flush, peaks, steps, warm)
    return ex


def decode_point(torch, sqnn, wl, i_s, i_m, flush, peaks, steps, warm, m=32768, n=32768):
    layer = wl.make_sweep_layer(i_s, i_m, m=m, n=n)
    blob, mask_words, stats = encode_layer(layer)
    desc = sqnn.sqnn_describe_host(blob)
    d_blob = torch.from_numpy(blob).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    words = (layer.mn + 63) // 64
    out = torch.empty(words, dtype=torch.int64, device="cuda")
    # stream + output (158 MB) exceed L2: timed back to back, no flush
    t = time_steps(torch, lambda: sqnn.sqnn_decode(desc, d_blob, None, None, sqnn.OUT_BITS, out, status),
                   steps, warm, lambda: None)
    sink = torch.zeros(2, dtype=torch.int64, device="cuda")
    ts = time_steps(torch, lambda: sqnn.sqnn_decode(desc, d_blob, None, None, sqnn.OUT_SINK, sink, status),
                    steps, warm, flush)
    # context for the roofline: this kernel writes 5.5 x what it reads, and a write-only stream
    # (a plain fill of 1 GiB) runs well below the copy peak on this part
    big = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
    tf = time_steps(torch, lambda: big.fill_(1), 5, 3, lambda: None)
    write_only_gbs = (1 << 30) / (float(np.median(tf)) * 1e-3) / 1e9
    del big
    sec = float(np.median(t)) * 1e-3
    in_bytes = stream_bytes(stats, layer, False)
    alg = in_bytes + layer.mn / 8
    return {"weights": layer.mn, "us": sec * 1e6, "weights_per_s": layer.mn / sec,
            "compressed_stream_gbs": in_bytes / sec / 1e9,
            "roofline": {"bound": "hbm", "achieved": alg / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": alg / sec / 1e9 / peaks["hbm_gbs"],
                         "traffic": NCU_DRAM_BYTES_PER_LAUNCH["k_decode_bits"] if (i_s, i_m, m, n) == (2, 2, 32768, 32768) else None,
                         "kernel": "k_decode_bits",
                         "algorithmic_bytes": alg, "peaks": peaks["source"],
                         "write_only_fill_gbs": write_only_gbs,
                         "frac_of_write_only_fill": alg / sec / 1e9 / write_only_gbs},
            "sink_us": float(np.median(ts)) * 1e3, "sink_stream_gbs": in_bytes / (float(np.median(ts)) * 1e-3) / 1e9,
            "bits_per_weight_eq1": stats["bpw_eq1"], "bits_per_weight_stored": stats["bpw_actual"],
            "status": int(status.item())}


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
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="headline line only (no extra reference points)")
    ap.add_argument("--skip-decode-sweep", action="store_true", help="skip the 2^30-weight decode-only point")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
