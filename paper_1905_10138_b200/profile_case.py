"""Runs one kernel of the library a few times on a synthetic case, for profilers and quick timing.

    python -m paper_1905_10138_b200.profile_case decode  --sweep 2 2 --rows 16384 --cols 32768 --iters 3
    python -m paper_1905_10138_b200.profile_case sink    --sweep 2 2
    python -m paper_1905_10138_b200.profile_case bf16    --cfg 3
    python -m paper_1905_10138_b200.profile_case matmul  --cfg 2 --batch 1
    python -m paper_1905_10138_b200.profile_case search  --cfg 2          (exhaustive seed search)

--cfg 1..4 picks a layer of the benchmark configurations (optionally --rows / --cols smaller),
--sweep I_S I_M a point of the decode-only sweep (prune rate index, network index).
Prints the CUDA-event time of every iteration.
"""
from __future__ import annotations

import argparse

import numpy as np


def main():
    import torch
    from . import sqnn, workloads as wl
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["decode", "sink", "bf16", "matmul", "search"])
    ap.add_argument("--cfg", type=int, default=0)
    ap.add_argument("--sweep", type=int, nargs=2, default=None)
    ap.add_argument("--repeat", type=int, default=0,
                    help="also time REPEAT calls inside one event interval (finer than one event tick)")
    ap.add_argument("--rows", type=int, default=None)
    ap.add_argument("--cols", type=int, default=None)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--flush", action="store_true", help="write 256 MB between iterations (evict L2)")
    a = ap.parse_args()
    if a.sweep is not None:
        layer = wl.make_sweep_layer(a.sweep[0], a.sweep[1], m=a.rows or 32768, n=a.cols or 32768)
    else:
        layer = wl.make_layer(a.cfg or 2, m=a.rows, n=a.cols)
    planes_words = np.concatenate([wl.pack_bits(layer.planes[i]) for i in range(layer.n_q)])
    mask_words = wl.pack_bits(layer.mask)
    blob, stats = sqnn.sqnn_encode_host(wl.network_rows(layer.M), layer.n_in, layer.m, layer.n, layer.n_q,
                                        planes_words, mask_words)
    desc = sqnn.sqnn_describe_host(blob)
    d_blob = torch.from_numpy(blob).cuda()
    d_mask = torch.from_numpy(mask_words.view(np.int64)).cuda()
    d_alpha = torch.from_numpy(layer.alpha).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    words = (layer.mn + 63) // 64
    if a.what == "decode":
        out = torch.empty(layer.n_q * words, dtype=torch.int64, device="cuda")
        fn = lambda: sqnn.sqnn_decode(desc, d_blob, None, None, sqnn.OUT_BITS, out, status)
    elif a.what == "sink":
        out = torch.empty(2, dtype=torch.int64, device="cuda")
        fn = lambda: sqnn.sqnn_decode(desc, d_blob, None, None, sqnn.OUT_SINK, out, status)
    elif a.what == "search":
        slices = (layer.mn + layer.n_out - 1) // layer.n_out
        d_planes = torch.from_numpy(planes_words.view(np.int64)).cuda()
        d_wc = torch.empty(layer.n_q * slices, dtype=torch.int32, device="cuda")
        d_np = torch.empty(layer.n_q * slices, dtype=torch.int16, device="cuda")
        rows = wl.network_rows(layer.M)
        fn = lambda: sqnn.sqnn_search_seeds(rows, layer.n_in, layer.m, layer.n, layer.n_q, d_planes, d_mask,
                                            d_wc, d_np)
    elif a.what == "bf16":
        out = torch.empty((layer.m, layer.n), dtype=torch.bfloat16, device="cuda")
        fn = lambda: sqnn.sqnn_decode(desc, d_blob, d_mask, d_alpha, sqnn.OUT_BF16, out, status)
    else:
        x = torch.from_numpy(layer.activations(a.batch)).cuda()
        if layer.x_dtype == "bf16":
            x = x.to(torch.bfloat16)
        y = torch.empty((a.batch, layer.m), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(sqnn.sqnn_workspace_bytes(desc, a.batch), 256), dtype=torch.uint8, device="cuda")
        fn = lambda: sqnn.sqnn_decode_matmul(desc, d_blob, d_mask, d_alpha, x, y, ws, status)
    scratch = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if a.flush else None
    times = []
    for it in range(a.iters):
        if scratch is not None:
            scratch.fill_(it & 0x7F)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(400_000)          # let the host queue the call before the GPU gets to it
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3)
    if a.repeat > 0:
        def interval(f):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(2_000_000)
            e0.record()
            for _ in range(a.repeat):
                f()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e3 / a.repeat
        if scratch is not None:
            both = min(interval(lambda: (scratch.fill_(1), fn())) for _ in range(3))
            alone = min(interval(lambda: scratch.fill_(1)) for _ in range(3))
            print(f"{a.repeat} x (flush + call) {both:.2f} us each, flush alone {alone:.2f}: call {both - alone:.2f} us (cold L2)")
        else:
            print(f"{a.repeat} calls back to back: {min(interval(fn) for _ in range(3)):.2f} us each (warm L2)")
    if a.what == "search":
        found = d_np.cpu().numpy().view(np.uint16).reshape(layer.n_q, -1).astype(np.int64).sum(axis=1)
        print(f"exhaustive search patches per plane {found.tolist()} vs Algorithm 1 {stats['patches'][:layer.n_q]}")
    print(f"{a.what} {layer.name} {layer.m}x{layer.n} n_q={layer.n_q} M {layer.n_out}x{layer.n_in}: "
          f"us per iteration {['%.1f' % t for t in times[:8]]} mean after the first {np.mean(times[1:]) if len(times) > 1 else times[0]:.2f}  patches {stats['patches'][:layer.n_q]} "
          f"stored bits/weight {stats['bpw_actual']:.4f}  status {int(status.item())}")


if __name__ == "__main__":
    main()
