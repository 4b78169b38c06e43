"""Synthetic sweeps in the shape of the paper's figures, run with the library's host encoder.

    python -m paper_1905_10138_b200.sweeps grace      memory reduction against n_out (Section 3.3, first figure)
    python -m paper_1905_10138_b200.sweeps n_in       best reduction against n_in at S = 0.8 / 0.9 / 0.95 (second figure)
    python -m paper_1905_10138_b200.sweeps prune      reduction against the pruning rate S at fixed n_in (third figure)
    python -m paper_1905_10138_b200.sweeps fifo       relative execution time against n_FIFO, beside CSR (Section 5.1)
    python -m paper_1905_10138_b200.sweeps blocked    n_patch bits with per-block widths (Section 5.2)
    python -m paper_1905_10138_b200.sweeps conv       a convolution tensor flattened to a matrix (Section 3.1)

Inputs follow the experiment of Section 3.3: every element is a don't-care with probability S,
otherwise 0 or 1 with equal probability; M is drawn with equal probability per entry.  The paper's
curves come without numbers except the point "about 0.83 at n_in = 20, S = 0.9, n_out near 200";
the sweeps reproduce the shape of the curves around it.  The device format takes n_in <= 32 and
n_out <= 256; the figures go further (n_in to 60, best n_out in the hundreds), so the sweeps use the
library's wide host encoder (64-bit rows of M, n_out up to 4096), which builds no blob.  Everything
here is host work: encoder, Eq. 1 accounting and the FIFO model are the library's C functions; this
file only loops and prints.
"""
from __future__ import annotations

import argparse

import numpy as np

from . import sqnn
from . import workloads as wl


def encode_counts(count: int, prune_rate: float, n_out: int, n_in: int, seed: int, flags=None):
    """Encodes one synthetic plane of `count` elements; returns (stats, n_patch counts)."""
    bits, care = wl.synthetic_plane(count, prune_rate, seed)
    M = wl.xor_network(n_out, n_in, seed + 1)
    blob, stats = sqnn.sqnn_encode_host(wl.network_rows(M), n_in, 1, count, 1, wl.pack_bits(bits),
                                        wl.pack_bits(care), sqnn.ENCODE_ALG1 if flags is None else flags)
    _, n_patch, _ = sqnn.sqnn_unpack_host(blob, 0)
    return stats, n_patch, blob


def memory_reduction(count: int, prune_rate: float, n_out: int, n_in: int, seed: int = 1) -> dict:
    """One point of the first figure: the parts of Eq. 1 in bits per weight and 1 - 1/r."""
    bits, care = wl.synthetic_plane(count, prune_rate, seed)
    M = wl.xor_network(n_out, n_in, seed + 1)
    _, n_patch, _, bpw = sqnn.sqnn_encode_wide_host(wl.network_rows64(M), n_in, count, wl.pack_bits(bits),
                                                    wl.pack_bits(care))
    patches = int(n_patch.astype(np.int64).sum())
    lg_out = int(np.ceil(np.log2(n_out)))
    bits_dp = patches * lg_out / count
    bits_wc = n_in / n_out
    return {"n_out": n_out, "n_in": n_in, "S": prune_rate, "bits_wc": bits_wc, "bits_dpatch": bits_dp,
            "bits_npatch": max(bpw - bits_wc - bits_dp, 0.0), "bits_per_weight": bpw, "reduction": 1.0 - bpw,
            "patches_per_slice": patches / n_patch.size}


def reduction_vs_n_out(count: int, prune_rate: float, n_in: int, n_outs, seed: int = 1):
    return [memory_reduction(count, prune_rate, n_out, n_in, seed) for n_out in n_outs]


def best_reduction(count: int, prune_rate: float, n_in: int, seed: int = 1, step: float = 1.15):
    """Walks n_out upwards from n_in / (1 - S) / 2 until the reduction has fallen twice in a row (the
    figure's lines 'stop when the memory reduction begins to fall'); returns the best point."""
    n_out = max(n_in + 1, int(n_in / (1.0 - prune_rate) / 2))
    best, falls = None, 0
    while n_out <= 4096 and falls < 2:
        p = memory_reduction(count, prune_rate, n_out, n_in, seed)
        if best is None or p["reduction"] > best["reduction"]:
            best, falls = p, 0
        else:
            falls += 1
        n_out = max(n_out + 1, int(n_out * step))
    return best


def fifo_table(count: int, prune_rate: float, n_out: int, n_in: int, banks=(1, 2, 4, 8), depth: int = 256,
               rows: int = 512, lanes: int = 32, seed: int = 1):
    """Relative execution time of the decoder for several n_FIFO (stream as fast as the banks), and of
    lock-step CSR rows at the same pruning rate (Section 5.1's comparison)."""
    _, n_patch, _ = encode_counts(count, prune_rate, n_out, n_in, seed)
    out = {"patches_per_slice": float(n_patch.mean()), "max_patch": int(n_patch.max()), "n_fifo": {}}
    for b in banks:
        out["n_fifo"][b] = sqnn.sqnn_fifo_model_host(n_patch, b, b, depth)["relative_time"]
    # CSR: `rows` rows of count / rows columns, each kept with probability 1 - S, `lanes` rows side by side
    rng = np.random.Generator(np.random.PCG64(seed + 2))
    nnz = rng.binomial(max(count // rows, 1), 1.0 - prune_rate, rows)
    groups = nnz[: rows - rows % lanes].reshape(-1, lanes)
    out["csr"] = float(groups.max(axis=1).sum() / max(groups.sum() / lanes, 1))
    return out


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("what", choices=["grace", "n_in", "prune", "fifo", "blocked", "conv"])
    ap.add_argument("--count", type=int, default=10000, help="elements of the synthetic plane")
    ap.add_argument("--seed", type=int, default=1)
    a = ap.parse_args()
    if a.what == "grace":
        print("n_in = 20, S = 0.9 (bits per weight)\n n_out   w^c    n_patch  d_patch  reduction")
        for p in reduction_vs_n_out(a.count, 0.9, 20, (40, 60, 80, 100, 120, 140, 160, 180, 200, 220, 240, 256), a.seed):
            print(f"{p['n_out']:6d}  {p['bits_wc']:.4f}  {p['bits_npatch']:.4f}   {p['bits_dpatch']:.4f}   {p['reduction']:.4f}")
    elif a.what == "n_in":
        print("best memory reduction over n_out\n  n_in   S=0.8 (n_out)   S=0.9 (n_out)   S=0.95 (n_out)")
        for n_in in (12, 16, 20, 24, 28, 32, 40, 48, 60):
            cells = [best_reduction(a.count, s, n_in, a.seed) for s in (0.8, 0.9, 0.95)]
            print(f"{n_in:6d}   " + "   ".join(f"{c['reduction']:.4f} ({c['n_out']:4d})" for c in cells))
    elif a.what == "prune":
        print("n_in = 20\n    S    best reduction (n_out)   S - reduction")
        for s in (0.5, 0.6, 0.7, 0.8, 0.85, 0.9, 0.95):
            c = best_reduction(a.count, s, 20, a.seed)
            print(f"{s:5.2f}   {c['reduction']:.4f} ({c['n_out']:3d})          {s - c['reduction']:.4f}")
    elif a.what == "fifo":
        print("relative execution time (1.0 = one slice per cycle)\n    S   (n_out,n_in)  patches/slice  max   " +
              "  ".join(f"n_FIFO={b}" for b in (1, 2, 4, 8)) + "   CSR, 32 rows side by side")
        for s in (0.6, 0.8, 0.9, 0.95):
            for n_out, n_in in ((100, 10), (200, 10), (80, 16)):
                t = fifo_table(max(a.count, 200000), s, n_out, n_in, seed=a.seed)
                print(f"{s:5.2f}   ({n_out:3d},{n_in:2d})     {t['patches_per_slice']:8.3f}   {t['max_patch']:4d}   " +
                      "  ".join(f"{t['n_fifo'][b]:8.3f}" for b in (1, 2, 4, 8)) + f"   {t['csr']:.3f}")
    elif a.what == "blocked":
        print("n_patch bits per weight, one width per plane against one per block (S = 0.9, M 100 x 10,\n"
              "first tenth of the plane pruned at 0.5 only)\n   block   bits/weight (n_patch)   bits/weight (Eq. 1)")
        count = max(a.count, 200000)
        bits, care = wl.synthetic_plane(count, 0.9, a.seed)
        dense = np.random.Generator(np.random.PCG64(a.seed + 3)).random(count // 10) >= 0.5
        care[: count // 10] = dense
        M = wl.xor_network(100, 10, a.seed + 1)
        blob, stats = sqnn.sqnn_encode_host(wl.network_rows(M), 10, 1, count, 1, wl.pack_bits(bits), wl.pack_bits(care))
        for block in (stats["slices"], 1024, 128, 16):
            b = sqnn.sqnn_stats_blocked_host(blob, block)
            print(f"{block:8d}   {b['bits_npatch'] / count:.4f}                  {b['bpw_eq1']:.4f}")
    else:
        print("ResNet-shaped 3 x 3 convolutions, 2-bit binary codes, 70 % pruned, M 40 x 12 (Section 3.1: a 4-D tensor\n"
              "is flattened like any other)\n  c_out x c_in x 3 x 3   weights   patches/slice   bits/weight (Eq. 1)   stored")
        for c in (16, 32, 64, 128):
            layer = wl.make_conv_layer(c, c, 3, 3, seed=a.seed)
            planes = np.concatenate([wl.pack_bits(layer.planes[i]) for i in range(layer.n_q)])
            _, st = sqnn.sqnn_encode_host(wl.network_rows(layer.M), layer.n_in, layer.m, layer.n, layer.n_q, planes,
                                          wl.pack_bits(layer.mask))
            print(f"  {c:4d} x {c:4d} x 3 x 3   {layer.mn:8d}   {sum(st['patches']) / (layer.n_q * st['slices']):8.3f}        "
                  f"{st['bpw_eq1']:.4f}              {st['bpw_actual']:.4f}")


if __name__ == "__main__":
    main()
