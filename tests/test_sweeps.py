"""CPU tests of the synthetic sweeps (Section 3.3 figures, Section 5.1 comparison) run with the library's
host encoder: the paper's printed point and the trends its figures show."""
import numpy as np
import pytest

from paper_1905_10138_b200 import sweeps


def golden():
    import os
    out = {}
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "paper_points.txt")
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            key, value, _ = [f.strip() for f in line.split("|")]
            out[key] = value
    return out


def test_paper_point_memory_reduction_near_0_83():
    g = golden()
    p = sweeps.memory_reduction(int(g["grace_elements"]), float(g["grace_prune_rate"]), int(g["grace_n_out"]),
                                int(g["grace_n_in"]))
    # Section 3.3 prints "about 0.83"; one random matrix of 10,000 elements scatters around it
    assert abs(p["reduction"] - float(g["grace_memory_reduction"])) <= 0.04
    assert p["bits_wc"] == pytest.approx(0.1)


def test_trade_off_between_seed_bits_and_patch_bits():
    pts = sweeps.reduction_vs_n_out(10000, 0.9, 20, (60, 120, 180, 240))
    assert [p["bits_wc"] for p in pts] == sorted((p["bits_wc"] for p in pts), reverse=True)   # w^c shrinks
    assert pts[-1]["bits_dpatch"] > pts[0]["bits_dpatch"]                                      # patches grow
    best = max(pts, key=lambda p: p["reduction"])
    assert best["n_out"] in (120, 180)                                                         # an interior optimum
    assert best["reduction"] < 0.9                                                             # bounded by S


def test_larger_n_in_and_higher_pruning_help():
    a, b = sweeps.best_reduction(10000, 0.8, 12), sweeps.best_reduction(10000, 0.8, 20)
    assert b["reduction"] > a["reduction"] and b["n_out"] > a["n_out"]
    gap = [s - sweeps.best_reduction(10000, s, 20)["reduction"] for s in (0.6, 0.8, 0.9)]
    assert gap[0] > gap[1] > gap[2] > 0              # the reduction approaches S as S grows


def test_fifo_banks_and_csr_rows():
    t = sweeps.fifo_table(100000, 0.8, 100, 10)
    times = [t["n_fifo"][b] for b in (1, 2, 4, 8)]
    assert times == sorted(times, reverse=True) and times[0] >= t["patches_per_slice"] and times[-1] < 1.2
    assert t["csr"] > 1.1                            # rows of unequal length make lock-step CSR wait
    light = sweeps.fifo_table(100000, 0.95, 100, 10)
    assert light["n_fifo"][2] < 1.01                 # few patches: two banks already remove the stalls


def test_conv_tensor_is_flattened_to_rows_of_output_channels():
    assert sweeps.conv_as_matrix(64, 32, 3, 3) == (64, 288)
