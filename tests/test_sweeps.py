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


def test_n_in_sweep_reaches_the_papers_range():
    """Second figure of Section 3.3: the best reduction keeps growing with n_in up to 60, the best n_out moves
    into the hundreds (beyond what the device format stores), and the gap to S shrinks."""
    best = {n_in: sweeps.best_reduction(20000, 0.9, n_in) for n_in in (20, 40, 60)}
    red = [best[k]["reduction"] for k in (20, 40, 60)]
    assert red[0] < red[1] < red[2] < 0.9
    assert best[40]["n_out"] > 256 and best[60]["n_out"] > best[40]["n_out"]
    assert 0.9 - red[2] < 0.04


def test_wide_host_encoder_matches_the_oracle_bit_for_bit():
    """Algorithm 1 with 64-bit rows of M (n_in = 40, 60, 64; n_out beyond 256) against the oracle's."""
    from oracle import oracle as orc
    from paper_1905_10138_b200 import sqnn, workloads as wl
    for n_out, n_in, count, S in ((300, 40, 9000, 0.9), (600, 60, 12000, 0.9), (333, 64, 7001, 0.8), (90, 33, 4000, 0.5)):
        bits, care = wl.synthetic_plane(count, S, 5)
        M = wl.xor_network(n_out, n_in, 6)
        wc, np_, dp, bpw = sqnn.sqnn_encode_wide_host(wl.network_rows64(M), n_in, count, wl.pack_bits(bits), wl.pack_bits(care))
        r_wc, r_np, r_dp = orc.encode_plane(M, bits, care)
        assert np.array_equal(wc, r_wc) and np.array_equal(np_, r_np) and np.array_equal(dp, r_dp)
        assert bpw == pytest.approx(orc.eq1(count, n_out, n_in, r_np)["bits_per_weight"], rel=1e-12)
        out = orc.decode_plane(M, count, wc, np_, dp)
        assert np.array_equal(out[care == 1], bits[care == 1])
    with pytest.raises(sqnn.SqnnError):
        sqnn.sqnn_encode_wide_host(np.zeros(8, np.uint64), 65, 64, np.zeros(1, np.uint64), np.zeros(1, np.uint64))


def test_conv_layer_is_a_flattened_4d_tensor():
    from paper_1905_10138_b200 import workloads as wl
    layer = wl.make_conv_layer(16, 8, 3, 3)
    assert (layer.m, layer.n, layer.n_q) == (16, 72, 2)
    assert abs(layer.mask.mean() - 0.30) < 0.01 and layer.alpha.shape == (16, 2)
