"""Pins for the CPU oracle: every expectation below comes from brute force, a closed
form, a numpy / torch library routine, a hand computation or a value the paper
prints -- never from the oracle itself and never from the CUDA library."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import oracle as orc
from paper_1905_10138_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_points.txt")


def golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or "|" not in line:
                continue
            k, v, _ = [t.strip() for t in line.split("|", 2)]
            out[k] = v
    return out


def seed_bits(v, n_in):
    return np.array([(v >> t) & 1 for t in range(n_in)], dtype=np.uint8)


# ----------------------------------------------------------------------------------
# Decryption w~ = M . w^c over GF(2)  (Section 3.1)
# ----------------------------------------------------------------------------------
@pytest.mark.parametrize("n_out,n_in,seed", [(8, 4, 1), (16, 8, 2), (13, 5, 3), (4, 3, 4)])
def test_xor_network_equals_integer_matvec_mod_2_for_every_seed(n_out, n_in, seed):
    M = wl.xor_network(n_out, n_in, seed)
    for v in range(1 << n_in):
        wc = seed_bits(v, n_in)
        expect = (M.astype(np.int64) @ wc.astype(np.int64)) % 2
        assert np.array_equal(orc.xor_network(M, wc), expect.astype(np.uint8))


def test_xor_network_unit_seeds_give_columns_and_zero_gives_zero():
    M = wl.xor_network(40, 12, 7)
    assert not orc.xor_network(M, np.zeros(12, np.uint8)).any()
    for t in range(12):
        e = np.zeros(12, np.uint8)
        e[t] = 1
        assert np.array_equal(orc.xor_network(M, e), M[:, t])


def test_xor_network_is_linear():
    rng = np.random.default_rng(5)
    M = wl.xor_network(100, 10, 11)
    for _ in range(50):
        a = rng.integers(0, 2, 10, dtype=np.uint8)
        b = rng.integers(0, 2, 10, dtype=np.uint8)
        assert np.array_equal(orc.xor_network(M, a ^ b), orc.xor_network(M, a) ^ orc.xor_network(M, b))


def test_transposed_network_would_fail():
    """A transposed operand is caught: for a non-square M only one orientation type-checks, and
    for a square non-symmetric M the column pin above distinguishes M from M^T."""
    M = np.array([[1, 1, 0], [0, 1, 0], [0, 0, 1]], dtype=np.uint8)
    e0 = np.array([1, 0, 0], np.uint8)
    assert np.array_equal(orc.xor_network(M, e0), np.array([1, 0, 0], np.uint8))  # column 0, not row 0


# ----------------------------------------------------------------------------------
# Algorithm 1 against a brute-force statement of what it computes
# ----------------------------------------------------------------------------------
def all_outputs(M):
    n_out, n_in = M.shape
    outs = np.zeros((1 << n_in, n_out), dtype=np.uint8)
    for v in range(1 << n_in):
        outs[v] = (M.astype(np.int64) @ seed_bits(v, n_in).astype(np.int64)) % 2
    return outs


def brute_force_alg1(M, wq, care):
    """Greedy of Algorithm 1 with solvability decided by listing every seed: a care row is kept
    iff some seed satisfies it together with all rows kept so far.  Then the seed: among all
    seeds satisfying the kept rows, the one whose free variables are 0, where the pivot columns
    are those columns of the kept coefficient matrix not spanned by the columns before them."""
    n_out, n_in = M.shape
    outs = all_outputs(M)
    alive = np.ones(1 << n_in, dtype=bool)
    kept, rejected = [], []
    for i in range(n_out):
        if not care[i]:
            continue
        cand = alive & (outs[:, i] == wq[i])
        if cand.any():
            alive = cand
            kept.append(i)
        else:
            rejected.append(i)
    A = M[kept, :] if kept else np.zeros((0, n_in), dtype=np.uint8)
    pivots = []
    for c in range(n_in):
        col = A[:, c]
        spanned = False
        for r in range(len(pivots) + 1):       # combos of earlier *pivot* columns span the same space
            for combo in itertools.combinations(pivots, r):
                s = np.zeros(A.shape[0], dtype=np.uint8)
                for q in combo:
                    s ^= A[:, q]
                if np.array_equal(s, col):
                    spanned = True
                    break
            if spanned:
                break
        if not spanned:
            pivots.append(c)
    free = [c for c in range(n_in) if c not in pivots]
    sols = [v for v in np.flatnonzero(alive) if all(((v >> f) & 1) == 0 for f in free)]
    assert len(sols) == 1
    return int(sols[0]), rejected


@pytest.mark.parametrize("n_out,n_in,keep", [(8, 4, 0.5), (10, 4, 0.7), (12, 5, 0.5), (16, 6, 0.6), (9, 3, 1.0)])
def test_alg1_matches_brute_force_greedy_and_free_variables_zero(n_out, n_in, keep):
    rng = np.random.default_rng(100 * n_out + n_in)
    for trial in range(60):
        M = rng.integers(0, 2, (n_out, n_in), dtype=np.uint8)
        wq = rng.integers(0, 2, n_out, dtype=np.uint8)
        care = (rng.random(n_out) < keep).astype(np.uint8)
        wc, dp = orc.encode_slice(M, wq, care)
        v_expect, rej_expect = brute_force_alg1(M, wq, care)
        v = int(sum(int(b) << t for t, b in enumerate(wc)))
        assert list(dp) == rej_expect, (trial, M, wq, care)
        assert v == v_expect, (trial, M, wq, care)


def test_reduced_system_keeps_only_care_rows_like_the_papers_8x4_example():
    """Section 3.1: with care bits {3,4,5,7} (1-based) of 8 the system is the 4 x 4 one made of
    those rows; don't-care rows impose nothing.  The figure's entries are not printed, so the
    check runs over random 8 x 4 networks: the encoder's answer must not depend on the wanted
    bits at don't-care positions, and must satisfy the brute-force minimum over the 16 seeds
    when that minimum is 0."""
    care_rows = [int(t) - 1 for t in golden()["fig_overall_care_rows"].split(",")]
    care = np.zeros(8, np.uint8)
    care[care_rows] = 1
    rng = np.random.default_rng(3457)
    for _ in range(100):
        M = rng.integers(0, 2, (8, 4), dtype=np.uint8)
        wq = rng.integers(0, 2, 8, dtype=np.uint8)
        wc, dp = orc.encode_slice(M, wq, care)
        wq2 = wq.copy()
        wq2[care == 0] ^= 1
        wc2, dp2 = orc.encode_slice(M, wq2, care)
        assert np.array_equal(wc, wc2) and np.array_equal(dp, dp2)
        outs = all_outputs(M)
        wrong = ((outs != wq[None, :]) & (care[None, :] == 1)).sum(axis=1)
        if wrong.min() == 0:
            assert dp.size == 0
        assert set(dp.tolist()) <= set(care_rows)


def test_lossless_every_care_bit_reproduced_after_patches():
    """Section 3.2: with n_patch / d_patch all care bits come back."""
    rng = np.random.default_rng(9)
    for (n_out, n_in, keep) in [(80, 8, 0.1), (100, 10, 0.09), (60, 12, 0.2), (40, 12, 0.3), (200, 10, 0.4)]:
        M = wl.xor_network(n_out, n_in, n_out + n_in)
        for _ in range(40):
            wq = rng.integers(0, 2, n_out, dtype=np.uint8)
            care = (rng.random(n_out) < keep).astype(np.uint8)
            wc, dp = orc.encode_slice(M, wq, care)
            out = orc.decode_slice(M, wc, dp)
            assert np.array_equal(out[care == 1], wq[care == 1])
            assert np.all(care[dp] == 1) and np.all(np.diff(dp.astype(int)) > 0)
            raw = orc.xor_network(M, wc)
            assert np.array_equal(np.flatnonzero((raw != wq) & (care == 1)), dp)


def test_no_care_bits_gives_zero_seed_and_no_patches():
    M = wl.xor_network(80, 8, 1)
    wc, dp = orc.encode_slice(M, np.ones(80, np.uint8), np.zeros(80, np.uint8))
    assert not wc.any() and dp.size == 0


def test_square_invertible_network_with_all_care_bits_is_plain_linear_solve():
    """Textbook special case: no don't-cares, M square and invertible => w^c = M^-1 w^q, no patch."""
    rng = np.random.default_rng(21)
    found = 0
    while found < 20:
        M = rng.integers(0, 2, (8, 8), dtype=np.uint8)
        if round(abs(np.linalg.det(M.astype(np.float64)))) % 2 == 0:
            continue          # singular over GF(2)
        found += 1
        outs = all_outputs(M)
        wq = rng.integers(0, 2, 8, dtype=np.uint8)
        wc, dp = orc.encode_slice(M, wq, np.ones(8, np.uint8))
        hits = np.flatnonzero((outs == wq[None, :]).all(axis=1))
        assert hits.size == 1
        assert dp.size == 0 and int(sum(int(b) << t for t, b in enumerate(wc))) == int(hits[0])


def test_consistent_systems_need_no_patch():
    """If the care bits are the network's own output for some seed, the system is solvable."""
    rng = np.random.default_rng(33)
    M = wl.xor_network(100, 10, 5)
    for _ in range(50):
        wq = orc.xor_network(M, rng.integers(0, 2, 10, dtype=np.uint8))
        care = (rng.random(100) < 0.5).astype(np.uint8)
        _, dp = orc.encode_slice(M, wq, care)
        assert dp.size == 0


def test_exhaustive_search_keeps_the_smallest_of_equally_good_seeds():
    """Reading taken for Section 5.2 (the paper does not say which of several minimal seeds to keep): the
    numerically smallest.  Hand-made slices whose optimal seeds are known by inspection."""
    # one output = w0 xor w1, wanted 1: seeds 01 and 10 are both perfect, 00 and 11 both miss
    M = np.array([[1, 1]], dtype=np.uint8)
    wc, dp = orc.encode_slice(M, np.array([1], np.uint8), np.array([1], np.uint8), exhaustive=True)
    assert wc.tolist() == [1, 0] and dp.size == 0                      # seed 1, not seed 2
    # outputs (w0, w0, w1 xor w2) wanted (1, 0, 1): one of the first two care bits is lost whatever w0 is;
    # the four seeds with w1 xor w2 = 1 tie at one patch: 2 (010), 3 (110), 4 (001), 5 (101) -> seed 2
    M = np.array([[1, 0, 0], [1, 0, 0], [0, 1, 1]], dtype=np.uint8)
    wq, care = np.array([1, 0, 1], np.uint8), np.ones(3, np.uint8)
    wc, dp = orc.encode_slice(M, wq, care, exhaustive=True)
    assert wc.tolist() == [0, 1, 0] and dp.tolist() == [0]
    # a don't-care on the contested position breaks the tie the other way round
    wc, dp = orc.encode_slice(M, wq, np.array([0, 1, 1], np.uint8), exhaustive=True)
    assert wc.tolist() == [0, 1, 0] and dp.size == 0
    wc, dp = orc.encode_slice(M, wq, np.array([1, 0, 1], np.uint8), exhaustive=True)
    assert wc.tolist() == [1, 1, 0] and dp.size == 0                   # seed 3 is the smallest with w0 = 1


def test_exhaustive_search_is_a_lower_bound_and_alg1_is_close():
    """Section 5.2 / 3.3: the exhaustive search minimises the patch count; Algorithm 1 needs
    somewhat more.  The paper reports up to 10 % more in its own (unspecified) experiments; at
    the small n_in used here the measured excess is 20-45 %, so only a loose bound is held."""
    rng = np.random.default_rng(77)
    M = wl.xor_network(60, 8, 4)
    outs = all_outputs(M)
    tot_a = tot_e = 0
    for _ in range(300):
        wq = rng.integers(0, 2, 60, dtype=np.uint8)
        care = (rng.random(60) < 0.13).astype(np.uint8)
        _, dp_a = orc.encode_slice(M, wq, care)
        wc_e, dp_e = orc.encode_slice(M, wq, care, exhaustive=True)
        brute_min = ((outs != wq[None, :]) & (care[None, :] == 1)).sum(axis=1).min()
        assert dp_e.size == brute_min
        assert dp_e.size <= dp_a.size
        out = orc.decode_slice(M, wc_e, dp_e)
        assert np.array_equal(out[care == 1], wq[care == 1])
        tot_a += dp_a.size
        tot_e += dp_e.size
    assert tot_e <= tot_a <= 1.6 * tot_e


# ----------------------------------------------------------------------------------
# Patch statistics: closed form from Algorithm 1 with iid uniform rows and bits
# ----------------------------------------------------------------------------------
def expected_rank(k, n_in):
    """E[rank] of a k x n_in matrix of iid uniform bits: rank goes r -> r+1 w.p. 1 - 2^(r-n_in)."""
    dist = np.zeros(n_in + 1)
    dist[0] = 1.0
    for _ in range(k):
        new = np.zeros_like(dist)
        for r in range(n_in + 1):
            up = 1.0 - 2.0 ** (r - n_in)
            new[r] += dist[r] * (1 - up)
            if r < n_in:
                new[r + 1] += dist[r] * up
        dist = new
    return float((dist * np.arange(n_in + 1)).sum())


def expected_patches(n_out, n_in, prune):
    """A tried row is rejected iff it lies in the span of the kept rows (prob 2^(rank-n_in)) and its
    bit disagrees (prob 1/2): E[n_patch | k] = (k - E[rank_k]) / 2, k ~ Binomial(n_out, 1 - S)."""
    tot = 0.0
    for k in range(n_out + 1):
        pk = math.comb(n_out, k) * (1 - prune) ** k * prune ** (n_out - k)
        tot += pk * (k - expected_rank(k, n_in)) / 2.0
    return tot


@pytest.mark.parametrize("n_out,n_in,prune", [(100, 10, 0.90), (60, 12, 0.80), (80, 8, 0.90), (200, 10, 0.80)])
def test_mean_patch_count_follows_closed_form(n_out, n_in, prune):
    want = expected_patches(n_out, n_in, prune)
    got = []
    for rep in range(6):                     # several draws of M: the closed form averages over M
        M = wl.xor_network(n_out, n_in, 900 + rep)
        bits, care = wl.synthetic_plane(n_out * 1500, prune, 40 + rep)
        _, np_, dp = orc.encode_plane(M, bits, care)
        assert dp.size == int(np_.sum())
        got.append(np_.mean())
    got = float(np.mean(got))
    assert abs(got - want) <= 0.06 * want + 0.01, (got, want)


def test_closed_form_limit_many_care_bits():
    assert abs(expected_patches(200, 10, 0.0) - (200 - 10) / 2) < 0.01


# ----------------------------------------------------------------------------------
# Eq. 1 and the paper's printed point
# ----------------------------------------------------------------------------------
def test_eq1_hand_computed():
    # mn = 1000, n_out = 100, n_in = 10, l = 10; p = (0,1,3,0,0,2,0,0,1,0): max 3 -> 2 bits, sum 7,
    # ceil(lg 100) = 7.  bits = 100 + 10*2 + 7*7 = 169.
    p = np.array([0, 1, 3, 0, 0, 2, 0, 0, 1, 0], dtype=np.uint16)
    e = orc.eq1(1000, 100, 10, p)
    assert e["bits_wc"] == 100 and e["bits_npatch"] == 20 and e["bits_dpatch"] == 49
    assert abs(e["r"] - 1000 / 169) < 1e-12
    # ragged tail: mn = 950 -> l = 10 still, first term 95
    e = orc.eq1(950, 100, 10, p)
    assert abs(e["r"] - 950 / (95 + 20 + 49)) < 1e-12
    # no patches at all: both patch terms vanish, r = n_out / n_in
    e = orc.eq1(1000, 100, 10, np.zeros(10, np.uint16))
    assert abs(e["r"] - 10.0) < 1e-12
    # max p = 1 -> ceil(lg 1) = 0 bits, max p = 4 -> 2 bits, max p = 5 -> 3 bits (literal reading)
    assert orc.eq1(1000, 100, 10, np.array([1] + [0] * 9, np.uint16))["bits_npatch"] == 0
    assert orc.eq1(1000, 100, 10, np.array([4] + [0] * 9, np.uint16))["bits_npatch"] == 20
    assert orc.eq1(1000, 100, 10, np.array([5] + [0] * 9, np.uint16))["bits_npatch"] == 30
    # n_out = 128 -> 7 bits per position, 129 -> 8
    assert orc.eq1(1280, 128, 10, np.array([1] * 10, np.uint16))["bits_dpatch"] == 70
    assert orc.eq1(1290, 129, 10, np.array([1] * 10, np.uint16))["bits_dpatch"] == 80


def test_papers_synthetic_point_memory_reduction():
    """Section 3.3: 10,000 random elements, S = 0.9, n_in = 20, n_out near 200 -> memory reduction
    about 0.83.  The closed form gives 0.84-0.85 (0.100 + 0.038 + about 0.015 bits/weight)."""
    g = golden()
    n_in, n_out = int(g["grace_n_in"]), int(g["grace_n_out"])
    count, prune = int(g["grace_elements"]), float(g["grace_prune_rate"])
    target = float(g["grace_memory_reduction"])
    reds = []
    for rep in range(4):
        M = wl.xor_network(n_out, n_in, 200 + rep)
        bits, care = wl.synthetic_plane(count, prune, 300 + rep)
        wc, np_, dp = orc.encode_plane(M, bits, care)
        out = orc.decode_plane(M, count, wc, np_, dp)
        assert np.array_equal(out[care == 1], bits[care == 1])
        reds.append(1.0 - 1.0 / orc.eq1(count, n_out, n_in, np_)["r"])
    red = float(np.mean(reds))
    assert target - 0.03 <= red <= target + 0.04, reds


def test_memory_reduction_tradeoff_and_asymptote():
    """Section 3.3: w^c bits fall as n_out grows while patch bits rise; the reduction stays
    below S (ratio below 1/(1-S)) and gets near it at the best n_out."""
    prune, n_in, count = 0.9, 20, 40000
    bits, care = wl.synthetic_plane(count, prune, 17)
    last_wc, last_patch, best = None, None, 0.0
    for n_out in (80, 140, 200, 260):
        M = wl.xor_network(n_out, n_in, n_out)
        _, np_, _ = orc.encode_plane(M, bits, care)
        e = orc.eq1(count, n_out, n_in, np_)
        patch_bits = e["bits_npatch"] + e["bits_dpatch"]
        if last_wc is not None:
            assert e["bits_wc"] < last_wc and patch_bits > last_patch
        last_wc, last_patch = e["bits_wc"], patch_bits
        red = 1 - 1 / e["r"]
        assert red < prune
        best = max(best, red)
    assert best > 0.80


# ----------------------------------------------------------------------------------
# plane-level encode / decode bookkeeping (slicing, tail padding, patch stream order)
# ----------------------------------------------------------------------------------
def test_plane_encode_equals_slice_by_slice_and_handles_ragged_tail():
    M = wl.xor_network(80, 8, 1003)
    mn = 80 * 7 + 16                        # last slice has 16 real positions
    bits, care = wl.synthetic_plane(mn, 0.8, 5)
    wc, np_, dp = orc.encode_plane(M, bits, care)
    assert wc.size == 8
    cursor = 0
    for s in range(8):
        wq = np.zeros(80, np.uint8)
        cr = np.zeros(80, np.uint8)
        seg = slice(s * 80, min(mn, (s + 1) * 80))
        wq[: seg.stop - seg.start] = bits[seg]
        cr[: seg.stop - seg.start] = care[seg]
        wcs, dps = orc.encode_slice(M, wq, cr)
        assert int(sum(int(b) << t for t, b in enumerate(wcs))) == int(wc[s])
        assert np_[s] == dps.size and np.array_equal(dp[cursor:cursor + dps.size], dps)
        cursor += dps.size
    assert cursor == dp.size
    out = orc.decode_plane(M, mn, wc, np_, dp)
    assert np.array_equal(out[care == 1], bits[care == 1])
    # don't-care outputs are the raw network outputs
    raw = np.concatenate([orc.xor_network(M, seed_bits(int(v), 8)) for v in wc])[:mn]
    flips = np.zeros(mn, np.uint8)
    starts = np.concatenate([[0], np.cumsum(np_.astype(np.int64))]).astype(np.int64)
    for s in range(8):
        for k in range(starts[s], starts[s + 1]):
            flips[s * 80 + dp[k]] ^= 1
    assert np.array_equal(out, raw ^ flips)


def test_decode_plane_partial_range_only_touches_its_slices():
    M = wl.xor_network(40, 12, 2)
    bits, care = wl.synthetic_plane(4000, 0.7, 6)
    wc, np_, dp = orc.encode_plane(M, bits, care)
    full = orc.decode_plane(M, 4000, wc, np_, dp)
    part = orc.decode_plane(M, 4000, wc, np_, dp, 10, 20, out=np.full(4000, 9, np.uint8))
    assert np.array_equal(part[400:800], full[400:800])
    assert np.all(part[:400] == 9) and np.all(part[800:] == 9)


# ----------------------------------------------------------------------------------
# bf16 rounding, reconstruction, product
# ----------------------------------------------------------------------------------
def test_bf16_rounding_matches_torch_cpu():
    import torch
    rng = np.random.default_rng(1)
    x = np.concatenate([
        rng.standard_normal(2000).astype(np.float32),
        (rng.standard_normal(500) * 1e-30).astype(np.float32),
        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 3.3895314e38,
                  np.inf, -np.inf, 65504.0, 1e-45], dtype=np.float32)])
    ours = orc.bf16_from_f32(x)
    theirs = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, theirs)


def test_reconstruct_values_are_enumerable_and_masked():
    rng = np.random.default_rng(2)
    m, n, n_q = 6, 50, 3
    planes = rng.integers(0, 2, (n_q, m, n), dtype=np.uint8)
    mask = (rng.random((m, n)) < 0.4).astype(np.uint8)
    alpha = rng.random((m, n_q)).astype(np.float32)
    w32, wbf = orc.reconstruct(planes, mask, alpha)
    assert np.all(w32[mask == 0] == 0)
    sign = planes.astype(np.float32) * 2 - 1                     # numpy float32 arithmetic, plane order
    acc = sign[0] * alpha[:, 0][:, None]
    for i in range(1, n_q):
        acc = (acc + sign[i] * alpha[:, i][:, None]).astype(np.float32)
    acc = np.where(mask == 1, acc, np.float32(0))
    assert np.array_equal(w32, acc)
    for r in range(m):
        assert len(set(np.abs(w32[r][mask[r] == 1]).tolist())) <= 2 ** (n_q - 1)
    import torch
    assert np.array_equal(wbf, torch.from_numpy(w32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))
    # one plane: exactly +-alpha
    w1, _ = orc.reconstruct(planes[:1], mask, alpha[:, :1])
    assert np.array_equal(np.abs(w1[mask == 1]), np.broadcast_to(alpha[:, :1], (m, n))[mask == 1])
    assert np.array_equal(w1[mask == 1] > 0, planes[0][mask == 1] == 1)


def test_matmul_special_case_is_a_plus_minus_one_matvec():
    rng = np.random.default_rng(3)
    m, n = 7, 33
    planes = rng.integers(0, 2, (1, m, n), dtype=np.uint8)
    X = rng.standard_normal((3, n))
    Y = orc.matmul(planes, np.ones((m, n), np.uint8), np.ones((m, 1), np.float32), X)
    W = planes[0].astype(np.float64) * 2 - 1
    assert np.allclose(Y, X @ W.T, rtol=0, atol=1e-12)


def test_matmul_general_case_against_numpy():
    rng = np.random.default_rng(4)
    m, n, n_q, batch = 9, 70, 3, 4
    planes = rng.integers(0, 2, (n_q, m, n), dtype=np.uint8)
    mask = (rng.random((m, n)) < 0.3).astype(np.uint8)
    alpha = rng.random((m, n_q)).astype(np.float32)
    X = rng.standard_normal((batch, n))
    W = ((planes.astype(np.float64) * 2 - 1) * alpha.astype(np.float64).T[:, :, None]).sum(axis=0) * mask
    Y = orc.matmul(planes, mask, alpha, X)
    assert Y.shape == (batch, m)
    assert np.allclose(Y, X @ W.T, rtol=1e-13, atol=1e-13)
    # dropping the mask changes the result (the mask really is applied)
    W_unmasked = ((planes.astype(np.float64) * 2 - 1) * alpha.astype(np.float64).T[:, :, None]).sum(axis=0)
    assert not np.allclose(Y, X @ W_unmasked.T)


# ---------------------------------------------------------------------------------------------
# Section 5.2, blocked n_patch assignment
# ---------------------------------------------------------------------------------------------
def _ceil_lg(v):
    v = np.asarray(v, dtype=np.float64)
    return np.where(v <= 1, 0.0, np.ceil(np.log2(np.maximum(v, 1))))


def test_blocked_npatch_hand_computed_and_limits():
    # six slices of 100 weights, n_in = 10: blocks of two have max p 1, 5, 3 -> widths 0, 3, 2 bits
    p = np.array([0, 1, 2, 5, 0, 3], dtype=np.uint16)
    b = orc.eq1_blocked(600, 100, 10, p, 2)
    assert b["bits_npatch"] == 2 * 0 + 2 * 3 + 2 * 2 and b["blocks"] == 3
    assert b["r"] == pytest.approx(600 / (60 + 10 + 11 * 7))
    # one block covering the plane is Eq. 1 itself
    whole = orc.eq1_blocked(600, 100, 10, p, 6)
    plain = orc.eq1(600, 100, 10, p)
    assert whole["bits_npatch"] == plain["bits_npatch"] == 6 * 3 and whole["r"] == pytest.approx(plain["r"])
    # blocks of one slice: every slice pays for its own count only
    rng = np.random.default_rng(11)
    q = rng.integers(0, 40, 997).astype(np.uint16)
    mn = 997 * 80 - 13                                   # ragged last slice, still 997 slices
    one = orc.eq1_blocked(mn, 80, 16, q, 1)
    assert one["bits_npatch"] == float(_ceil_lg(q).sum()) and one["blocks"] == 997
    # a finer blocking never needs more n_patch bits than a coarser one that it refines
    sizes = [997, 256, 64, 16, 4, 1]
    bits = [orc.eq1_blocked(mn, 80, 16, q, s)["bits_npatch"] for s in sizes]
    assert bits[0] == orc.eq1(mn, 80, 16, q)["bits_npatch"]
    assert all(bits[i + 1] <= bits[i] for i in range(1, len(bits) - 1))   # 256 | 64 | 16 | 4 | 1 refine one another
    assert max(bits[1:]) <= bits[0]


def test_blocked_npatch_helps_when_one_region_is_dense():
    # Section 5.2's case: a few slices with many care bits force a wide field on every slice
    p = np.zeros(1024, dtype=np.uint16)
    p[:8] = 37
    plain = orc.eq1(1024 * 100, 100, 10, p)
    blocked = orc.eq1_blocked(1024 * 100, 100, 10, p, 128)
    assert plain["bits_npatch"] == 1024 * 6
    assert blocked["bits_npatch"] == 128 * 6            # only the first block pays
    assert blocked["r"] > plain["r"]


# ---------------------------------------------------------------------------------------------
# Section 5.1, patch-data FIFO of one XOR-gate network
# ---------------------------------------------------------------------------------------------
def test_fifo_model_worked_example():
    # n_fifo = 2 banks, two entries arrive per cycle: slices with 0,1,2 patches take one cycle,
    # 5 patches take three, 3 patches take two; the FIFO never runs dry
    f = orc.fifo_model(np.array([0, 1, 2, 5, 0, 3], dtype=np.uint16), n_fifo=2, rate=2, depth=256)
    assert f["cycles"] == 1 + 1 + 1 + 3 + 1 + 2
    assert f["stall_bandwidth"] == 2 + 1 and f["stall_empty"] == 0 and f["stall_full"] == 0
    assert f["relative_time"] == pytest.approx(9 / 6)


def test_fifo_model_closed_forms():
    rng = np.random.default_rng(12)
    p = rng.poisson(0.8, 5000).astype(np.uint16)
    l = p.size
    # no patches at all: one slice per cycle
    z = orc.fifo_model(np.zeros(100, np.uint16), 1, 1, 4)
    assert z["cycles"] == 100 and z["stall_bandwidth"] == z["stall_empty"] == z["stall_full"] == 0
    # enough banks for the largest count and a stream that keeps up: no stall (relative time 1.0)
    big = orc.fifo_model(p, n_fifo=int(p.max()), rate=int(p.max()), depth=256)
    assert big["cycles"] == l and big["relative_time"] == 1.0
    # bank-limited only (stream as fast as the banks, FIFO deep enough): each slice costs
    # max(1, ceil(p / n_fifo)) cycles
    for banks in (1, 2, 3):
        f = orc.fifo_model(p, n_fifo=banks, rate=banks, depth=256)
        expect = int(np.maximum(1, -(-p.astype(np.int64) // banks)).sum())
        assert f["cycles"] == expect and f["stall_empty"] == 0
        assert f["stall_bandwidth"] == expect - l
    # more banks never cost cycles
    c = [orc.fifo_model(p, n_fifo=b, rate=b, depth=256)["cycles"] for b in (1, 2, 4, 8)]
    assert c == sorted(c, reverse=True) and c[-1] == l
    # stream-limited: two patches per slice but one entry per cycle arrives -> two cycles per slice
    s = orc.fifo_model(np.full(50, 2, np.uint16), n_fifo=4, rate=1, depth=256)
    assert s["cycles"] == 100 and s["stall_empty"] == 50 and s["stall_bandwidth"] == 0
    # lower bounds that hold for any setting
    for banks, rate, depth in ((1, 1, 2), (2, 1, 8), (3, 5, 4), (4, 2, 256)):
        f = orc.fifo_model(p, banks, rate, depth)
        total = int(p.sum())
        assert f["cycles"] >= max(l, -(-total // banks), -(-total // rate))
        assert f["peak"] <= depth
    # a stream faster than the patch logic fills a shallow FIFO and then waits
    full = orc.fifo_model(np.full(200, 1, np.uint16), n_fifo=1, rate=4, depth=8)
    assert full["cycles"] == 200 and full["stall_full"] > 0 and full["peak"] == 8


def test_csr_relative_time():
    assert orc.csr_relative_time([3, 3, 3, 3], 2) == 1.0              # no variation between rows
    assert orc.csr_relative_time([1, 5, 2, 2], 2) == pytest.approx((5 + 2) / (10 / 2))
    assert orc.csr_relative_time([1, 5, 2, 2], 1) == 1.0              # one row at a time: nothing waits
    rng = np.random.default_rng(13)
    nnz = rng.binomial(1000, 0.1, 512)
    t = orc.csr_relative_time(nnz, 32)
    groups = nnz.reshape(-1, 32)
    assert t == pytest.approx(groups.max(axis=1).sum() / (nnz.sum() / 32))
    assert t > 1.05                                                   # Section 5.1: CSR rows vary


def test_blocked_field_widths_that_can_hold_every_count():
    """Section 5.2 as a stored format: hand-computed widths ceil(lg(max p + 1)) per block."""
    p = np.array([0, 0, 1, 0, 3, 4, 0, 0, 0, 7, 8, 2, 1], dtype=np.uint16)
    # blocks of 4: max (1, 4, 8, 1) -> widths (1, 3, 4, 1) over (4, 4, 4, 1) slices
    assert orc.blocked_field_bits(p, 4) == {"bits_npatch": 4 * 1 + 4 * 3 + 4 * 4 + 1 * 1, "blocks": 4}
    # one block: max 8 needs 4 bits (Eq. 1's ceil(lg 8) = 3 could not hold the value 8)
    assert orc.blocked_field_bits(p, 100) == {"bits_npatch": 13 * 4, "blocks": 1}
    # blocks of one slice: 0 -> 0 bits, 1 -> 1, 2..3 -> 2, 4..7 -> 3, 8 -> 4
    assert orc.blocked_field_bits(p, 1)["bits_npatch"] == 0 + 0 + 1 + 0 + 2 + 3 + 0 + 0 + 0 + 3 + 4 + 2 + 1
    assert orc.blocked_field_bits(np.zeros(9, np.uint16), 2) == {"bits_npatch": 0, "blocks": 5}
    # never narrower than Eq. 1's literal width, and at most one bit wider per slice
    rng = np.random.default_rng(5)
    q = rng.poisson(2.0, 1000).astype(np.uint16)
    for block in (1, 7, 128, 1000):
        literal = orc.eq1_blocked(1000 * 80, 80, 16, q, block)["bits_npatch"]
        real = orc.blocked_field_bits(q, block)["bits_npatch"]
        assert literal <= real <= literal + 1000
