"""CPU tests of the C-ABI library's host side: exported symbols, the encoder against the
oracle's Algorithm 1 (logical arrays must be identical), blob packing / validation, stats."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import oracle as orc
from paper_1905_10138_b200 import sqnn
from paper_1905_10138_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def oracle_arrays(layer):
    """Per-plane (wc, np, dp) from the oracle's encoder."""
    care = layer.mask.ravel()
    return [orc.encode_plane(layer.M, layer.planes[i].ravel(), care) for i in range(layer.n_q)]


def library_blob(layer, flags=sqnn.ENCODE_ALG1):
    planes_words = np.concatenate([wl.pack_bits(layer.planes[i]) for i in range(layer.n_q)])
    return sqnn.sqnn_encode_host(wl.network_rows(layer.M), layer.n_in, layer.m, layer.n, layer.n_q,
                                 planes_words, wl.pack_bits(layer.mask), flags)


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "sqnn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(sqnn_[a-z_]+)\s*\(", text))
    assert {"sqnn_encode_host", "sqnn_decode", "sqnn_decode_matmul"} <= names
    L = sqnn.lib()
    for name in sorted(names):
        assert hasattr(L, name), name


def test_struct_layouts_match_the_header_sizes():
    # sizes computed by hand from include/sqnn.h (natural alignment)
    assert ctypes.sizeof(sqnn.Desc) == 4 * 8 + 4 * 4 + 4 * 4 + 3 * 8 + 4 * 8 * 8 + 8
    assert ctypes.sizeof(sqnn.Stats) == 8 + 64 + 32 + 32 + 8 + 16 * 8 + 16


LAYERS = [
    ("cfg1", lambda: wl.make_layer(1)),
    ("cfg2-small", lambda: wl.make_layer(2, m=96, n=1000)),
    ("cfg3-small", lambda: wl.make_layer(3, m=120, n=300)),
    ("cfg4-small", lambda: wl.make_layer(4, m=64, n=1030)),
    ("sweep-heavy", lambda: wl.make_sweep_layer(0, 3, m=64, n=1000)),     # S=0.6, (200,10): many patches
    ("sweep-80x16", lambda: wl.make_sweep_layer(1, 1, m=50, n=999)),
    ("sweep-40x16", lambda: wl.make_sweep_layer(3, 0, m=33, n=777)),
]


@pytest.mark.parametrize("name,make", LAYERS, ids=[n for n, _ in LAYERS])
def test_encoder_matches_oracle_algorithm1_bit_for_bit(name, make):
    layer = make()
    blob, stats = library_blob(layer)
    ref = oracle_arrays(layer)
    d = sqnn.sqnn_describe_host(blob)
    assert (d.m, d.n, d.n_q, d.n_out, d.n_in) == (layer.m, layer.n, layer.n_q, layer.n_out, layer.n_in)
    assert d.slices == (layer.mn + layer.n_out - 1) // layer.n_out
    eq1_bits = 0.0
    for i in range(layer.n_q):
        wc, np_, dp = sqnn.sqnn_unpack_host(blob, i)
        assert np.array_equal(wc.astype(np.uint64), ref[i][0])
        assert np.array_equal(np_, ref[i][1])
        assert np.array_equal(dp, ref[i][2])
        assert stats["patches"][i] == int(ref[i][1].sum())
        assert stats["max_patch"][i] == int(ref[i][1].max())
        e = orc.eq1(layer.mn, layer.n_out, layer.n_in, ref[i][1])
        eq1_bits += e["bits_wc"] + e["bits_npatch"] + e["bits_dpatch"]
    assert abs(stats["bpw_eq1"] - eq1_bits / layer.mn) < 1e-12
    stored = stats["bits_wc"] + stats["bits_npatch"] + stats["bits_dpatch"] + stats["bits_index"]
    assert abs(stats["bpw_actual"] - stored / layer.mn) < 1e-12
    # packing the oracle's arrays gives the very same bytes
    blob2 = sqnn.sqnn_pack_host(wl.network_rows(layer.M), layer.n_in, layer.m, layer.n,
                                [r[0].astype(np.uint32) for r in ref], [r[1] for r in ref], [r[2] for r in ref])
    assert np.array_equal(blob, blob2)


def test_exhaustive_encoder_matches_oracle_exhaustive():
    layer = wl.make_layer(1, m=40, n=100)
    blob, stats = library_blob(layer, sqnn.ENCODE_EXHAUSTIVE)
    wc, np_, dp = sqnn.sqnn_unpack_host(blob, 0)
    rwc, rnp, rdp = orc.encode_plane(layer.M, layer.planes[0].ravel(), layer.mask.ravel(), exhaustive=True)
    assert np.array_equal(wc.astype(np.uint64), rwc) and np.array_equal(np_, rnp) and np.array_equal(dp, rdp)
    _, stats_a = library_blob(layer)
    assert stats["patches"][0] <= stats_a["patches"][0]


def test_odd_network_shapes_and_tiny_layers():
    rng = np.random.default_rng(8)
    for (n_out, n_in, m, n) in [(13, 5, 7, 31), (1, 1, 3, 5), (256, 32, 9, 300), (33, 20, 40, 41), (64, 7, 1, 64)]:
        M = wl.xor_network(n_out, n_in, n_out * 100 + n_in)
        bits = rng.integers(0, 2, (m, n), dtype=np.uint8)
        mask = (rng.random((m, n)) < 0.3).astype(np.uint8)
        blob, _ = sqnn.sqnn_encode_host(wl.network_rows(M), n_in, m, n, 1, wl.pack_bits(bits), wl.pack_bits(mask))
        wc, np_, dp = sqnn.sqnn_unpack_host(blob, 0)
        rwc, rnp, rdp = orc.encode_plane(M, bits.ravel(), mask.ravel())
        assert np.array_equal(wc.astype(np.uint64), rwc) and np.array_equal(np_, rnp) and np.array_equal(dp, rdp)
        out = orc.decode_plane(M, m * n, rwc, rnp, rdp)
        assert np.array_equal(out[mask.ravel() == 1], bits.ravel()[mask.ravel() == 1])


def test_blob_layout_invariants():
    layer = wl.make_layer(3, m=60, n=300)
    blob, _ = library_blob(layer)
    d = sqnn.sqnn_describe_host(blob)
    assert d.total_bytes == blob.size and d.slices_padded % 1024 == 0 and d.tile_slices == 256
    tiles = d.slices_padded // 256
    for i in range(d.n_q):
        for off in (d.off_wc[i], d.off_idx[i], d.off_pp[i]):
            assert off % 16 == 0
        idx = blob[d.off_idx[i]: d.off_idx[i] + 4 * (tiles + 1)].view(np.uint32)
        _, np_, dp = sqnn.sqnn_unpack_host(blob, i)
        padded = np.zeros(d.slices_padded, np.int64)
        padded[: np_.size] = np_
        expect = np.concatenate([[0], np.cumsum(padded.reshape(-1, 256).sum(axis=1))])
        assert np.array_equal(idx.astype(np.int64), expect)
        assert idx[-1] == d.n_pp[i]
        # a stored entry is the bit position inside its tile: (slice in tile) * n_out + d_patch
        pp = blob[d.off_pp[i]: d.off_pp[i] + 2 * d.n_pp[i]].view(np.uint16)
        slice_of = np.repeat(np.arange(np_.size), np_)
        assert np.array_equal(pp.astype(np.int64), (slice_of % 256) * d.n_out + dp)
    rows = blob[d.off_xornet: d.off_xornet + 4 * d.n_out].view(np.uint32)
    assert np.array_equal(rows, wl.network_rows(layer.M))


def test_lookup_tables_in_the_blob_are_the_networks_outputs():
    """Entry (chunk, value) of the stored tables = M . (value placed at the chunk's bit positions), checked
    against the oracle's XOR network for every entry."""
    for cfg, m, n in ((1, 20, 80), (3, 10, 120), (4, 8, 160)):
        layer = wl.make_layer(cfg, m=m, n=n)
        blob, _ = library_blob(layer)
        d = sqnn.sqnn_describe_host(blob)
        tab = blob[d.off_tables: d.off_tables + d.tables_bytes].view(np.uint32)
        nwp, cb = d.tab_entry_words, d.tab_chunk_bits
        assert d.tab_chunks * cb >= d.n_in and nwp * 32 >= d.n_out
        rng = np.random.default_rng(cfg)
        for ch in range(d.tab_chunks):
            for v in rng.integers(0, 1 << cb, 64):
                seed = (int(v) << (ch * cb)) & ((1 << d.n_in) - 1)
                want = orc.xor_network(layer.M, [(seed >> t) & 1 for t in range(d.n_in)])
                e = tab[((ch << cb) | int(v)) * nwp: ((ch << cb) | int(v)) * nwp + nwp]
                got = wl.unpack_bits(e.astype(np.uint32).view(np.uint8), nwp * 32)
                assert np.array_equal(got[: d.n_out], want) and not got[d.n_out:].any()


def test_patch_histogram_counts_slices_by_n_patch():
    layer = wl.make_sweep_layer(0, 3, m=64, n=1000)           # ~35 patches per slice: the last bin fills
    blob, stats = library_blob(layer)
    _, np_, _ = sqnn.sqnn_unpack_host(blob, 0)
    want = np.bincount(np.minimum(np_, 15), minlength=16)
    assert stats["patch_hist"] == want.tolist() and sum(stats["patch_hist"]) == stats["slices"]
    light = wl.make_layer(2, m=96, n=1000)
    blob, stats = library_blob(light)
    _, np_, _ = sqnn.sqnn_unpack_host(blob, 0)
    assert stats["patch_hist"] == np.bincount(np.minimum(np_, 15), minlength=16).tolist()


def test_malformed_blobs_are_rejected_on_the_host():
    layer = wl.make_sweep_layer(1, 2, m=40, n=1000)           # has patches
    blob, _ = library_blob(layer)
    d = sqnn.sqnn_describe_host(blob)
    assert d.n_pp[0] > 1

    def bad(mutate):
        b = blob.copy()
        mutate(b)
        with pytest.raises(sqnn.SqnnError) as e:
            sqnn.sqnn_describe_host(b)
        assert e.value.status == sqnn.E_BAD_BLOB

    def set_u16(b, off, v):
        b[off: off + 2] = np.frombuffer(np.uint16(v).tobytes(), dtype=np.uint8)

    pp0 = int(d.off_pp[0])
    first, second = (int(v) for v in blob[pp0: pp0 + 4].view(np.uint16))
    bad(lambda b: b.__setitem__(0, b[0] ^ 1))                                  # magic
    bad(lambda b: b.__setitem__(8, 9))                                         # version
    bad(lambda b: set_u16(b, pp0, 256 * d.n_out))                              # position outside the tile
    bad(lambda b: set_u16(b, pp0 + 2, first))                                  # not ascending inside the tile
    bad(lambda b: b.__setitem__(int(d.off_idx[0]) + 4, b[int(d.off_idx[0]) + 4] ^ 1))   # tile offsets
    bad(lambda b: b.__setitem__(int(d.off_tables) + 5, b[int(d.off_tables) + 5] ^ 2))   # a table entry
    bad(lambda b: b.__setitem__(int(d.off_wc[0]) + (d.slices * d.n_in + 7) // 8 + 1, 1))   # a padding slice with a seed
    with pytest.raises(sqnn.SqnnError):
        sqnn.sqnn_describe_host(blob[:-16])                                    # truncated
    with pytest.raises(sqnn.SqnnError):
        sqnn.sqnn_describe_host(blob[:100])
    hdr = blob.copy()
    hdr[16:24] = np.frombuffer(np.uint64(1 << 50).tobytes(), dtype=np.uint8)   # absurd m
    with pytest.raises(sqnn.SqnnError):
        sqnn.sqnn_describe_host(hdr)
    assert second > first


def test_invalid_arguments_return_codes_not_crashes():
    M = wl.xor_network(8, 4, 1)
    rows = wl.network_rows(M)
    bits = np.zeros(64, np.uint8)
    with pytest.raises(sqnn.SqnnError) as e:
        sqnn.sqnn_encode_host(rows, 40, 8, 8, 1, wl.pack_bits(bits), wl.pack_bits(bits))     # n_in > 32
    assert e.value.status == sqnn.E_INVALID_ARG
    with pytest.raises(sqnn.SqnnError):
        sqnn.sqnn_encode_host(rows, 4, 8, 8, 9, np.zeros(9, np.uint64), wl.pack_bits(bits))  # n_q > 8
    with pytest.raises(sqnn.SqnnError):      # seed does not fit n_in bits
        sqnn.sqnn_pack_host(rows, 4, 1, 8, [np.array([16], np.uint32)], [np.array([0], np.uint16)],
                            [np.zeros(0, np.uint16)])
    with pytest.raises(sqnn.SqnnError):      # patch position >= n_out
        sqnn.sqnn_pack_host(rows, 4, 1, 8, [np.array([3], np.uint32)], [np.array([1], np.uint16)],
                            [np.array([8], np.uint16)])
    with pytest.raises(sqnn.SqnnError):      # positions of a slice must ascend
        sqnn.sqnn_pack_host(rows, 4, 1, 8, [np.array([3], np.uint32)], [np.array([2], np.uint16)],
                            [np.array([5, 2], np.uint16)])
    assert sqnn.status_string(0) == "ok" and "unknown" in sqnn.status_string(-99)


def test_device_entry_points_reject_bad_arguments_without_a_gpu():
    layer = wl.make_layer(1, m=16, n=80)
    blob, _ = library_blob(layer)
    d = sqnn.sqnn_describe_host(blob)
    L = sqnn.lib()
    # NULL blob / NULL output are refused before any CUDA call
    assert L.sqnn_decode(ctypes.byref(d), None, None, None, 0, None, 0, None, None) == sqnn.E_INVALID_ARG
    assert L.sqnn_decode(ctypes.byref(d), ctypes.c_void_p(16), None, None, 0, None, 0, None, None) == sqnn.E_INVALID_ARG
    assert L.sqnn_decode(ctypes.byref(d), ctypes.c_void_p(24), None, None, 0, ctypes.c_void_p(16), 1 << 20,
                         None, None) == sqnn.E_INVALID_ARG                      # misaligned blob
    assert L.sqnn_decode(ctypes.byref(d), ctypes.c_void_p(32), None, None, 0, ctypes.c_void_p(16), 8,
                         None, None) == sqnn.E_INVALID_ARG                      # out too small
    assert L.sqnn_decode_matmul(ctypes.byref(d), ctypes.c_void_p(32), None, None, None, 0, 1, 80, None, 16,
                                None, 0, None, None) == sqnn.E_INVALID_ARG
    assert sqnn.sqnn_workspace_bytes(d, 1) == 0
    assert sqnn.sqnn_workspace_bytes(d, 16) >= (16 * 80 + 63) // 64 * 8


@pytest.mark.parametrize("name,make", LAYERS[:5], ids=[n for n, _ in LAYERS[:5]])
def test_blocked_npatch_accounting_matches_the_oracle(name, make):
    """Section 5.2: per-block n_patch widths, library (from the blob) against the oracle (from its own arrays)."""
    layer = make()
    blob, stats = library_blob(layer)
    ref = oracle_arrays(layer)
    l = (layer.mn + layer.n_out - 1) // layer.n_out
    for block in (1, 7, 128, l, 10 * l):
        got = sqnn.sqnn_stats_blocked_host(blob, block)
        per_plane = [orc.eq1_blocked(layer.mn, layer.n_out, layer.n_in, a[1], block) for a in ref]
        assert got["bits_npatch"] == sum(int(p["bits_npatch"]) for p in per_plane)
        assert got["bpw_eq1"] == pytest.approx(sum(p["bits_per_weight"] for p in per_plane), rel=1e-12)
    # one block per plane is the plain Eq. 1 figure
    assert sqnn.sqnn_stats_blocked_host(blob, l)["bpw_eq1"] == pytest.approx(stats["bpw_eq1"], rel=1e-12)
    with pytest.raises(sqnn.SqnnError):
        sqnn.sqnn_stats_blocked_host(blob, 0)


def test_fifo_model_matches_the_oracle():
    """Section 5.1: the library's cycle model against the oracle's on encoder output and on random counts."""
    rng = np.random.default_rng(77)
    cases = [oracle_arrays(wl.make_sweep_layer(0, 3, m=64, n=1000))[0][1],      # heavy patch load
             oracle_arrays(wl.make_layer(2, m=96, n=1000))[0][1],
             rng.poisson(3.0, 4000).astype(np.uint16), np.zeros(17, np.uint16), np.zeros(0, np.uint16)]
    for counts in cases:
        for n_fifo, rate, depth in ((1, 1, 4), (2, 2, 256), (4, 1, 16), (3, 7, 5), (8, 8, 256)):
            got = sqnn.sqnn_fifo_model_host(counts, n_fifo, rate, depth)
            ref = orc.fifo_model(counts, n_fifo, rate, depth)
            for key in ("cycles", "stall_bandwidth", "stall_empty", "stall_full", "peak"):
                assert got[key] == ref[key], (key, n_fifo, rate, depth)
    with pytest.raises(sqnn.SqnnError):
        sqnn.sqnn_fifo_model_host(cases[0], 0, 1, 1)


@pytest.mark.parametrize("name,make", LAYERS[:6], ids=[n for n, _ in LAYERS[:6]])
def test_storage_form_with_blocked_npatch_widths_round_trips(name, make):
    """Section 5.2 as a format: per-block field widths, sizes against the oracle's accounting, and the device
    blob rebuilt byte for byte."""
    layer = make()
    blob, stats = library_blob(layer)
    ref = oracle_arrays(layer)
    l = (layer.mn + layer.n_out - 1) // layer.n_out
    lg_n_out = int(np.ceil(np.log2(layer.n_out)))
    for block in (1, 16, 128, l, 3 * l):
        stored, info = sqnn.sqnn_store_host(blob, block)
        want = [orc.blocked_field_bits(a[1], block) for a in ref]
        assert info["bits_npatch"] == sum(w["bits_npatch"] for w in want)
        assert info["bits_widths"] == 8 * sum(w["blocks"] for w in want)
        assert info["bits_wc"] == layer.n_q * l * layer.n_in
        assert info["bits_dpatch"] == sum(int(a[1].sum()) for a in ref) * lg_n_out
        assert info["total_bytes"] == stored.size
        assert info["bpw"] == pytest.approx((info["bits_wc"] + info["bits_widths"] + info["bits_npatch"] +
                                             info["bits_dpatch"]) / layer.mn)
        assert np.array_equal(sqnn.sqnn_load_host(stored), blob)
    with pytest.raises(sqnn.SqnnError):
        sqnn.sqnn_store_host(blob, 0)


def test_storage_form_dense_region_case_and_rejection_of_damaged_buffers():
    """Section 5.2's motivating case: patches concentrated in one region.  One field width for the whole plane
    pays for the worst slice everywhere; per-block widths pay only where the patches are (blocks without
    patches take no n_patch bits at all)."""
    n_out, n_in, l = 100, 10, 2048
    rng = np.random.default_rng(3)
    M = wl.xor_network(n_out, n_in, 77)
    wc = rng.integers(0, 1 << n_in, l).astype(np.uint32)
    counts = np.zeros(l, dtype=np.uint16)
    counts[512:640] = rng.integers(1, 8, 128)                  # one busy block of 128 slices
    dp = np.concatenate([np.sort(rng.choice(n_out, c, replace=False)) for c in counts if c]).astype(np.uint16)
    blob = sqnn.sqnn_pack_host(wl.network_rows(M), n_in, l, n_out, [wc], [counts], [dp])
    whole, info_whole = sqnn.sqnn_store_host(blob, l)
    blocked, info_blocked = sqnn.sqnn_store_host(blob, 128)
    assert info_whole["bits_npatch"] == l * 3                   # max 7 -> 3 bits for every slice
    assert info_blocked["bits_npatch"] == 128 * 3               # only the busy block stores counts
    assert info_blocked["bits_npatch"] == orc.blocked_field_bits(counts, 128)["bits_npatch"]
    assert info_blocked["bits_widths"] == 8 * 16
    assert blocked.size < whole.size
    for stored in (whole, blocked):
        assert np.array_equal(sqnn.sqnn_load_host(stored), blob)
    # damaged buffers: magic, truncated, a width byte that no longer matches the counts, trailing bytes
    def bad(buf):
        with pytest.raises(sqnn.SqnnError) as e:
            sqnn.sqnn_load_host(buf)
        assert e.value.status == sqnn.E_BAD_BLOB
    b = blocked.copy(); b[0] ^= 1; bad(b)
    bad(blocked[:-3])
    bad(np.concatenate([blocked, np.zeros(4, np.uint8)]))
    widths_at = 128 + 4 * n_out + (l * n_in + 7) // 8           # header, rows of M, seed stream
    b = blocked.copy(); b[widths_at + 4] = 0; bad(b)            # the busy block's width set to 0: counts no longer add up
    b = blocked.copy(); b[widths_at + 4] = 12; bad(b)           # a width no count needs
    # a header that claims far more rows than the buffer could hold seeds for is refused before anything of
    # that size is allocated (m is the first 64-bit field after the magic)
    import time
    b = blocked.copy()
    b[8 + 3] |= 0x40                                            # m += 2^30: 10^9 slices claimed
    t0 = time.perf_counter()
    bad(b)
    assert time.perf_counter() - t0 < 1.0
