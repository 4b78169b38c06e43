"""GPU parity: the CUDA decode kernels against the CPU oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_1905_10138_b200 import sqnn
from paper_1905_10138_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu

SMALL = [
    ("cfg1", lambda: wl.make_layer(1)),                                   # 820 slices, ragged last slice
    ("cfg2-s", lambda: wl.make_layer(2, m=37, n=9216)),                   # 13.3 warp tiles, rows straddle slices
    ("cfg3-s", lambda: wl.make_layer(3, m=203, n=3000)),                  # 2 planes
    ("cfg4-s", lambda: wl.make_layer(4, m=41, n=16384)),                  # 3 planes
    ("sw-40x16-S60", lambda: wl.make_sweep_layer(0, 0, m=61, n=4099)),
    ("sw-80x16-S60", lambda: wl.make_sweep_layer(0, 1, m=61, n=4099)),
    ("sw-100x10-S60", lambda: wl.make_sweep_layer(0, 2, m=61, n=4099)),   # ~15 patches per slice
    ("sw-200x10-S60", lambda: wl.make_sweep_layer(0, 3, m=61, n=4099)),   # ~35 patches per slice
    ("sw-100x10-S90", lambda: wl.make_sweep_layer(2, 2, m=129, n=4001)),
    ("sw-200x10-S95", lambda: wl.make_sweep_layer(3, 3, m=129, n=4001)),
    ("sw-40x16-S95", lambda: wl.make_sweep_layer(3, 0, m=129, n=4001)),   # no patches at all
]


def generic_layer(n_out, n_in, m, n, keep, seed, n_q=1):
    """A layer with an arbitrary network shape (exercises the run-time-shape kernels)."""
    rng = np.random.default_rng(seed)
    planes = rng.integers(0, 2, (n_q, m, n), dtype=np.uint8)
    mask = (rng.random((m, n)) < keep).astype(np.uint8)
    alpha = (rng.random((m, n_q)) + 0.5).astype(np.float32)
    return wl.Layer(name=f"gen-{n_out}x{n_in}", cfg=0, m=m, n=n, n_q=n_q, n_out=n_out, n_in=n_in,
                    prune_rate=1 - keep, M=wl.xor_network(n_out, n_in, seed + 1), planes=planes, mask=mask,
                    alpha=alpha, x_dtype="f32", batches=(1,), seed_x=seed + 2)


GENERIC = [
    ("gen-13x5", lambda: generic_layer(13, 5, 57, 1001, 0.3, 11)),
    ("gen-256x32", lambda: generic_layer(256, 32, 64, 3000, 0.15, 12)),
    ("gen-33x20", lambda: generic_layer(33, 20, 31, 2049, 0.5, 13, n_q=2)),
    ("gen-64x7", lambda: generic_layer(64, 7, 16, 4096, 0.2, 14)),
    ("gen-1x1", lambda: generic_layer(1, 1, 5, 77, 0.5, 15)),
    ("gen-96x9-q8", lambda: generic_layer(96, 9, 20, 999, 0.1, 16, n_q=8)),
    ("gen-tiny", lambda: generic_layer(100, 10, 1, 3, 1.0, 17)),
    # patch runs of 300-600 entries per tile: three and four rounds of the single-window patch step, and tiles on
    # either side of its 512-byte limit in the same layer (the longer ones take the windowed form)
    ("gen-100x10-keep12", lambda: generic_layer(100, 10, 129, 4001, 0.12, 31)),
    ("gen-100x10-keep135", lambda: generic_layer(100, 10, 129, 4001, 0.135, 32)),
    ("gen-60x12-keep255-q2", lambda: generic_layer(60, 12, 77, 3000, 0.255, 33, n_q=2)),
]


@pytest.mark.parametrize("name,make", SMALL + GENERIC, ids=[n for n, _ in SMALL + GENERIC])
def test_decode_bits_sink_and_bf16_match_oracle_exactly(name, make):
    layer = make()
    arrays = H.oracle_encode(layer)
    ref_bits = H.oracle_decode(layer, arrays)
    dev = H.DeviceLayer(layer, H.blob_from_oracle(layer, arrays))
    # packed bits: every position, don't-cares included; bits past mn in the last word are zero
    got = dev.decode_bits()
    for i in range(layer.n_q):
        assert np.array_equal(got[i], wl.pack_bits(ref_bits[i])), (name, i)
    # checksum sink
    expect_sink = 0
    for i in range(layer.n_q):
        expect_sink ^= int(np.bitwise_xor.reduce(wl.pack_bits(ref_bits[i])))
    assert dev.decode_sink() == expect_sink
    # masked, rescaled bf16 weights
    _, ref_bf16 = orc.reconstruct(ref_bits, layer.mask, layer.alpha, want_f32=False)
    assert np.array_equal(dev.decode_bf16(), ref_bf16)
    assert dev.status_value() == 0


def test_library_encoded_blob_decodes_to_the_same_bits():
    layer = wl.make_layer(3, m=203, n=3000)
    blob, _ = H.blob_from_library(layer)
    dev = H.DeviceLayer(layer, blob)
    got = dev.decode_bits()
    ref = H.oracle_decode(layer, H.oracle_encode(layer))
    for i in range(layer.n_q):
        assert np.array_equal(got[i], wl.pack_bits(ref[i]))


def test_layer_restored_from_the_storage_form_with_mixed_block_widths_decodes_bit_exactly():
    """Section 5.2: a layer whose blocks of 128 slices need different n_patch widths (0 bits where a region
    is fully pruned) goes through the storage form and back, then through the GPU decoder."""
    rng = np.random.default_rng(61)
    m, n = 96, 4000
    keep = np.concatenate([np.zeros(32), np.full(32, 0.35), np.full(32, 0.04)])          # per row
    mask = (rng.random((m, n)) < keep[:, None]).astype(np.uint8)
    planes = rng.integers(0, 2, (1, m, n), dtype=np.uint8)
    layer = wl.Layer(name="mixed", cfg=0, m=m, n=n, n_q=1, n_out=100, n_in=10, prune_rate=0.0,
                     M=wl.xor_network(100, 10, 62), planes=planes, mask=mask,
                     alpha=np.ones((m, 1), np.float32), x_dtype="f32", batches=(1,), seed_x=63)
    blob, _ = H.blob_from_library(layer)
    _, np_, _ = sqnn.sqnn_unpack_host(blob, 0)
    per_block = [int(np_[a:a + 128].max()) for a in range(0, np_.size, 128)]
    widths = {int(np.ceil(np.log2(p + 1))) for p in per_block}
    assert 0 in widths and len(widths) >= 3
    stored, info = sqnn.sqnn_store_host(blob, 128)
    assert info["bits_npatch"] == orc.blocked_field_bits(np_, 128)["bits_npatch"] < np_.size * max(widths)
    restored = sqnn.sqnn_load_host(stored)
    assert np.array_equal(restored, blob)
    dev = H.DeviceLayer(layer, restored)
    ref = H.oracle_decode(layer, H.oracle_encode(layer))
    assert np.array_equal(dev.decode_bits()[0], wl.pack_bits(ref[0]))
    assert dev.status_value() == 0


def test_malformed_device_patch_entries_set_the_status_word_and_do_not_fault():
    """The host validator rejects such blobs; if a device copy is damaged anyway the kernel
    skips the entry and reports through the status word."""
    import torch
    layer = wl.make_sweep_layer(1, 2, m=40, n=1000)
    blob, _ = H.blob_from_library(layer)
    dev = H.DeviceLayer(layer, blob)
    d = dev.desc
    assert d.n_pp[0] > 0
    clean = dev.decode_bits()
    assert dev.status_value() == 0
    dev.blob[int(d.off_pp[0]) + 1] = 255                 # first entry becomes >= 65280 > 256 * n_out
    torch.cuda.synchronize()
    damaged = dev.decode_bits()
    assert dev.status_value() == 1
    diff = np.bitwise_xor(clean, damaged)
    assert sum(bin(int(w)).count("1") for w in diff.ravel()) == 1      # exactly the skipped flip


def test_output_buffer_size_and_alignment_are_checked():
    import torch
    layer = wl.make_layer(1, m=16, n=80)
    blob, _ = H.blob_from_library(layer)
    dev = H.DeviceLayer(layer, blob)
    small = torch.zeros(1, dtype=torch.int64, device="cuda")
    with pytest.raises(sqnn.SqnnError) as e:
        sqnn.sqnn_decode(dev.desc, dev.blob, None, None, sqnn.OUT_BITS, small)
    assert e.value.status == sqnn.E_INVALID_ARG
    with pytest.raises(sqnn.SqnnError):
        sqnn.sqnn_decode(dev.desc, dev.blob, None, None, sqnn.OUT_BF16,
                         torch.zeros(16 * 80, dtype=torch.bfloat16, device="cuda"))   # mask / alpha missing
