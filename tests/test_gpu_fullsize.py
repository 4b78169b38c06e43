"""GPU parity at the benchmark's full sizes, in the launch configurations the benchmark times.

The oracle's *encoder* (a full elimination per care bit) is too slow for whole layers, its decoder
and its fp64 product are not.  So every full-size layer is encoded by the library, the library's
logical arrays (``sqnn_unpack_host``) are decoded by the oracle over *all* slices, and the GPU's
decoded planes must equal that bit for bit -- don't-care positions included -- while every care bit
must be the layer's own bit (Section 3.2: the patches make the format lossless).  The library's
encoder itself is held against the oracle's Algorithm 1 on sampled slices.  Products are compared
with the oracle's fp64 product over all rows at every batch size the configurations name.

Layers of 67 M weights and more give every warp of the decode kernel several tiles, so these cases
also cover its steady-state loop (fetches two tiles ahead, bulk store of tile t under tile t + 1);
``test_decode_loop_with_many_tiles_per_warp_run_time_shape`` does the same for the run-time-shape
kernel."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_1905_10138_b200 import sqnn
from paper_1905_10138_b200 import workloads as wl
from tests import helpers as H
from tests.test_gpu_decode import generic_layer

pytestmark = pytest.mark.gpu


def check_whole_decode(layer, dev, blob, n_samples=40, seed=0):
    """Returns the oracle-decoded planes uint8 [n_q, m, n] after checking the GPU's against them."""
    words = dev.decode_bits()
    mask_flat = layer.mask.ravel()
    care = mask_flat == 1
    rng = np.random.default_rng(seed)
    l = (layer.mn + layer.n_out - 1) // layer.n_out
    picks = np.unique(np.concatenate([[0, l - 1, l // 2], rng.integers(0, l, n_samples)]))
    ref = np.empty((layer.n_q, layer.m, layer.n), dtype=np.uint8)
    for i in range(layer.n_q):
        wc, np_, dp = sqnn.sqnn_unpack_host(blob, i)
        bits = orc.decode_plane(layer.M, layer.mn, wc.astype(np.uint64), np_, dp)      # all slices
        assert np.array_equal(words[i], wl.pack_bits(bits)), f"plane {i}: decoded bits differ from the oracle's"
        want = layer.planes[i].ravel()
        assert np.array_equal(bits[care], want[care]), f"plane {i}: a care bit was not reproduced"
        ref[i] = bits.reshape(layer.m, layer.n)
        # the stored seeds and patches are what the oracle's Algorithm 1 gives for the same slices
        starts = np.concatenate([[0], np.cumsum(np_.astype(np.int64))])
        for s in picks:
            lo, hi = s * layer.n_out, min(layer.mn, (s + 1) * layer.n_out)
            wq = np.zeros(layer.n_out, np.uint8)
            cr = np.zeros(layer.n_out, np.uint8)
            wq[: hi - lo] = want[lo:hi]
            cr[: hi - lo] = mask_flat[lo:hi]
            o_wc, o_dp = orc.encode_slice(layer.M, wq, cr)
            assert int(sum(int(b) << t for t, b in enumerate(o_wc))) == int(wc[s])
            assert np.array_equal(dp[starts[s]:starts[s + 1]], o_dp)
    assert dev.status_value() == 0
    return ref


def check_whole_product(layer, dev, ref_bits, batch, tol):
    import torch
    x = layer.activations(batch)
    y = dev.matmul(x, torch.float32 if layer.x_dtype == "f32" else torch.bfloat16)
    want = orc.matmul(ref_bits, layer.mask, layer.alpha, x.astype(np.float64))            # all rows
    assert y.shape == want.shape and np.all(np.isfinite(y))
    err = H.rel_err(y, want)
    assert err <= tol, (layer.name, batch, err)
    assert dev.status_value() == 0


@pytest.mark.parametrize("cfg,gemv_batches,mma_batches",
                         [(1, (1,), ()), (2, (1,), (64,)), (3, (1, 8), (32,)), (4, (), (16, 128, 512))],
                         ids=["cfg1", "cfg2", "cfg3", "cfg4"])
def test_full_size_layers_every_bit_and_every_row(cfg, gemv_batches, mma_batches):
    layer = wl.make_layer(cfg)
    blob, stats = H.blob_from_library(layer)
    dev = H.DeviceLayer(layer, blob)
    ref = check_whole_decode(layer, dev, blob)
    for b in gemv_batches:
        check_whole_product(layer, dev, ref, b, 1e-4)
    for b in mma_batches:
        check_whole_product(layer, dev, ref, b, 1e-2)
    # bf16 output of the whole layer
    _, want = orc.reconstruct(ref, layer.mask, layer.alpha, want_f32=False)
    assert np.array_equal(dev.decode_bf16(), want)


SWEEP_CORNERS = [(0, 0), (0, 3), (3, 0), (3, 3), (2, 2)]     # the four corners and the headline point


@pytest.mark.parametrize("i_s,i_m", SWEEP_CORNERS, ids=[f"S{wl.SWEEP_PRUNE[a]:.2f}-{wl.SWEEP_NETS[b][0]}x{wl.SWEEP_NETS[b][1]}"
                                                        for a, b in SWEEP_CORNERS])
def test_full_size_decode_sweep_points_2p30_weights(i_s, i_m):
    """Decode-only points of the benchmark at 2^30 weights: every bit against the oracle, the checksum
    sink, and (headline point) bf16 output on sampled rows."""
    layer = wl.make_sweep_layer(i_s, i_m)
    blob, stats = H.blob_from_library(layer)
    dev = H.DeviceLayer(layer, blob)
    ref = check_whole_decode(layer, dev, blob, n_samples=30)
    sink = int(np.bitwise_xor.reduce(wl.pack_bits(ref[0])))
    assert dev.decode_sink() == sink
    if (i_s, i_m) == (2, 2):
        import torch
        out = torch.empty((layer.m, layer.n), dtype=torch.bfloat16, device="cuda")
        sqnn.sqnn_decode(dev.desc, dev.blob, dev.mask, dev.alpha, sqnn.OUT_BF16, out, dev.status)
        torch.cuda.synchronize()
        rows = np.array([0, 1, 12345, layer.m - 1])
        got = out[torch.from_numpy(rows).cuda()].view(torch.int16).cpu().numpy().view(np.uint16)
        _, want = orc.reconstruct(np.ascontiguousarray(ref[:, rows, :]), np.ascontiguousarray(layer.mask[rows]),
                                  np.ascontiguousarray(layer.alpha[rows]), want_f32=False)
        assert np.array_equal(got, want)
    assert dev.status_value() == 0


def test_decode_loop_with_many_tiles_per_warp_run_time_shape():
    """A network shape without a compile-time kernel (12 x 5), large enough that every warp of the
    run-time-shape decode kernel loops over four and more tiles; compared in full."""
    layer = generic_layer(12, 5, 4096, 12000, 0.2, 51)         # 49 M weights, 16 000 kernel tiles of 3072 bits
    blob, _ = H.blob_from_library(layer)
    dev = H.DeviceLayer(layer, blob)
    check_whole_decode(layer, dev, blob, n_samples=20)
