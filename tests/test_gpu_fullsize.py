"""GPU parity at the benchmark's full sizes.  The oracle cannot decode or multiply a whole layer
in test time, so the checks are (a) properties that hold at any size -- every care bit of every
plane comes back -- and (b) the oracle run on samples: randomly chosen slices are encrypted and
decrypted by the oracle and compared bit for bit (don't-care positions included) with what the
library's encoder stored and what the GPU decoded; randomly chosen rows of the product are
recomputed by the oracle in fp64 (the product depends on care bits only, which (a) shows to be
the layer's own bits)."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_1905_10138_b200 import sqnn
from paper_1905_10138_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def check_decode_on_samples(layer, dev, blob, n_samples=150, seed=0):
    words = dev.decode_bits()
    rng = np.random.default_rng(seed)
    l = (layer.mn + layer.n_out - 1) // layer.n_out
    picks = np.unique(np.concatenate([[0, l - 1, l // 2], rng.integers(0, l, n_samples)]))
    mask_flat = layer.mask.ravel()
    for i in range(layer.n_q):
        got = wl.unpack_bits(words[i], layer.mn)
        want = layer.planes[i].ravel()
        care = mask_flat == 1
        assert np.array_equal(got[care], want[care]), f"plane {i}: a care bit was not reproduced"
        wc, np_, dp = sqnn.sqnn_unpack_host(blob, i)
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
            o_bits = orc.decode_slice(layer.M, o_wc, o_dp)
            assert np.array_equal(got[lo:hi], o_bits[: hi - lo]), f"plane {i} slice {s}"
    assert dev.status_value() == 0
    return words


def check_product_on_sampled_rows(layer, dev, batch, tol, n_rows=24, seed=1):
    import torch
    rng = np.random.default_rng(seed)
    rows = np.unique(np.concatenate([[0, layer.m - 1], rng.integers(0, layer.m, n_rows)]))
    x = layer.activations(batch)
    y = dev.matmul(x, torch.float32 if layer.x_dtype == "f32" else torch.bfloat16)
    ref = orc.matmul(np.ascontiguousarray(layer.planes[:, rows, :]), np.ascontiguousarray(layer.mask[rows]),
                     np.ascontiguousarray(layer.alpha[rows]), x.astype(np.float64))
    assert np.all(np.isfinite(y))
    err = H.rel_err(y[:, rows], ref)
    assert err <= tol, (batch, err)
    assert dev.status_value() == 0


@pytest.mark.parametrize("cfg,gemv_batches,mma_batches", [(2, (1,), (64,)), (3, (1, 8), (32,)), (4, (), (16, 128))],
                         ids=["cfg2", "cfg3", "cfg4"])
def test_full_size_layers(cfg, gemv_batches, mma_batches):
    layer = wl.make_layer(cfg)
    blob, stats = H.blob_from_library(layer)
    dev = H.DeviceLayer(layer, blob)
    check_decode_on_samples(layer, dev, blob, n_samples=60)
    for b in gemv_batches:
        check_product_on_sampled_rows(layer, dev, b, 1e-4)
    for b in mma_batches:
        check_product_on_sampled_rows(layer, dev, b, 1e-2)


def test_full_size_decode_sweep_point_2p30_weights():
    """The benchmark's decode-only point: 2^30 weights, M 100 x 10, S = 0.9."""
    layer = wl.make_sweep_layer(2, 2)
    blob, stats = H.blob_from_library(layer)
    dev = H.DeviceLayer(layer, blob)
    words = check_decode_on_samples(layer, dev, blob, n_samples=100)
    sink = int(np.bitwise_xor.reduce(words[0]))
    assert dev.decode_sink() == sink
    # bf16 output on sampled rows
    import torch
    out = torch.empty((layer.m, layer.n), dtype=torch.bfloat16, device="cuda")
    sqnn.sqnn_decode(dev.desc, dev.blob, dev.mask, dev.alpha, sqnn.OUT_BF16, out, dev.status)
    torch.cuda.synchronize()
    rows = np.array([0, 1, 12345, layer.m - 1])
    got = out[torch.from_numpy(rows).cuda()].view(torch.int16).cpu().numpy().view(np.uint16)
    bits = wl.unpack_bits(words[0], layer.mn).reshape(layer.m, layer.n)[rows]
    _, want = orc.reconstruct(bits[None], layer.mask[rows], layer.alpha[rows], want_f32=False)
    assert np.array_equal(got, want)
    assert dev.status_value() == 0
