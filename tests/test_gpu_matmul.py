"""GPU parity: fused decode + product against the oracle's fp64 product, through the C ABI."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_1905_10138_b200 import workloads as wl
from tests import helpers as H
from tests.test_gpu_decode import generic_layer

pytestmark = pytest.mark.gpu

# Tolerances (max |y - y_ref| / max(|y_ref|, rms(y_ref))):
#  1e-4: fp32 accumulation of exact weights (GEMV path, batch <= 15)
#  1e-2: weights rounded to bf16 (tensor-core path, batch >= 16)
TOL_F32 = 1e-4
TOL_BF16 = 1e-2


def reference(layer, x):
    """The product depends on care bits only, and those are reproduced exactly (checked by the
    decode parity tests), so the oracle's product runs on the oracle-decoded planes."""
    ref_bits = H.oracle_decode(layer, H.oracle_encode(layer))
    return orc.matmul(ref_bits, layer.mask, layer.alpha, x.astype(np.float64))


GEMV = [
    ("cfg1-b1-f32", lambda: wl.make_layer(1), "f32", 1),
    ("cfg2-s-b1", lambda: wl.make_layer(2, m=37, n=9216), "bf16", 1),
    ("cfg3-s-b1", lambda: wl.make_layer(3, m=203, n=3000), "bf16", 1),
    ("cfg3-s-b8", lambda: wl.make_layer(3, m=203, n=3000), "bf16", 8),
    ("cfg4-s-b3", lambda: wl.make_layer(4, m=41, n=16384), "bf16", 3),
    ("cfg4-s-b15-f32", lambda: wl.make_layer(4, m=41, n=16384), "f32", 15),
    ("gen-13x5-b2", lambda: generic_layer(13, 5, 57, 1001, 0.3, 11), "f32", 2),
    ("gen-33x20-q2-b5", lambda: generic_layer(33, 20, 31, 2049, 0.5, 13, n_q=2), "bf16", 5),
    ("gen-narrow-n", lambda: generic_layer(40, 12, 300, 17, 0.4, 21), "f32", 4),        # rows shorter than a word
    ("gen-empty-rows", lambda: generic_layer(100, 10, 64, 500, 0.0, 22), "f32", 1),     # everything pruned
    # four and more planes (scales and plane words not held in registers) and rows too long for the
    # activations to be staged on chip: the plain C++ form of the walk
    ("gen-60x12-q5-b3", lambda: generic_layer(60, 12, 40, 3000, 0.2, 41, n_q=5), "bf16", 3),
    ("gen-long-rows-b2", lambda: generic_layer(40, 12, 5, 100003, 0.1, 42), "bf16", 2),
    ("gen-long-rows-f32-b1", lambda: generic_layer(100, 10, 3, 50001, 0.1, 43), "f32", 1),
    # patch runs on both sides of the single-window limit of the patch step
    ("gen-100x10-keep135", lambda: generic_layer(100, 10, 129, 4001, 0.135, 32), "f32", 2),
    # 828 warp tiles: five to six per SM, three warps share a tile and take its row segments in turn
    ("cfg2-2300rows-b1", lambda: wl.make_layer(2, m=2300, n=9216), "bf16", 1),
]


@pytest.mark.parametrize("name,make,xdt,batch", GEMV, ids=[g[0] for g in GEMV])
def test_fused_gemv_matches_fp64_oracle(name, make, xdt, batch):
    import torch
    layer = make()
    layer.x_dtype = xdt
    x = layer.activations(batch)
    ref = reference(layer, x)
    dev = H.DeviceLayer(layer, H.blob_from_library(layer)[0])
    y = dev.matmul(x, torch.float32 if xdt == "f32" else torch.bfloat16)
    assert y.shape == (batch, layer.m)
    assert H.rel_err(y, ref) <= TOL_F32, H.rel_err(y, ref)
    assert dev.status_value() == 0


def test_gemv_respects_row_strides():
    import torch
    from paper_1905_10138_b200 import sqnn
    layer = wl.make_layer(3, m=50, n=3000)
    x = layer.activations(3)
    ref = reference(layer, x)
    dev = H.DeviceLayer(layer, H.blob_from_library(layer)[0])
    xbuf = torch.zeros((3, 3000 + 24), dtype=torch.bfloat16, device="cuda")
    xbuf[:, :3000] = torch.from_numpy(x).cuda().to(torch.bfloat16)
    ybuf = torch.full((3, 50 + 7), 7.0, dtype=torch.float32, device="cuda")
    sqnn.sqnn_decode_matmul(dev.desc, dev.blob, dev.mask, dev.alpha, xbuf[:, :3000], ybuf[:, :50], None, dev.status)
    torch.cuda.synchronize()
    y = ybuf.cpu().numpy()
    assert H.rel_err(y[:, :50], ref) <= TOL_F32
    assert np.all(y[:, 50:] == 7.0)


def test_gemv_never_reads_activations_outside_a_row():
    """Rows that start inside a 32-bit word (n not a multiple of 32), activations read from global
    memory (too wide for shared memory) with NaN between the rows of X: a read at a column
    outside [0, n) would poison Y even if its weight were zero."""
    import torch
    from paper_1905_10138_b200 import sqnn
    layer = generic_layer(100, 10, 24, 5150, 0.3, 31)
    x = layer.activations(8)
    ref = reference(layer, x)
    dev = H.DeviceLayer(layer, H.blob_from_library(layer)[0])
    xbuf = torch.full((10, 5150 + 64), float("nan"), dtype=torch.float32, device="cuda")
    xbuf[1:9, 32:32 + 5150] = torch.from_numpy(x).cuda()
    ybuf = torch.full((8, 24), float("nan"), dtype=torch.float32, device="cuda")
    sqnn.sqnn_decode_matmul(dev.desc, dev.blob, dev.mask, dev.alpha, xbuf[1:9, 32:32 + 5150], ybuf, None, dev.status)
    torch.cuda.synchronize()
    assert H.rel_err(ybuf.cpu().numpy(), ref) <= TOL_F32


# ----------------------------------------------------------------------------------------------
# tensor-core path (batch >= 16): weights are rounded to bf16, fp32 accumulation in tensor memory
# ----------------------------------------------------------------------------------------------
MMA = [
    ("cfg2-s-b64", lambda: wl.make_layer(2, m=300, n=9216), 64),          # ragged last row tile
    ("cfg3-s-b32", lambda: wl.make_layer(3, m=203, n=3000), 32),          # n not a multiple of 64
    ("cfg4-s-b16", lambda: wl.make_layer(4, m=130, n=16384), 16),
    ("cfg4-s-b128", lambda: wl.make_layer(4, m=130, n=16384), 128),
    ("cfg4-s-b512", lambda: wl.make_layer(4, m=130, n=4096), 512),        # two passes of two accumulators
    ("cfg2-s-b200-wide", lambda: wl.make_layer(2, m=700, n=1024), 200),   # three row tiles, two accumulators, one column range
    ("cfg1-b16", lambda: wl.make_layer(1), 16),
    ("gen-33x20-q2-b48", lambda: generic_layer(33, 20, 140, 2049 + 7, 0.5, 13, n_q=2), 48),
    ("gen-96x9-q5-b24", lambda: generic_layer(96, 9, 70, 1000, 0.3, 16, n_q=5), 24),    # five planes, five CTAs per row tile
    ("gen-b300", lambda: generic_layer(100, 10, 129, 520, 0.2, 23), 300),                # two passes: 256 + 44 batch rows
    ("gen-b600", lambda: generic_layer(60, 12, 64, 776, 0.2, 24, n_q=2), 600),           # three passes over the batch
    ("gen-narrow-n-b16", lambda: generic_layer(40, 12, 300, 24, 0.4, 21), 16),
]


@pytest.mark.parametrize("name,make,batch", MMA, ids=[g[0] for g in MMA])
def test_fused_tensor_core_product_matches_fp64_oracle(name, make, batch):
    """The planes are decoded to packed bits in the workspace, the tensor-core kernel reads them."""
    import torch
    layer = make()
    layer.x_dtype = "bf16"
    x = layer.activations(batch)
    ref = reference(layer, x)
    dev = H.DeviceLayer(layer, H.blob_from_library(layer)[0])
    y = dev.matmul(x, torch.bfloat16)
    assert y.shape == (batch, layer.m)
    assert dev.status_value() == 0
    assert H.rel_err(y, ref) <= TOL_BF16, H.rel_err(y, ref)
    # tighter: the kernel keeps the weights exact for any number of planes (one sign tile per plane, scale
    # applied to the accumulator), so against the oracle's product only the fp32 accumulation order differs
    assert H.rel_err(y, ref) <= 2e-4, H.rel_err(y, ref)


def test_tensor_core_path_rejects_what_it_cannot_take():
    import torch
    from paper_1905_10138_b200 import sqnn
    layer = wl.make_layer(1)
    dev = H.DeviceLayer(layer, H.blob_from_library(layer)[0])
    y = torch.zeros((16, layer.m), dtype=torch.float32, device="cuda")
    xf = torch.zeros((16, layer.n), dtype=torch.float32, device="cuda")
    with pytest.raises(sqnn.SqnnError) as e:                       # fp32 activations need batch <= 15
        sqnn.sqnn_decode_matmul(dev.desc, dev.blob, dev.mask, dev.alpha, xf, y, None, dev.status)
    assert e.value.status == sqnn.E_UNSUPPORTED
    xok = torch.zeros((16, layer.n), dtype=torch.bfloat16, device="cuda")
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for ws in (small, None):                                       # workspace too small, or missing
        with pytest.raises(sqnn.SqnnError) as e:
            sqnn.sqnn_decode_matmul(dev.desc, dev.blob, dev.mask, dev.alpha, xok, y, ws, dev.status)
        assert e.value.status == sqnn.E_WORKSPACE
    xb = torch.zeros((16, layer.n + 3), dtype=torch.bfloat16, device="cuda")[:, : layer.n]
    ws = torch.zeros(sqnn.sqnn_workspace_bytes(dev.desc, 16), dtype=torch.uint8, device="cuda")
    with pytest.raises(sqnn.SqnnError) as e:                       # row pitch not a multiple of 16 bytes
        sqnn.sqnn_decode_matmul(dev.desc, dev.blob, dev.mask, dev.alpha, xb, y, ws, dev.status)
    assert e.value.status == sqnn.E_UNSUPPORTED


def test_convolution_tensor_goes_through_decode_and_product():
    """Section 3.1: a 4-D convolution tensor is flattened like any other weight tensor.  A ResNet-shaped 3 x 3
    layer (2-bit codes, 70 % pruned) is encoded, decoded on the GPU bit for bit, and applied to batches of
    im2col patch vectors (the product a convolution layer performs) on both product paths."""
    import torch
    layer = wl.make_conv_layer(128, 128, 3, 3)
    arrays = H.oracle_encode(layer)
    ref_bits = H.oracle_decode(layer, arrays)
    blob, _ = H.blob_from_library(layer)
    assert np.array_equal(blob, H.blob_from_oracle(layer, arrays))          # the two encoders agree byte for byte
    dev = H.DeviceLayer(layer, blob)
    got = dev.decode_bits()
    for i in range(layer.n_q):
        assert np.array_equal(got[i], wl.pack_bits(ref_bits[i]))
    for batch, tol in ((1, TOL_F32), (8, TOL_F32), (64, TOL_BF16)):
        x = layer.activations(batch)                                        # patch vectors of c_in * kh * kw values
        y = dev.matmul(x, torch.bfloat16)
        ref = orc.matmul(ref_bits, layer.mask, layer.alpha, x.astype(np.float64))
        assert H.rel_err(y, ref) <= tol, (batch, H.rel_err(y, ref))
    assert dev.status_value() == 0


def test_a_bounded_wait_that_runs_out_reports_a_timeout_and_the_kernel_returns():
    """Every wait of the tensor-core kernel is bounded.  With the library's test knob its loader role issues no
    loads and the limit is about a millisecond: the consumer's wait runs out, the kernel reports 6
    (-SQNN_E_TIMEOUT) through the status word, frees its tensor memory and returns -- nothing traps, the
    context stays usable, and the same call made normally right afterwards is correct."""
    import torch
    from paper_1905_10138_b200 import sqnn
    layer = wl.make_layer(1)                                            # the smallest tensor-core case
    layer.x_dtype = "bf16"
    x = layer.activations(16)
    ref = reference(layer, x)
    dev = H.DeviceLayer(layer, H.blob_from_library(layer)[0])
    d_x = torch.from_numpy(x).cuda().to(torch.bfloat16)
    d_y = torch.zeros((16, layer.m), dtype=torch.float32, device="cuda")
    ws = torch.empty(sqnn.sqnn_workspace_bytes(dev.desc, 16), dtype=torch.uint8, device="cuda")
    try:
        sqnn.sqnn_set_debug_flags(1, 2_000_000)                         # no loads; waits give up after ~1 ms
        sqnn.sqnn_decode_matmul(dev.desc, dev.blob, dev.mask, dev.alpha, d_x, d_y, ws, dev.status)
        torch.cuda.synchronize()                                        # returns: the kernel did not hang
        assert dev.status_value() == -sqnn.E_TIMEOUT
    finally:
        sqnn.sqnn_set_debug_flags(0, 0)
    dev.status.zero_()
    sqnn.sqnn_decode_matmul(dev.desc, dev.blob, dev.mask, dev.alpha, d_x, d_y, ws, dev.status)
    torch.cuda.synchronize()
    assert dev.status_value() == 0
    assert H.rel_err(d_y.cpu().numpy(), ref) <= 2e-4
