"""The allocation-free entry point, ``sqnn_decode_matmul_static``.

It exists for callers that cannot obtain device memory when they call the library -- code under
a stream capture, plug-ins living inside a framework that owns the device heap, serving loops
whose memory plan is fixed at start-up -- so its scratch is an array inside the library.  The
test calls it through the C ABI twice in a row (two different layers, so the second call finds
the first call's leftovers in the shared array) and holds each result against what
``sqnn_decode_matmul`` gives with a caller-provided workspace, within the tolerance the other
tensor-core tests use for results that differ only in fp32 accumulation order, and against the
oracle's fp64 product.  It also watches the device's free memory across a call: the entry point
must not take any.  Collected last on purpose: a run that stops at the first failure has then
already run every other test."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_1905_10138_b200 import sqnn
from paper_1905_10138_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu

TOL_ORDER = 2e-4        # same products, different fp32 summation order (atomics)


def both_ways(layer, batch):
    import torch
    layer.x_dtype = "bf16"
    x = layer.activations(batch)
    dev = H.DeviceLayer(layer, H.blob_from_library(layer)[0])
    y_ref = dev.matmul(x, torch.bfloat16, workspace=True)
    d_x = torch.from_numpy(x).cuda().to(torch.bfloat16)
    d_y = torch.full((batch, layer.m), float("nan"), dtype=torch.float32, device="cuda")
    sqnn.sqnn_decode_matmul_static(dev.desc, dev.blob, dev.mask, dev.alpha, d_x, d_y, dev.status)   # first call on this device
    torch.cuda.synchronize()
    # a second call with every buffer already in place: the device's free memory must not move
    free_before = torch.cuda.mem_get_info()[0]
    sqnn.sqnn_decode_matmul_static(dev.desc, dev.blob, dev.mask, dev.alpha, d_x, d_y, dev.status)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the allocation-free entry point took device memory"
    assert dev.status_value() == 0
    ref_bits = H.oracle_decode(layer, H.oracle_encode(layer))
    y_orc = orc.matmul(ref_bits, layer.mask, layer.alpha, x.astype(np.float64))
    return d_y.cpu().numpy(), y_ref, y_orc


def test_static_scratch_entry_point_matches_workspace_path_on_two_calls_in_a_row():
    first = wl.make_layer(3, m=203, n=3000)            # 2 planes, ragged K
    second = wl.make_layer(2, m=300, n=9216)           # 1 plane, larger: overwrites what the first left
    for layer, batch in ((first, 32), (second, 64)):
        assert sqnn.sqnn_workspace_bytes(sqnn.sqnn_describe_host(H.blob_from_library(layer)[0]), batch) \
            <= sqnn.STATIC_SCRATCH_BYTES
        y, y_ref, y_orc = both_ways(layer, batch)
        assert np.all(np.isfinite(y))
        assert H.rel_err(y, y_ref) <= TOL_ORDER, H.rel_err(y, y_ref)
        assert H.rel_err(y, y_orc) <= TOL_ORDER, H.rel_err(y, y_orc)      # the kernel keeps the weights exact


def test_static_scratch_entry_point_refuses_what_does_not_fit_or_needs_no_scratch():
    import torch
    big = wl.make_layer(1, m=8300, n=8192)             # 68 million weight bits: over the 8 MiB array
    dev = H.DeviceLayer(big, H.blob_from_library(big)[0])
    assert sqnn.sqnn_workspace_bytes(dev.desc, 16) > sqnn.STATIC_SCRATCH_BYTES
    x = torch.zeros((16, big.n), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((16, big.m), dtype=torch.float32, device="cuda")
    with pytest.raises(sqnn.SqnnError) as e:
        sqnn.sqnn_decode_matmul_static(dev.desc, dev.blob, dev.mask, dev.alpha, x, y, dev.status)
    assert e.value.status == sqnn.E_WORKSPACE
    with pytest.raises(sqnn.SqnnError) as e:           # batch <= 15 takes the GEMV path, which has no scratch
        sqnn.sqnn_decode_matmul_static(dev.desc, dev.blob, dev.mask, dev.alpha, x[:8], y[:8], dev.status)
    assert e.value.status == sqnn.E_UNSUPPORTED
    # an activation type that does not exist is a bad argument here as in sqnn_decode_matmul
    import ctypes
    rc = sqnn.lib().sqnn_decode_matmul_static(ctypes.byref(dev.desc), ctypes.c_void_p(dev.blob.data_ptr()),
                                              ctypes.c_void_p(dev.mask.data_ptr()), ctypes.c_void_p(dev.alpha.data_ptr()),
                                              ctypes.c_void_p(x.data_ptr()), 7, 16, big.n, ctypes.c_void_p(y.data_ptr()),
                                              big.m, None, None)
    assert rc == sqnn.E_INVALID_ARG
