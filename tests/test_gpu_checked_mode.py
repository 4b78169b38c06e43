"""Checked mode of the device entry points (environment variable SQNN_DEBUG_CHECKS=1, read once per
process): the call waits for its stream and returns what the kernels left in the status word as an
error code.  Runs in a child process, because the variable is read at the first device call."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

CHILD = r"""
import numpy as np, torch
from paper_1905_10138_b200 import sqnn
from paper_1905_10138_b200 import workloads as wl
from tests import helpers as H

layer = wl.make_sweep_layer(1, 2, m=40, n=1000)
blob, _ = H.blob_from_library(layer)
dev = H.DeviceLayer(layer, blob)
d = dev.desc
assert d.n_pp[0] > 0
clean = dev.decode_bits()                                # returns normally: nothing to report
assert dev.status_value() == 0
dev.blob[int(d.off_pp[0]) + 1] = 255                     # first patch position now lies outside its tile
torch.cuda.synchronize()
try:
    dev.decode_bits()
    raise SystemExit("a damaged patch entry did not turn into an error code")
except sqnn.SqnnError as e:
    assert e.status == sqnn.E_BAD_BLOB, e.status
assert dev.status_value() == 1                           # the status word is left as the kernel set it

# a bounded wait that runs out comes back as SQNN_E_TIMEOUT, and the next call works
layer = wl.make_layer(1)                                 # the smallest tensor-core case
layer.x_dtype = "bf16"
blob, _ = H.blob_from_library(layer)
dev = H.DeviceLayer(layer, blob)
x = layer.activations(16)
want = dev.matmul(x, torch.bfloat16)
sqnn.sqnn_set_debug_flags(1, 2_000_000)                  # the loader issues no loads; waits give up after 2 M cycles
try:
    dev.matmul(x, torch.bfloat16)
    raise SystemExit("the timeout did not turn into an error code")
except sqnn.SqnnError as e:
    assert e.status == sqnn.E_TIMEOUT, e.status
finally:
    sqnn.sqnn_set_debug_flags(0, 0)
dev.status.zero_()
again = dev.matmul(x, torch.bfloat16)
assert np.allclose(again, want, rtol=1e-5, atol=1e-5)    # the product adds into Y with atomics: order differs
print("checked mode ok")
"""


def test_checked_mode_returns_device_side_findings_as_error_codes():
    env = dict(os.environ, SQNN_DEBUG_CHECKS="1")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env["PYTHONPATH"] = root + os.pathsep + env.get("PYTHONPATH", "")
    r = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=root, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "checked mode ok" in r.stdout
