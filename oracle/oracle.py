"""numpy front end of the CPU oracle (``sqnn_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The CUDA library never imports this module and
this module never imports the CUDA library.

Array conventions (all numpy, C-contiguous):
  M      uint8  [n_out, n_in]   the XOR-gate network over GF(2) (Section 3.1)
  bits   uint8  [mn]            one bit-plane, flattened row-major, 1 <-> +1
  care   uint8  [mn]            1 = unpruned (care), 0 = pruned (don't care)
  wc     uint64 [l]             seed per slice, bit t = w^c[t]
  np_    uint16 [l]             n_patch per slice (Section 3.2)
  dp     uint16 [sum n_patch]   d_patch positions, slice order, ascending
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sqnn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP for the outer slice / row loops only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        lib.orc_num_threads.restype = i32
        lib.orc_set_num_threads.argtypes = [i32]
        lib.orc_xor_network.argtypes = [i32, i32, vp, vp, vp]
        lib.orc_encode_slice.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        lib.orc_encode_slice.restype = i32
        lib.orc_encode_slice_exhaustive.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        lib.orc_encode_slice_exhaustive.restype = i32
        lib.orc_decode_slice.argtypes = [i32, i32, vp, vp, i32, vp, vp]
        lib.orc_encode_plane.argtypes = [i64, i32, i32, vp, vp, vp, i32, vp, vp, vp, i64]
        lib.orc_encode_plane.restype = i64
        lib.orc_decode_plane.argtypes = [i64, i32, i32, vp, vp, vp, vp, i64, i64, vp]
        lib.orc_decode_plane.restype = i32
        lib.orc_bf16_from_f32.argtypes = [ctypes.c_float]
        lib.orc_bf16_from_f32.restype = ctypes.c_uint16
        lib.orc_reconstruct.argtypes = [i64, i64, i32, vp, vp, vp, vp, vp]
        lib.orc_matmul.argtypes = [i64, i64, i32, vp, vp, vp, vp, i64, vp]
        lib.orc_eq1.argtypes = [i64, i32, i32, vp, vp]
        lib.orc_eq1_blocked.argtypes = [i64, i32, i32, vp, i64, vp]
        lib.orc_blocked_field_bits.argtypes = [i64, vp, i64, vp]
        lib.orc_fifo_model.argtypes = [i64, vp, i32, i32, i32, vp]
        lib.orc_csr_relative_time.argtypes = [i64, vp, i32]
        lib.orc_csr_relative_time.restype = ctypes.c_double
        _lib = lib
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _u8(a):
    return np.ascontiguousarray(a, dtype=np.uint8)


def num_threads() -> int:
    return int(_L().orc_num_threads())


def set_num_threads(t: int) -> None:
    _L().orc_set_num_threads(int(t))


def xor_network(M, wc_bits):
    """w~ = M . w^c over GF(2) (Section 3.1).  wc_bits: uint8 [n_in] -> uint8 [n_out]."""
    M = _u8(M)
    wc_bits = _u8(wc_bits)
    n_out, n_in = M.shape
    out = np.empty(n_out, dtype=np.uint8)
    _L().orc_xor_network(n_out, n_in, _p(M), _p(wc_bits), _p(out))
    return out


def encode_slice(M, wq, care, exhaustive: bool = False):
    """Algorithm 1 (or the exhaustive search of Section 5.2) on one slice.

    Returns (wc_bits uint8 [n_in], d_patch uint16 [n_patch])."""
    M, wq, care = _u8(M), _u8(wq), _u8(care)
    n_out, n_in = M.shape
    assert wq.shape == (n_out,) and care.shape == (n_out,)
    wc = np.zeros(n_in, dtype=np.uint8)
    dp = np.zeros(max(n_out, 1), dtype=np.uint16)
    fn = _L().orc_encode_slice_exhaustive if exhaustive else _L().orc_encode_slice
    n = fn(n_out, n_in, _p(M), _p(wq), _p(care), _p(wc), _p(dp))
    if n < 0:
        raise RuntimeError("oracle encode_slice failed")
    return wc, dp[:n].copy()


def decode_slice(M, wc_bits, d_patch):
    """Network output with the d_patch positions flipped (Sections 3.1, 3.2)."""
    M, wc_bits = _u8(M), _u8(wc_bits)
    d_patch = np.ascontiguousarray(d_patch, dtype=np.uint16)
    n_out, n_in = M.shape
    out = np.empty(n_out, dtype=np.uint8)
    _L().orc_decode_slice(n_out, n_in, _p(M), _p(wc_bits), int(d_patch.size), _p(d_patch), _p(out))
    return out


def encode_plane(M, bits, care, exhaustive: bool = False):
    """Encode a flattened plane.  Returns (wc uint64 [l], np uint16 [l], dp uint16 [sum np])."""
    M, bits, care = _u8(M), _u8(bits).ravel(), _u8(care).ravel()
    n_out, n_in = M.shape
    mn = bits.size
    assert care.size == mn
    l = (mn + n_out - 1) // n_out
    wc = np.zeros(l, dtype=np.uint64)
    np_ = np.zeros(l, dtype=np.uint16)
    cap = int(care.sum()) + 1
    dp = np.zeros(cap, dtype=np.uint16)
    tot = _L().orc_encode_plane(mn, n_out, n_in, _p(M), _p(bits), _p(care), int(exhaustive),
                                _p(wc), _p(np_), _p(dp), cap)
    if tot < 0:
        raise RuntimeError("oracle encode_plane failed")
    return wc, np_, dp[:tot].copy()


def decode_plane(M, mn, wc, np_, dp, s_begin: int = 0, s_end: int | None = None, out=None):
    """Decode slices [s_begin, s_end) of a plane into uint8 bits (one byte per position).

    Returns the full-length array (positions outside the range are left as they were / 0)."""
    M = _u8(M)
    n_out, n_in = M.shape
    l = (mn + n_out - 1) // n_out
    if s_end is None:
        s_end = l
    wc = np.ascontiguousarray(wc, dtype=np.uint64)
    np_ = np.ascontiguousarray(np_, dtype=np.uint16)
    dp = np.ascontiguousarray(dp, dtype=np.uint16)
    assert wc.size == l and np_.size == l and dp.size == int(np_.astype(np.int64).sum())
    if out is None:
        out = np.zeros(mn, dtype=np.uint8)
    rc = _L().orc_decode_plane(mn, n_out, n_in, _p(M), _p(wc), _p(np_), _p(dp),
                               int(s_begin), int(s_end), _p(out))
    if rc != 0:
        raise RuntimeError("oracle decode_plane failed")
    return out


def bf16_from_f32(x) -> np.ndarray:
    """Round fp32 values to bf16 bit patterns (uint16), nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    flat = x.ravel()
    out = np.empty(flat.size, dtype=np.uint16)
    f = _L().orc_bf16_from_f32
    for i in range(flat.size):
        out[i] = f(float(flat[i]))
    return out.reshape(x.shape)


def reconstruct(planes, mask, alpha, want_f32: bool = True, want_bf16: bool = True):
    """Masked, rescaled weights from decoded planes.

    planes uint8 [n_q, m, n]; mask uint8 [m, n]; alpha float32 [m, n_q].
    Returns (W float32 [m, n] or None, W_bf16_bits uint16 [m, n] or None)."""
    planes, mask = _u8(planes), _u8(mask)
    alpha = np.ascontiguousarray(alpha, dtype=np.float32)
    n_q, m, n = planes.shape
    assert mask.shape == (m, n) and alpha.shape == (m, n_q)
    w32 = np.empty((m, n), dtype=np.float32) if want_f32 else None
    wbf = np.empty((m, n), dtype=np.uint16) if want_bf16 else None
    _L().orc_reconstruct(m, n, n_q, _p(planes), _p(mask), _p(alpha), _p(w32), _p(wbf))
    return w32, wbf


def matmul(planes, mask, alpha, X):
    """Y[b, r] = sum_c W[r, c] X[b, c] in fp64 from decoded planes.  X: [batch, n] -> Y: [batch, m]."""
    planes, mask = _u8(planes), _u8(mask)
    alpha = np.ascontiguousarray(alpha, dtype=np.float32)
    X = np.ascontiguousarray(X, dtype=np.float64)
    n_q, m, n = planes.shape
    batch = X.shape[0]
    assert X.shape == (batch, n)
    Y = np.empty((batch, m), dtype=np.float64)
    _L().orc_matmul(m, n, n_q, _p(planes), _p(mask), _p(alpha), _p(X), batch, _p(Y))
    return Y


def eq1(mn: int, n_out: int, n_in: int, np_) -> dict:
    """Eq. 1 for one plane, literally.  bits/weight = 1 / r."""
    np_ = np.ascontiguousarray(np_, dtype=np.uint16)
    assert np_.size == (mn + n_out - 1) // n_out
    out = np.zeros(6, dtype=np.float64)
    _L().orc_eq1(mn, n_out, n_in, _p(np_), _p(out))
    return {"r": out[0], "bits_wc": out[1], "bits_npatch": out[2], "bits_dpatch": out[3],
            "max_p": int(out[4]), "sum_p": int(out[5]), "bits_per_weight": 1.0 / out[0]}


def eq1_blocked(mn: int, n_out: int, n_in: int, np_, block: int) -> dict:
    """Eq. 1 with the n_patch width chosen per block of `block` slices (Section 5.2)."""
    np_ = np.ascontiguousarray(np_, dtype=np.uint16)
    assert np_.size == (mn + n_out - 1) // n_out and block >= 1
    out = np.zeros(4, dtype=np.float64)
    _L().orc_eq1_blocked(mn, n_out, n_in, _p(np_), block, _p(out))
    return {"r": out[0], "bits_npatch": out[1], "blocks": int(out[2]), "bits_widths": out[3],
            "bits_per_weight": 1.0 / out[0]}


def blocked_field_bits(np_, block: int) -> dict:
    """Bits of the n_patch fields when every block of `block` slices gets the narrowest field that holds
    all its counts, ceil(lg(max p + 1)) (Section 5.2 as a stored format)."""
    np_ = np.ascontiguousarray(np_, dtype=np.uint16)
    assert block >= 1
    out = np.zeros(2, dtype=np.float64)
    _L().orc_blocked_field_bits(np_.size, _p(np_), block, _p(out))
    return {"bits_npatch": int(out[0]), "blocks": int(out[1])}


def fifo_model(np_, n_fifo: int, rate: int, depth: int) -> dict:
    """Cycle-by-cycle model of the patch-data FIFO of one XOR-gate network (Section 5.1)."""
    np_ = np.ascontiguousarray(np_, dtype=np.uint16)
    assert n_fifo >= 1 and rate >= 1 and depth >= 1
    out = np.zeros(5, dtype=np.float64)
    _L().orc_fifo_model(np_.size, _p(np_), n_fifo, rate, depth, _p(out))
    return {"cycles": int(out[0]), "stall_bandwidth": int(out[1]), "stall_empty": int(out[2]),
            "stall_full": int(out[3]), "peak": int(out[4]),
            "relative_time": out[0] / max(np_.size, 1)}


def csr_relative_time(nnz_per_row, lanes: int) -> float:
    """Lock-step CSR rows, `lanes` at a time: cycles / (sum nnz / lanes) (Section 5.1)."""
    nnz = np.ascontiguousarray(nnz_per_row, dtype=np.int64)
    return float(_L().orc_csr_relative_time(nnz.size, _p(nnz), lanes))
