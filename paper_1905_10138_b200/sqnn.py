"""Thin ctypes binding over ``libsqnn.so`` -- same names as ``include/sqnn.h``.

Argument marshalling only: every step of the decode / product path runs in the library's
kernels.  Device buffers are torch CUDA tensors (torch is used for device memory and
streams, nothing else).  There is no CPU fallback: if the library cannot be loaded every
call raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# SQNN_LIBRARY overrides the in-tree build (e.g. to try a differently compiled library)
LIB_PATH = os.environ.get("SQNN_LIBRARY") or os.path.join(_HERE, "libsqnn.so")

MAX_PLANES = 8
STATIC_SCRATCH_BYTES = 8 << 20
OUT_BITS, OUT_BF16, OUT_SINK = 0, 1, 2
X_F32, X_BF16 = 0, 1
ENCODE_ALG1, ENCODE_EXHAUSTIVE = 0, 1
OK, E_INVALID_ARG, E_BAD_BLOB, E_UNSUPPORTED, E_NOMEM, E_CUDA, E_TIMEOUT, E_WORKSPACE = 0, -1, -2, -3, -4, -5, -6, -7


class SqnnError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} ({status})")


class XorNet(ctypes.Structure):
    _fields_ = [("n_out", ctypes.c_uint32), ("n_in", ctypes.c_uint32), ("rows", ctypes.c_void_p)]


class Planes(ctypes.Structure):
    _fields_ = [("m", ctypes.c_uint64), ("n", ctypes.c_uint64), ("n_q", ctypes.c_uint32),
                ("planes", ctypes.c_void_p), ("mask", ctypes.c_void_p)]


PATCH_HIST_BINS = 16


class Stats(ctypes.Structure):
    _fields_ = [("slices", ctypes.c_uint64), ("patches", ctypes.c_uint64 * MAX_PLANES),
                ("max_patch", ctypes.c_uint32 * MAX_PLANES),
                ("bits_wc", ctypes.c_uint64), ("bits_npatch", ctypes.c_uint64),
                ("bits_dpatch", ctypes.c_uint64), ("bits_index", ctypes.c_uint64),
                ("bits_tables", ctypes.c_uint64), ("patch_hist", ctypes.c_uint64 * PATCH_HIST_BINS),
                ("bpw_eq1", ctypes.c_double), ("bpw_actual", ctypes.c_double)]

    def as_dict(self, n_q: int) -> dict:
        return {"slices": int(self.slices), "patches": [int(v) for v in self.patches[:n_q]],
                "max_patch": [int(v) for v in self.max_patch[:n_q]],
                "bits_wc": int(self.bits_wc), "bits_npatch": int(self.bits_npatch),
                "bits_dpatch": int(self.bits_dpatch), "bits_index": int(self.bits_index),
                "bits_tables": int(self.bits_tables), "patch_hist": [int(v) for v in self.patch_hist],
                "bpw_eq1": float(self.bpw_eq1), "bpw_actual": float(self.bpw_actual)}


class StoreInfo(ctypes.Structure):
    _fields_ = [("bits_wc", ctypes.c_uint64), ("bits_widths", ctypes.c_uint64), ("bits_npatch", ctypes.c_uint64),
                ("bits_dpatch", ctypes.c_uint64), ("total_bytes", ctypes.c_uint64), ("bpw", ctypes.c_double)]


class FifoResult(ctypes.Structure):
    _fields_ = [("cycles", ctypes.c_uint64), ("stall_bandwidth", ctypes.c_uint64),
                ("stall_empty", ctypes.c_uint64), ("stall_full", ctypes.c_uint64), ("peak", ctypes.c_uint64)]


class Desc(ctypes.Structure):
    _fields_ = [("m", ctypes.c_uint64), ("n", ctypes.c_uint64), ("slices", ctypes.c_uint64),
                ("slices_padded", ctypes.c_uint64),
                ("n_q", ctypes.c_uint32), ("n_out", ctypes.c_uint32), ("n_in", ctypes.c_uint32),
                ("tile_slices", ctypes.c_uint32),
                ("tab_chunks", ctypes.c_uint32), ("tab_chunk_bits", ctypes.c_uint32),
                ("tab_entry_words", ctypes.c_uint32), ("reserved", ctypes.c_uint32),
                ("off_xornet", ctypes.c_uint64), ("off_tables", ctypes.c_uint64), ("tables_bytes", ctypes.c_uint64),
                ("off_wc", ctypes.c_uint64 * MAX_PLANES), ("off_idx", ctypes.c_uint64 * MAX_PLANES),
                ("off_pp", ctypes.c_uint64 * MAX_PLANES),
                ("n_pp", ctypes.c_uint64 * MAX_PLANES), ("total_bytes", ctypes.c_uint64)]


_lib = None


def lib():
    """The loaded C library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with "
                              "`python -m paper_1905_10138_b200.build` (needs nvcc, sm_100a)")
        L = ctypes.CDLL(LIB_PATH)
        vp, u32, u64, i64, i32, sz = (ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int64,
                                      ctypes.c_int, ctypes.c_size_t)
        P = ctypes.POINTER
        L.sqnn_encode_host.argtypes = [P(XorNet), P(Planes), u32, P(vp), P(sz), P(Stats)]
        L.sqnn_encode_seeds_host.argtypes = [P(XorNet), P(Planes), P(vp), P(vp), P(sz), P(Stats)]
        L.sqnn_encode_seeds_host.restype = i32
        L.sqnn_search_seeds.argtypes = [P(XorNet), u64, u64, u32, vp, vp, vp, vp, vp]
        L.sqnn_search_seeds.restype = i32
        L.sqnn_pack_host.argtypes = [P(XorNet), u64, u64, u32, P(vp), P(vp), P(vp), P(vp), P(sz)]
        L.sqnn_unpack_host.argtypes = [vp, sz, u32, P(vp), P(vp), P(vp), P(u64)]
        L.sqnn_describe_host.argtypes = [vp, sz, P(Desc)]
        L.sqnn_stats_host.argtypes = [vp, sz, P(Stats)]
        L.sqnn_stats_blocked_host.argtypes = [vp, sz, u64, P(ctypes.c_double), P(u64)]
        L.sqnn_stats_blocked_host.restype = i32
        L.sqnn_encode_wide_host.argtypes = [u32, u32, vp, u64, vp, vp, P(vp), P(vp), P(vp), P(u64), P(ctypes.c_double)]
        L.sqnn_encode_wide_host.restype = i32
        L.sqnn_store_host.argtypes = [vp, sz, u64, P(vp), P(sz), P(StoreInfo)]
        L.sqnn_store_host.restype = i32
        L.sqnn_load_host.argtypes = [vp, sz, P(vp), P(sz)]
        L.sqnn_load_host.restype = i32
        L.sqnn_fifo_model_host.argtypes = [vp, u64, u32, u32, u32, P(FifoResult)]
        L.sqnn_fifo_model_host.restype = i32
        L.sqnn_free.argtypes = [vp]
        L.sqnn_free.restype = None
        L.sqnn_decode.argtypes = [P(Desc), vp, vp, vp, i32, vp, sz, vp, vp]
        L.sqnn_decode_matmul.argtypes = [P(Desc), vp, vp, vp, vp, i32, u32, i64, vp, i64, vp, sz, vp, vp]
        L.sqnn_decode_matmul_static.argtypes = [P(Desc), vp, vp, vp, vp, i32, u32, i64, vp, i64, vp, vp]
        L.sqnn_decode_matmul_static.restype = i32
        L.sqnn_store_probe.argtypes = [vp, sz, u32, vp]
        L.sqnn_store_probe.restype = i32
        L.sqnn_set_debug_flags.argtypes = [u32, u64]
        L.sqnn_set_debug_flags.restype = None
        L.sqnn_workspace_bytes.argtypes = [P(Desc), u32]
        L.sqnn_workspace_bytes.restype = sz
        L.sqnn_status_string.argtypes = [i32]
        L.sqnn_status_string.restype = ctypes.c_char_p
        for name in ("sqnn_encode_host", "sqnn_pack_host", "sqnn_unpack_host", "sqnn_describe_host",
                     "sqnn_stats_host", "sqnn_decode", "sqnn_decode_matmul"):
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().sqnn_status_string(int(status)).decode()


def _check(status: int, what: str):
    if status != OK:
        raise SqnnError(status, what)


def _np_ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _take(ptr: ctypes.c_void_p, nbytes: int) -> np.ndarray:
    """Copies a library-owned host buffer into a numpy array and frees it."""
    out = np.empty(nbytes, dtype=np.uint8)
    if nbytes:
        ctypes.memmove(out.ctypes.data, ptr.value, nbytes)
    lib().sqnn_free(ptr)
    return out


def _net(rows: np.ndarray, n_in: int):
    rows = np.ascontiguousarray(rows, dtype=np.uint32)
    return XorNet(int(rows.size), int(n_in), rows.ctypes.data), rows


def sqnn_encode_host(rows, n_in, m, n, n_q, planes_words, mask_words, flags=ENCODE_ALG1):
    """rows uint32 [n_out]; planes_words uint64 [n_q * ceil(mn/64)]; mask_words uint64 [ceil(mn/64)].
    Returns (blob uint8 array, stats dict)."""
    net, _keep = _net(rows, n_in)
    planes_words = np.ascontiguousarray(planes_words, dtype=np.uint64)
    mask_words = np.ascontiguousarray(mask_words, dtype=np.uint64)
    words = (m * n + 63) // 64
    if planes_words.size != n_q * words or mask_words.size != words:
        raise ValueError("packed plane / mask size mismatch")
    layer = Planes(m, n, n_q, planes_words.ctypes.data, mask_words.ctypes.data)
    blob, nbytes, st = ctypes.c_void_p(), ctypes.c_size_t(), Stats()
    _check(lib().sqnn_encode_host(ctypes.byref(net), ctypes.byref(layer), flags, ctypes.byref(blob),
                                  ctypes.byref(nbytes), ctypes.byref(st)), "sqnn_encode_host")
    return _take(blob, nbytes.value), st.as_dict(n_q)


def sqnn_encode_seeds_host(rows, n_in, m, n, n_q, planes_words, mask_words, wc):
    """As sqnn_encode_host with the seeds given: wc is a list (one per plane) of uint32 [l]."""
    net, _keep = _net(rows, n_in)
    planes_words = np.ascontiguousarray(planes_words, dtype=np.uint64)
    mask_words = np.ascontiguousarray(mask_words, dtype=np.uint64)
    wc = [np.ascontiguousarray(a, dtype=np.uint32) for a in wc]
    layer = Planes(m, n, n_q, planes_words.ctypes.data, mask_words.ctypes.data)
    arr = (ctypes.c_void_p * n_q)(*[a.ctypes.data for a in wc])
    blob, nbytes, st = ctypes.c_void_p(), ctypes.c_size_t(), Stats()
    _check(lib().sqnn_encode_seeds_host(ctypes.byref(net), ctypes.byref(layer), arr, ctypes.byref(blob),
                                        ctypes.byref(nbytes), ctypes.byref(st)), "sqnn_encode_seeds_host")
    return _take(blob, nbytes.value), st.as_dict(n_q)


def sqnn_search_seeds(rows, n_in, m, n, n_q, d_planes, d_mask, d_wc, d_np, stream=None):
    """Exhaustive seed search on the device.  d_planes / d_mask: CUDA int64 tensors (packed bits);
    d_wc: CUDA int32 [n_q * l]; d_np: CUDA int16 [n_q * l].  Queues on ``stream``."""
    net, _keep = _net(rows, n_in)
    _check(lib().sqnn_search_seeds(ctypes.byref(net), m, n, n_q, _dev_ptr(d_planes), _dev_ptr(d_mask),
                                   _dev_ptr(d_wc), _dev_ptr(d_np), _stream_ptr(stream)), "sqnn_search_seeds")


def sqnn_pack_host(rows, n_in, m, n, wc, np_, dp):
    """wc / np_ / dp: lists (one entry per plane) of uint32 [l], uint16 [l], uint16 [sum np]."""
    net, _keep = _net(rows, n_in)
    n_q = len(wc)
    wc = [np.ascontiguousarray(a, dtype=np.uint32) for a in wc]
    np_ = [np.ascontiguousarray(a, dtype=np.uint16) for a in np_]
    dp = [np.ascontiguousarray(np.concatenate([a, [0]]) if a.size == 0 else a, dtype=np.uint16) for a in dp]
    arr = ctypes.c_void_p * n_q
    blob, nbytes = ctypes.c_void_p(), ctypes.c_size_t()
    _check(lib().sqnn_pack_host(ctypes.byref(net), m, n, n_q,
                                arr(*[a.ctypes.data for a in wc]), arr(*[a.ctypes.data for a in np_]),
                                arr(*[a.ctypes.data for a in dp]), ctypes.byref(blob), ctypes.byref(nbytes)),
           "sqnn_pack_host")
    return _take(blob, nbytes.value)


def sqnn_describe_host(blob: np.ndarray) -> Desc:
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    d = Desc()
    _check(lib().sqnn_describe_host(_np_ptr(blob), blob.size, ctypes.byref(d)), "sqnn_describe_host")
    return d


def sqnn_stats_host(blob: np.ndarray) -> dict:
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    st = Stats()
    _check(lib().sqnn_stats_host(_np_ptr(blob), blob.size, ctypes.byref(st)), "sqnn_stats_host")
    d = sqnn_describe_host(blob)
    return st.as_dict(d.n_q)


def sqnn_stats_blocked_host(blob: np.ndarray, block_slices: int) -> dict:
    """Eq. 1 with the n_patch width chosen per block of `block_slices` slices (Section 5.2)."""
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    bpw, bits = ctypes.c_double(), ctypes.c_uint64()
    _check(lib().sqnn_stats_blocked_host(_np_ptr(blob), blob.size, int(block_slices), ctypes.byref(bpw),
                                         ctypes.byref(bits)), "sqnn_stats_blocked_host")
    return {"bpw_eq1": bpw.value, "bits_npatch": int(bits.value)}


def sqnn_encode_wide_host(rows64, n_in, mn, plane_words, mask_words):
    """Algorithm 1 for networks of up to 64 inputs / 4096 outputs (host only, no blob).  rows64: uint64 [n_out].
    Returns (wc uint64 [l], np uint16 [l], dp uint16 [sum np], bits per weight by Eq. 1)."""
    rows64 = np.ascontiguousarray(rows64, dtype=np.uint64)
    plane_words = np.ascontiguousarray(plane_words, dtype=np.uint64)
    mask_words = np.ascontiguousarray(mask_words, dtype=np.uint64)
    if plane_words.size != (mn + 63) // 64 or mask_words.size != plane_words.size:
        raise ValueError("packed plane / mask size mismatch")
    wc, np_, dp, n_dp, bpw = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_uint64(), ctypes.c_double()
    _check(lib().sqnn_encode_wide_host(int(rows64.size), int(n_in), _np_ptr(rows64), int(mn), _np_ptr(plane_words),
                                       _np_ptr(mask_words), ctypes.byref(wc), ctypes.byref(np_), ctypes.byref(dp),
                                       ctypes.byref(n_dp), ctypes.byref(bpw)), "sqnn_encode_wide_host")
    l = (mn + rows64.size - 1) // rows64.size
    return (_take(wc, 8 * l).view(np.uint64), _take(np_, 2 * l).view(np.uint16),
            _take(dp, 2 * int(n_dp.value)).view(np.uint16), float(bpw.value))


def sqnn_store_host(blob: np.ndarray, block_slices: int):
    """Device blob -> storage form with per-block n_patch widths (Sections 3.2, 5.2).  Returns (bytes, info dict)."""
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    out, nbytes, info = ctypes.c_void_p(), ctypes.c_size_t(), StoreInfo()
    _check(lib().sqnn_store_host(_np_ptr(blob), blob.size, int(block_slices), ctypes.byref(out), ctypes.byref(nbytes),
                                 ctypes.byref(info)), "sqnn_store_host")
    return _take(out, nbytes.value), {k: getattr(info, k) for k, _ in StoreInfo._fields_}


def sqnn_load_host(stored: np.ndarray) -> np.ndarray:
    """Storage form -> device blob."""
    stored = np.ascontiguousarray(stored, dtype=np.uint8)
    out, nbytes = ctypes.c_void_p(), ctypes.c_size_t()
    _check(lib().sqnn_load_host(_np_ptr(stored), stored.size, ctypes.byref(out), ctypes.byref(nbytes)), "sqnn_load_host")
    return _take(out, nbytes.value)


def sqnn_fifo_model_host(n_patch: np.ndarray, n_fifo: int, rate: int, depth: int) -> dict:
    """Cycle model of the patch-data FIFO of Section 5.1 over the n_patch counts of one plane."""
    n_patch = np.ascontiguousarray(n_patch, dtype=np.uint16)
    res = FifoResult()
    _check(lib().sqnn_fifo_model_host(_np_ptr(n_patch), n_patch.size, int(n_fifo), int(rate), int(depth),
                                      ctypes.byref(res)), "sqnn_fifo_model_host")
    out = {k: int(getattr(res, k)) for k, _ in FifoResult._fields_}
    out["relative_time"] = out["cycles"] / max(n_patch.size, 1)
    return out


def sqnn_unpack_host(blob: np.ndarray, plane: int):
    """Returns (wc uint32 [l], np uint16 [l], dp uint16 [n_dp]) of one plane."""
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    d = sqnn_describe_host(blob)
    wc, np_, dp, n_dp = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_uint64()
    _check(lib().sqnn_unpack_host(_np_ptr(blob), blob.size, plane, ctypes.byref(wc), ctypes.byref(np_),
                                  ctypes.byref(dp), ctypes.byref(n_dp)), "sqnn_unpack_host")
    l = int(d.slices)
    return (_take(wc, 4 * l).view(np.uint32), _take(np_, 2 * l).view(np.uint16),
            _take(dp, 2 * int(n_dp.value)).view(np.uint16))


def _dev_ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def _stream_ptr(stream):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def sqnn_decode(desc: Desc, d_blob, d_mask, d_alpha, mode: int, d_out, d_status=None, stream=None):
    """Queues the decode kernel on ``stream`` (default: torch's current stream).  Tensors are CUDA."""
    _check(lib().sqnn_decode(ctypes.byref(desc), _dev_ptr(d_blob), _dev_ptr(d_mask), _dev_ptr(d_alpha),
                             int(mode), _dev_ptr(d_out), d_out.numel() * d_out.element_size(),
                             _dev_ptr(d_status), _stream_ptr(stream)), "sqnn_decode")


def sqnn_store_probe(d_out, chunk_bytes: int = 3200, stream=None):
    """Measurement aid: fills ``d_out`` (CUDA tensor) with the decode kernel's output path (bulk copies
    out of shared memory) and nothing else, to measure the write ceiling of that path."""
    _check(lib().sqnn_store_probe(_dev_ptr(d_out), d_out.numel() * d_out.element_size(), int(chunk_bytes),
                                  _stream_ptr(stream)), "sqnn_store_probe")


def sqnn_set_debug_flags(flags: int, wait_limit_cycles: int = 0) -> None:
    """Test knob: bit 0 = the tensor-core kernel's loader issues no loads; wait_limit_cycles bounds its waits."""
    lib().sqnn_set_debug_flags(int(flags), int(wait_limit_cycles))


def sqnn_workspace_bytes(desc: Desc, batch: int) -> int:
    return int(lib().sqnn_workspace_bytes(ctypes.byref(desc), int(batch)))


def sqnn_decode_matmul(desc: Desc, d_blob, d_mask, d_alpha, d_x, d_y, d_workspace=None, d_status=None,
                       stream=None):
    """Y[b, r] = sum_c W[r, c] X[b, c].  d_x: [batch, n] float32 or bfloat16 (row stride free);
    d_y: [batch, m] float32.  batch >= 16 needs ``d_workspace`` of ``sqnn_workspace_bytes`` bytes.
    Queues on ``stream``; does not synchronise."""
    import torch
    if d_x.dim() != 2 or d_y.dim() != 2 or d_x.stride(1) != 1 or d_y.stride(1) != 1:
        raise ValueError("X and Y must be 2-D with unit inner stride")
    if d_x.dtype == torch.float32:
        xdt = X_F32
    elif d_x.dtype == torch.bfloat16:
        xdt = X_BF16
    else:
        raise ValueError("X must be float32 or bfloat16")
    if d_y.dtype != torch.float32:
        raise ValueError("Y must be float32")
    batch = d_x.shape[0]
    ws_bytes = d_workspace.numel() * d_workspace.element_size() if d_workspace is not None else 0
    _check(lib().sqnn_decode_matmul(ctypes.byref(desc), _dev_ptr(d_blob), _dev_ptr(d_mask), _dev_ptr(d_alpha),
                                    _dev_ptr(d_x), xdt, batch, d_x.stride(0), _dev_ptr(d_y), d_y.stride(0),
                                    _dev_ptr(d_workspace), ws_bytes, _dev_ptr(d_status), _stream_ptr(stream)),
           "sqnn_decode_matmul")


def sqnn_decode_matmul_static(desc: Desc, d_blob, d_mask, d_alpha, d_x, d_y, d_status=None, stream=None):
    """Same product as ``sqnn_decode_matmul`` for bfloat16 X with batch >= 16, but the scratch comes
    from an array built into the library instead of a caller-provided workspace: for callers that
    cannot allocate device memory (stream capture, a framework-owned heap, a frozen memory plan).
    Layers whose ``sqnn_workspace_bytes`` exceeds ``STATIC_SCRATCH_BYTES`` are refused.  Calls share
    that one array, so calls that may overlap on the GPU must be serialised by the caller."""
    import torch
    if d_x.dim() != 2 or d_y.dim() != 2 or d_x.stride(1) != 1 or d_y.stride(1) != 1:
        raise ValueError("X and Y must be 2-D with unit inner stride")
    if d_x.dtype != torch.bfloat16 or d_y.dtype != torch.float32:
        raise ValueError("X must be bfloat16 and Y float32")
    _check(lib().sqnn_decode_matmul_static(ctypes.byref(desc), _dev_ptr(d_blob), _dev_ptr(d_mask),
                                           _dev_ptr(d_alpha), _dev_ptr(d_x), X_BF16, d_x.shape[0],
                                           d_x.stride(0), _dev_ptr(d_y), d_y.stride(0), _dev_ptr(d_status),
                                           _stream_ptr(stream)), "sqnn_decode_matmul_static")
