"""Shared test plumbing: oracle-side expectations and device buffers for a synthetic layer."""
import numpy as np

from oracle import oracle as orc
from paper_1905_10138_b200 import sqnn
from paper_1905_10138_b200 import workloads as wl


def oracle_encode(layer):
    care = layer.mask.ravel()
    return [orc.encode_plane(layer.M, layer.planes[i].ravel(), care) for i in range(layer.n_q)]


def oracle_decode(layer, arrays):
    """Decoded planes uint8 [n_q, m, n] from the oracle (all positions, don't-cares included)."""
    out = np.empty((layer.n_q, layer.m, layer.n), dtype=np.uint8)
    for i, (wc, np_, dp) in enumerate(arrays):
        out[i] = orc.decode_plane(layer.M, layer.mn, wc, np_, dp).reshape(layer.m, layer.n)
    return out


def blob_from_oracle(layer, arrays):
    return sqnn.sqnn_pack_host(wl.network_rows(layer.M), layer.n_in, layer.m, layer.n,
                               [a[0].astype(np.uint32) for a in arrays], [a[1] for a in arrays],
                               [a[2] for a in arrays])


def blob_from_library(layer, flags=0):
    planes_words = np.concatenate([wl.pack_bits(layer.planes[i]) for i in range(layer.n_q)])
    return sqnn.sqnn_encode_host(wl.network_rows(layer.M), layer.n_in, layer.m, layer.n, layer.n_q,
                                 planes_words, wl.pack_bits(layer.mask), flags)


class DeviceLayer:
    """Device copies of blob, mask and alpha plus a zeroed status word."""

    def __init__(self, layer, blob):
        import torch
        self.layer = layer
        self.desc = sqnn.sqnn_describe_host(blob)
        self.blob = torch.from_numpy(blob.copy()).cuda()
        self.mask = torch.from_numpy(wl.pack_bits(layer.mask).view(np.int64)).cuda()
        self.alpha = torch.from_numpy(np.ascontiguousarray(layer.alpha, dtype=np.float32)).cuda()
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.words64 = (layer.mn + 63) // 64

    def decode_bits(self):
        import torch
        out = torch.full((self.layer.n_q * self.words64,), -1, dtype=torch.int64, device="cuda")
        sqnn.sqnn_decode(self.desc, self.blob, None, None, sqnn.OUT_BITS, out, self.status)
        torch.cuda.synchronize()
        words = out.cpu().numpy().view(np.uint64).reshape(self.layer.n_q, self.words64)
        return words

    def decode_sink(self):
        import torch
        out = torch.full((2,), -1, dtype=torch.int64, device="cuda")
        sqnn.sqnn_decode(self.desc, self.blob, None, None, sqnn.OUT_SINK, out, self.status)
        torch.cuda.synchronize()
        return int(out.cpu().numpy().view(np.uint64)[0])

    def decode_bf16(self):
        import torch
        out = torch.full((self.layer.m, self.layer.n), float("nan"), dtype=torch.bfloat16, device="cuda")
        sqnn.sqnn_decode(self.desc, self.blob, self.mask, self.alpha, sqnn.OUT_BF16, out, self.status)
        torch.cuda.synchronize()
        return out.view(torch.int16).cpu().numpy().view(np.uint16)

    def matmul(self, x_np, dtype, workspace=True):
        """x_np: float32 [batch, n] (already bf16-representable when dtype is bfloat16)."""
        import torch
        x = torch.from_numpy(x_np).cuda().to(dtype)
        batch = x.shape[0]
        y = torch.full((batch, self.layer.m), float("nan"), dtype=torch.float32, device="cuda")
        ws_bytes = sqnn.sqnn_workspace_bytes(self.desc, batch)
        ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda") if workspace else None
        sqnn.sqnn_decode_matmul(self.desc, self.blob, self.mask, self.alpha, x, y, ws, self.status)
        torch.cuda.synchronize()
        return y.cpu().numpy()

    def status_value(self):
        return int(self.status.cpu().item())


def rel_err(y, ref):
    """max |y - ref| / max(|ref|, rms(ref)) over all outputs."""
    ref = np.asarray(ref, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    rms = np.sqrt(np.mean(ref ** 2))
    den = np.maximum(np.abs(ref), rms if rms > 0 else 1.0)
    return float(np.max(np.abs(y - ref) / den))
