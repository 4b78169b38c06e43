"""Seeded synthetic layers shaped like the paper's workloads.

This module only *draws inputs*: weights, pruning masks, binary-code planes with
their per-row scales, the random XOR-gate network M and activations.  It holds
none of the method's arithmetic (no encryption, decryption, patching or
product), so both the CUDA library's tests and the CPU oracle's tests can take
their inputs from it.  numpy only.

Randomness: ``numpy.random.Generator(PCG64(seed))`` with seed = 1000 * cfg + k,
k = 1 weights / plane bits, 2 mask, 3 network M, 4 activations, 5 scales.  Large Bernoulli
arrays (masks and the bit-planes of the decode-only sweep) are drawn in chunks of 2^24, chunk j
from ``PCG64(seed).jumped(j)``, so that the chunks can be drawn by several threads and the result
does not depend on how many there are.

The paper's experiments run on trained AlexNet / LSTM / ResNet weights
(Section 4, Table 2); those are not available, so each layer here keeps only
the shape, pruning rate and bit width, with the randomness assumptions of
Section 3.3 (random don't-care locations, equiprobable care bits).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(int(seed)))


def xor_network(n_out: int, n_in: int, seed: int) -> np.ndarray:
    """M in {0,1}^{n_out x n_in}, every entry 0 or 1 with equal probability (Section 3.1)."""
    return _rng(seed).integers(0, 2, size=(n_out, n_in), dtype=np.uint8)


def network_rows(M: np.ndarray) -> np.ndarray:
    """Row j of M as an integer, bit t = M[j, t] (the form the C interface takes)."""
    n_out, n_in = M.shape
    assert n_in <= 32
    w = (1 << np.arange(n_in, dtype=np.uint64))
    return (M.astype(np.uint64) * w).sum(axis=1).astype(np.uint32)


_CHUNK = 1 << 24


def _chunked(total: int, seed: int, draw) -> np.ndarray:
    """uint8 array of ``total`` entries; chunk j (2^24 entries) = draw(Generator(PCG64(seed).jumped(j)), count).
    Chunks are drawn by a small thread pool (numpy's generators release the interpreter lock)."""
    from concurrent.futures import ThreadPoolExecutor
    import os
    out = np.empty(total, dtype=np.uint8)
    starts = list(range(0, total, _CHUNK))

    def one(j):
        a = starts[j]
        b = min(total, a + _CHUNK)
        rng = np.random.Generator(np.random.PCG64(int(seed)).jumped(j))
        out[a:b] = draw(rng, b - a)

    if len(starts) == 1:
        one(0)
    else:
        with ThreadPoolExecutor(max_workers=min(len(starts), os.cpu_count() or 4)) as ex:
            list(ex.map(one, range(len(starts))))
    return out


def network_rows64(M: np.ndarray) -> np.ndarray:
    """As network_rows for up to 64 inputs (uint64 rows)."""
    n_out, n_in = M.shape
    assert n_in <= 64
    out = np.zeros(n_out, dtype=np.uint64)
    for t in range(n_in):
        out |= M[:, t].astype(np.uint64) << np.uint64(t)
    return out


def bernoulli_mask(shape, prune_rate: float, seed: int) -> np.ndarray:
    """1 = kept (care) with probability 1 - prune_rate, independently per weight."""
    keep = np.float32(1.0 - prune_rate)
    total = int(np.prod(shape))
    return _chunked(total, seed, lambda rng, cnt: rng.random(cnt, dtype=np.float32) < keep).reshape(shape)


def bernoulli_bits(total: int, seed: int) -> np.ndarray:
    """``total`` bits, 0 or 1 with equal probability (one random byte gives eight of them)."""
    return _chunked(total, seed, lambda rng, cnt: np.unpackbits(
        rng.integers(0, 256, size=(cnt + 7) // 8, dtype=np.uint8), bitorder="little", count=cnt))


def magnitude_mask(w: np.ndarray, keep_fraction: float) -> np.ndarray:
    """Keep exactly round(keep_fraction * size) weights of largest |w| over the whole
    layer; equal magnitudes are kept lower flat index first."""
    a = np.abs(w).ravel()
    total = a.size
    keep = int(round(keep_fraction * total))
    if keep <= 0:
        return np.zeros(w.shape, dtype=np.uint8)
    if keep >= total:
        return np.ones(w.shape, dtype=np.uint8)
    kth = np.partition(a, total - keep)[total - keep]
    mask = a > kth
    need = keep - int(mask.sum())
    if need > 0:
        ties = np.flatnonzero(a == kth)[:need]
        mask[ties] = True
    return mask.astype(np.uint8).reshape(w.shape)


def binary_code_quantize(w: np.ndarray, mask: np.ndarray, n_q: int):
    """Greedy binary-code quantization per row over the unpruned weights.

    r_0 = w; for i = 1..n_q: b_i = sign(r_{i-1}) (sign(0) = +1),
    alpha_i = mean |r_{i-1}| over the row's unpruned entries, r_i = r_{i-1} - alpha_i b_i.
    fp64 throughout, alpha stored as fp32.  A row without unpruned entries gets alpha = 0.
    Returns planes uint8 [n_q, m, n] (1 <-> +1) and alpha float32 [m, n_q]."""
    m, n = w.shape
    r = w.astype(np.float64).copy()
    keep = mask.astype(bool)
    cnt = keep.sum(axis=1)
    planes = np.empty((n_q, m, n), dtype=np.uint8)
    alpha = np.zeros((m, n_q), dtype=np.float32)
    for i in range(n_q):
        b = r >= 0
        planes[i] = b
        s = np.where(keep, np.abs(r), 0.0).sum(axis=1)
        a = np.where(cnt > 0, s / np.maximum(cnt, 1), 0.0)
        alpha[:, i] = a.astype(np.float32)
        r -= np.where(b, 1.0, -1.0) * a[:, None]
    return planes, alpha


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 values rounded to the nearest bf16 (ties to even), returned as fp32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16 << 16
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x_bf16_as_f32: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already exactly representable in bf16."""
    return (np.ascontiguousarray(x_bf16_as_f32, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def pack_bits(bits: np.ndarray) -> np.ndarray:
    """Flat 0/1 bytes -> uint64 words, bit p of the vector = (word[p >> 6] >> (p & 63)) & 1."""
    flat = np.ascontiguousarray(bits, dtype=np.uint8).ravel()
    by = np.packbits(flat, bitorder="little")
    pad = (-by.size) % 8
    if pad:
        by = np.concatenate([by, np.zeros(pad, dtype=np.uint8)])
    return by.view(np.uint64).copy()


def unpack_bits(words: np.ndarray, count: int) -> np.ndarray:
    """Inverse of pack_bits: uint64 words -> ``count`` 0/1 bytes."""
    by = np.ascontiguousarray(words).view(np.uint8)
    return np.unpackbits(by, bitorder="little", count=count)


@dataclass
class Layer:
    """One synthetic layer: everything the encoder, the decoder and the product take."""
    name: str
    cfg: int
    m: int
    n: int
    n_q: int
    n_out: int
    n_in: int
    prune_rate: float
    M: np.ndarray            # uint8 [n_out, n_in]
    planes: np.ndarray       # uint8 [n_q, m, n]
    mask: np.ndarray         # uint8 [m, n], 1 = care
    alpha: np.ndarray        # float32 [m, n_q]
    x_dtype: str             # "f32" or "bf16"
    batches: tuple
    seed_x: int
    extra: dict = field(default_factory=dict)

    @property
    def mn(self) -> int:
        return self.m * self.n

    def activations(self, batch: int) -> np.ndarray:
        """X [batch, n] fp32 values N(0,1); already rounded to bf16 values when x_dtype is bf16."""
        x = _rng(self.seed_x + 100 * batch).standard_normal((batch, self.n), dtype=np.float32)
        return round_to_bf16(x) if self.x_dtype == "bf16" else x


_SHAPES = {
    # cfg: (name, m, n, n_q, n_out, n_in, prune, weight law, mask law, x dtype, batches)
    1: ("tiny-fc", 256, 256, 1, 80, 8, 0.90, ("normal", 1.0), "bernoulli", "f32", (1,)),
    2: ("alexnet-fc6", 4096, 9216, 1, 100, 10, 0.91, ("normal", 0.01), "magnitude", "bf16", (1, 64)),
    3: ("lstm-gates", 6000, 3000, 2, 60, 12, 0.80, ("uniform", 0.05), "magnitude", "bf16", (1, 8, 32)),
    4: ("ffn", 4096, 16384, 3, 40, 12, 0.70, ("normal", 0.02), "magnitude", "bf16", (16, 128, 512)),
}


def make_layer(cfg: int, m: int | None = None, n: int | None = None) -> Layer:
    """Configs 1-4.  ``m`` / ``n`` override the shape (same recipe, smaller layer) for tests."""
    name, m0, n0, n_q, n_out, n_in, prune, wlaw, mlaw, xdt, batches = _SHAPES[cfg]
    m = m0 if m is None else m
    n = n0 if n is None else n
    base = 1000 * cfg
    rng = _rng(base + 1)
    if wlaw[0] == "normal":
        w = rng.standard_normal((m, n), dtype=np.float32) * np.float32(wlaw[1])
    else:
        w = (rng.random((m, n), dtype=np.float32) * 2.0 - 1.0).astype(np.float32) * np.float32(wlaw[1])
    if mlaw == "bernoulli":
        mask = bernoulli_mask((m, n), prune, base + 2)
    else:
        mask = magnitude_mask(w, 1.0 - prune)
    planes, alpha = binary_code_quantize(w, mask, n_q)
    M = xor_network(n_out, n_in, base + 3)
    return Layer(name=name, cfg=cfg, m=m, n=n, n_q=n_q, n_out=n_out, n_in=n_in, prune_rate=prune,
                 M=M, planes=planes, mask=mask, alpha=alpha, x_dtype=xdt, batches=batches,
                 seed_x=base + 4)


def make_conv_layer(c_out: int, c_in: int, kh: int, kw: int, n_q: int = 2, prune: float = 0.70,
                    n_out: int = 40, n_in: int = 12, seed: int = 1) -> Layer:
    """A convolution layer in the shape of the paper's ResNet32 experiment (Section 4: 2-bit codes, 70 %
    pruned): a 4-D weight tensor [c_out][c_in][kh][kw] ~ N(0, sqrt(2 / fan_in)), flattened in that order
    (Section 3.1), i.e. a matrix of c_out rows and c_in * kh * kw columns; magnitude pruning over the layer,
    greedy binary codes per output channel.  Its product is the layer applied to im2col patches."""
    base = 7000 + 10 * int(seed)
    fan_in = c_in * kh * kw
    w4 = _rng(base + 1).standard_normal((c_out, c_in, kh, kw), dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))
    w = np.ascontiguousarray(w4).reshape(c_out, fan_in)
    mask = magnitude_mask(w, 1.0 - prune)
    planes, alpha = binary_code_quantize(w, mask, n_q)
    return Layer(name=f"conv-{c_out}x{c_in}x{kh}x{kw}", cfg=7, m=c_out, n=fan_in, n_q=n_q, n_out=n_out, n_in=n_in,
                 prune_rate=prune, M=xor_network(n_out, n_in, base + 3), planes=planes, mask=mask, alpha=alpha,
                 x_dtype="bf16", batches=(1, 8, 64), seed_x=base + 4)


SWEEP_PRUNE = (0.60, 0.80, 0.90, 0.95)
SWEEP_NETS = ((40, 16), (80, 16), (100, 10), (200, 10))


def make_sweep_layer(i_s: int, i_m: int, m: int = 32768, n: int = 32768) -> Layer:
    """Config 5: one point of the decode-only sweep.  Plane bits are Bernoulli(1/2) directly,
    the mask prunes each weight independently with probability S, alpha_r ~ U(0.5, 1.5)."""
    prune = SWEEP_PRUNE[i_s]
    n_out, n_in = SWEEP_NETS[i_m]
    base = 5000 + 10 * i_s + i_m
    total = m * n
    planes = bernoulli_bits(total, base + 1)
    mask = bernoulli_mask((m, n), prune, base + 2)
    alpha = (_rng(base + 5).random((m, 1), dtype=np.float32) + np.float32(0.5)).astype(np.float32)
    M = xor_network(n_out, n_in, base + 3)
    return Layer(name=f"sweep-S{prune:.2f}-{n_out}x{n_in}", cfg=5, m=m, n=n, n_q=1, n_out=n_out,
                 n_in=n_in, prune_rate=prune, M=M, planes=planes.reshape(1, m, n), mask=mask,
                 alpha=alpha, x_dtype="bf16", batches=(), seed_x=base + 4)


def synthetic_plane(count: int, prune_rate: float, seed: int):
    """The experiment of Section 3.3: ``count`` elements, each a don't-care with probability
    ``prune_rate``, otherwise 0 or 1 with equal probability.  Returns (bits, care) uint8."""
    rng = _rng(seed)
    care = (rng.random(count) >= prune_rate).astype(np.uint8)
    bits = rng.integers(0, 2, size=count, dtype=np.uint8)
    return bits, care
