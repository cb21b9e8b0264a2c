"""Seeded synthetic layers and the packed-factor format.

This module only makes inputs and converts between one-byte-per-bit arrays and
the packed words of the C ABI.  It holds none of the method's arithmetic: no
Boolean product, no masking, no GEMM.  It needs numpy only (no torch, no CUDA),
so the CPU checker and the CUDA path can both be fed from the same buffers.

Layer shapes follow the layers the paper prunes (LeNet-5 FC1 500x800 with rank
16; AlexNet FC layers cut into 512x512 blocks with rank 32) plus a lowered 3x3
convolution and a transformer feed-forward layer.  Weights are zero-mean
Gaussians (the paper's assumption for trained layers); factor bits are i.i.d.
Bernoulli(p), the model behind Eq. 7, with p chosen so the decoded mask has
density d:  1 - d = (1 - p*p)^k.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Layer:
    """Geometry of one pruned layer: W is [rows, cols] = [out, in]."""

    name: str
    rows: int
    cols: int
    tile_rows: int
    tile_cols: int
    rank: int
    density: float
    w_std: float = 0.02
    batches: tuple = ()
    seed: int = 0

    @property
    def grid(self):
        return (-(-self.rows // self.tile_rows), -(-self.cols // self.tile_cols))

    @property
    def kw(self):
        return (self.rank + 31) // 32

    @property
    def p(self):
        """Bernoulli parameter of the factor bits (Eq. 7 with S = 1 - d, S_p = S_z = 1 - p)."""
        return math.sqrt(1.0 - (1.0 - self.density) ** (1.0 / self.rank))

    @property
    def index_bytes(self):
        """Bytes of the packed factors when k is a multiple of 8: k (tm + tn) / 8 per tile."""
        gr, gc = self.grid
        return gr * gc * self.rank * (self.tile_rows + self.tile_cols) // 8

    @property
    def mask_words(self):
        return self.rows * ((self.cols + 31) // 32)


CONFIGS = {
    "lenet_fc1": Layer("lenet_fc1", 500, 800, 500, 800, 16, 0.05, 0.05, (32,)),
    "decode_4096": Layer("decode_4096", 4096, 4096, 256, 256, 8, 0.10, 0.0, ()),
    "alexnet_fc": Layer("alexnet_fc", 4096, 9216, 512, 512, 32, 0.09, 0.01, (1, 16, 128)),
    "conv3x3_256": Layer("conv3x3_256", 256, 2304, 128, 256, 16, 0.30, 0.02, (12544,)),
    "ffn_16384x4096": Layer("ffn_16384x4096", 16384, 4096, 1024, 1024, 64, 0.20, 0.02, (4096,)),
}
# Not one of the five layer shapes: the decode-only configuration repeated over a grid 64 times larger
# (same 256 x 256 tiles, rank and density; 128 MiB of mask), so that a decode kernel's steady-state
# bandwidth can be measured on something larger than L2.
CONFIGS["decode_32768"] = Layer("decode_32768", 32768, 32768, 256, 256, 8, 0.10, 0.0, ())
CONFIG_ORDER = ["lenet_fc1", "decode_4096", "alexnet_fc", "conv3x3_256", "ffn_16384x4096"]

_ARRAY_IDS = {"Ip": 1, "Iz": 2, "W": 3, "X": 4}


def _rng(layer: Layer, array: str, extra: int = 0) -> np.random.Generator:
    """Independent counter-based stream per (seed, layer name, array)."""
    name_key = int.from_bytes(layer.name.encode()[:7].ljust(7, b"\0"), "little")
    key = (layer.seed & 0xFFFFFFFF) | (_ARRAY_IDS[array] << 32) | (extra << 40)
    return np.random.Generator(np.random.Philox(key=[key, name_key]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_factors(layer: Layer, p: float | None = None):
    """Unpacked factors: Ip uint8 [GR, GC, tm, k], Iz uint8 [GR, GC, k, tn]."""
    gr, gc = layer.grid
    p = layer.p if p is None else p
    thr = np.uint32(min(int(p * 2.0**32), 2**32 - 1))
    ip = (_rng(layer, "Ip").integers(0, 2**32, size=(gr, gc, layer.tile_rows, layer.rank), dtype=np.uint32) < thr)
    iz = (_rng(layer, "Iz").integers(0, 2**32, size=(gr, gc, layer.rank, layer.tile_cols), dtype=np.uint32) < thr)
    return ip.astype(np.uint8), iz.astype(np.uint8)


def make_weights(layer: Layer) -> np.ndarray:
    """W as bf16 bit patterns, uint16 [rows, cols], ~ N(0, w_std^2)."""
    w = _rng(layer, "W").standard_normal((layer.rows, layer.cols), dtype=np.float32) * np.float32(layer.w_std)
    return f32_to_bf16_bits(w)


def make_activations(layer: Layer, batch: int) -> np.ndarray:
    """X as bf16 bit patterns, uint16 [batch, cols], ~ N(0, 1)."""
    x = _rng(layer, "X", extra=batch).standard_normal((batch, layer.cols), dtype=np.float32)
    return f32_to_bf16_bits(x)


# ----------------------------------------------------------------------------
# Packed formats of the C ABI (KW = ceil(k / 32) words per row of Ip / column of Iz)
# ----------------------------------------------------------------------------
def _pack_last_axis(bits: np.ndarray) -> np.ndarray:
    """Pack the last axis into little-endian uint32 words: bit (l % 32) of word l // 32."""
    n = bits.shape[-1]
    nw = (n + 31) // 32
    pad = nw * 32 - n
    if pad:
        bits = np.concatenate([bits, np.zeros(bits.shape[:-1] + (pad,), dtype=np.uint8)], axis=-1)
    by = np.packbits(np.ascontiguousarray(bits, dtype=np.uint8), axis=-1, bitorder="little")
    return np.ascontiguousarray(by).view("<u4")


def pack_ip(Ip: np.ndarray) -> np.ndarray:
    """[GR, GC, tm, k] bytes -> uint32 [GR*GC*tm*KW]; word w of row i holds Ip[i, 32w .. 32w+31]."""
    return _pack_last_axis(Ip).reshape(-1).copy()


def pack_iz(Iz: np.ndarray) -> np.ndarray:
    """[GR, GC, k, tn] bytes -> uint32 [GR*GC*tn*KW]; word w of column j holds Iz[32w .. 32w+31, j]."""
    return _pack_last_axis(np.swapaxes(Iz, 2, 3)).reshape(-1).copy()


def pack_ranked(Ip: np.ndarray, Iz: np.ndarray, ranks: np.ndarray):
    """Ranked layout: tile t keeps its first ranks[t] bits, packed with ceil(ranks[t] / 32) words per row / column,
    tiles one after the other.  Returns (ip_words, iz_words, ip_offset, iz_offset), offsets in words (int64)."""
    gr, gc, tm, kmax = Ip.shape
    tn = Iz.shape[3]
    ranks = np.asarray(ranks, dtype=np.int64).ravel()
    ipw, izw, ipo, izo = [], [], [], []
    n_ip = n_iz = 0
    for t in range(gr * gc):
        k = int(ranks[t])
        ipo.append(n_ip)
        izo.append(n_iz)
        if k:
            a = _pack_last_axis(Ip.reshape(gr * gc, tm, kmax)[t][:, :k]).reshape(-1)
            z = _pack_last_axis(np.swapaxes(Iz.reshape(gr * gc, kmax, tn)[t][:k, :], 0, 1)).reshape(-1)
            ipw.append(a)
            izw.append(z)
            n_ip += a.size
            n_iz += z.size
    cat = lambda parts: np.concatenate(parts).astype(np.uint32) if parts else np.zeros(0, dtype=np.uint32)
    # keep the arrays non-empty and padded to whole 16-byte vectors
    pad = lambda a: np.concatenate([a, np.zeros((-a.size) % 4 + (4 if a.size == 0 else 0), dtype=np.uint32)])
    return pad(cat(ipw)), pad(cat(izw)), np.array(ipo, dtype=np.int64), np.array(izo, dtype=np.int64)


def pack_mask(M: np.ndarray) -> np.ndarray:
    """[rows, cols] bytes -> uint32 [rows, ceil(cols/32)]; bit (c % 32) of word c // 32 = M[r, c]."""
    return _pack_last_axis(M)


def unpack_mask(words: np.ndarray, cols: int) -> np.ndarray:
    by = np.ascontiguousarray(words, dtype="<u4").view(np.uint8)
    return np.unpackbits(by, axis=-1, bitorder="little")[..., :cols]


def popcount_words(words: np.ndarray) -> int:
    return int(np.unpackbits(np.ascontiguousarray(words).view(np.uint8)).sum(dtype=np.int64))
