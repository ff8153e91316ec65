"""Seeded synthetic inputs shaped like the paper's Llama-3 workloads.

This module only draws random tensors and rounds them to bf16 bit patterns; it holds none of
the method's arithmetic (no Hadamard, no quantizer, no product) so that the CUDA path and the
CPU oracle can both be fed from it without sharing any of the method's code.

Recipe (stands in for the Llama-3 weights and WikiText2 activations the paper uses, Sec. 4,
which are not available offline): activations N(0, 1) with floor(0.01 K) outlier channels,
shared by all tokens, scaled x50; for prefill shapes each token row is additionally scaled by
|t|, t ~ Student-t with 3 degrees of freedom; weights N(0, sigma = 0.02).  Everything is
rounded once to bf16 (round to nearest even) and travels as uint16 bit patterns.
"""
from __future__ import annotations

import zlib

import numpy as np


def _rng(seed: int, tag: str) -> np.random.Generator:
    """One independent counter-based stream per (seed, tensor tag)."""
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFF, zlib.crc32(tag.encode())]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round binary32 to bf16 (ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def activations(M: int, K: int, seed: int = 0, tag: str = "x", heavy_tail: bool = False) -> np.ndarray:
    """bf16 bits [M, K]: N(0,1), 1 % outlier channels x50, optional per-token Student-t(3) scale."""
    g = _rng(seed, "act:" + tag)
    x = g.standard_normal((M, K), dtype=np.float32)
    n_out = K // 100
    if n_out > 0:
        idx = g.choice(K, size=n_out, replace=False)
        x[:, idx] *= 50.0
    if heavy_tail:
        t = np.abs(g.standard_t(3.0, size=(M, 1))).astype(np.float32)
        x *= t
    return f32_to_bf16_bits(x)


def weights(N: int, K: int, seed: int = 0, tag: str = "w") -> np.ndarray:
    """bf16 bits [N, K] (out x in): N(0, sigma = 0.02)."""
    g = _rng(seed, "wgt:" + tag)
    w = g.standard_normal((N, K), dtype=np.float32) * np.float32(0.02)
    return f32_to_bf16_bits(w)


def int4_codes(rows: int, cols: int, seed: int = 0, tag: str = "q", lo: int = -8, hi: int = 7) -> np.ndarray:
    """int8 [rows, cols] drawn uniformly from lo..hi (full two's-complement nibble range by default)."""
    g = _rng(seed, "codes:" + tag)
    return g.integers(lo, hi + 1, size=(rows, cols), dtype=np.int8)


def scales(rows: int, seed: int = 0, tag: str = "s") -> np.ndarray:
    """float32 [rows], log-uniform in [2^-8, 2^-2]."""
    g = _rng(seed, "scales:" + tag)
    return np.exp2(g.uniform(-8.0, -2.0, size=rows)).astype(np.float32)


# Shapes of the workloads (K, Kp, N) per linear.
LLAMA_1B = {
    "qkv": (2048, 2176, 3072),
    "o": (2048, 2176, 2048),
    "gate": (2048, 2176, 8192),
    "up": (2048, 2176, 8192),
    "down": (8192, 8704, 2048),
}
LLAMA_8B = {
    "qkv": (4096, 4352, 6144),
    "gate": (4096, 4352, 14336),
    "up": (4096, 4352, 14336),
    "down": (14336, 15360, 4096),
}
# Down projections at the expansion sizes of the paper's Table 1 (8192 -> 2048 and 14336 -> 4096).
TABLE1_1B_DOWN = {
    "kp8960": (8192, 8960, 2048),
    "kp9728": (8192, 9728, 2048),
    "kp10240": (8192, 10240, 2048),
    "kp12288": (8192, 12288, 2048),
}
TABLE1_8B_DOWN = {
    "kp15360": (14336, 15360, 4096),
    "kp18432": (14336, 18432, 4096),
    "kp19968": (14336, 19968, 4096),
    "kp22016": (14336, 22016, 4096),
}
# Attention output projections with the head-wise rotation expanded (K, K', N, heads): 32 heads of 64 -> 72 / 80
# channels (Llama-3.2-1B-like) and of 128 -> 144 / 160 channels (Llama-3-8B-like).
HEADS_1B_O = {
    "hd72": (2048, 2304, 2048, 32),
    "hd80": (2048, 2560, 2048, 32),
}
HEADS_8B_O = {
    "hd144": (4096, 4608, 4096, 32),
    "hd160": (4096, 5120, 4096, 32),
}
SWEEP_4096 = {
    "kp4096": (4096, 4096, 4096),
    "kp4352": (4096, 4352, 4096),
    "kp4608": (4096, 4608, 4096),
    "kp5120": (4096, 5120, 4096),
}
