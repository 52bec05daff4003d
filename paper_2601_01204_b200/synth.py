"""Seeded synthetic Q/K/V for the compressed-KV stream (numpy, host side).

This module is the single definition of the input bytes.  It contains none of
the method's arithmetic (no pooling, scoring, quantisation or attention): only
a counter-based integer hash, a sum of twelve 16-bit uniform fields, and the
round-to-nearest-even conversion to bf16.  The CUDA generator kernel of the
library implements the same integer recipe and is tested byte-for-byte against
this file.

Recipe for element (layer, frame, tensor, head, token, channel):

    key  = mix64(mix64(mix64(seed ^ C0) + layer*C1 + frame) + tensor)  (per tensor)
    e    = (head * n_tokens + token) * head_dim + channel
    w_i  = mix64(key + 3*e + i), i = 0, 1, 2        (three 64-bit words)
    u    = sum of the twelve 16-bit fields of w_0, w_1, w_2
    x    = (u - 6*65535) * 2**-16                   (exact in fp32)
    x   *= 15 on the layer's outlier channels of that head (keys only)
    out  = bf16(x), round to nearest even

`u` is an Irwin-Hall(12) variate: mean 6*65535, variance 65536**2 - 1, so `x`
has unit variance (to 1e-10), support (-6, 6) and excess kurtosis -0.1.  It
stands in for N(0, 1).  Four outlier key channels per head, fixed per layer for
the whole stream, reproduce the channel-wise key outliers that motivate
per-channel key quantisation (Fig. 3 of the paper).
"""
from __future__ import annotations

import numpy as np

TENSOR_Q, TENSOR_K, TENSOR_V = 0, 1, 2
N_OUTLIER_CHANNELS = 4
OUTLIER_GAIN = 15.0

_M64 = (1 << 64) - 1
_C0 = 0x9E3779B97F4A7C15
_C1 = 0xD1B54A32D192ED03
_MIX_A = 0xBF58476D1CE4E5B9
_MIX_B = 0x94D049BB133111EB


def mix64_int(x: int) -> int:
    """64-bit finaliser (xor-shift-multiply), Python ints."""
    x &= _M64
    x ^= x >> 30
    x = (x * _MIX_A) & _M64
    x ^= x >> 27
    x = (x * _MIX_B) & _M64
    x ^= x >> 31
    return x


def _mix64_np(x: np.ndarray) -> np.ndarray:
    x = x ^ (x >> np.uint64(30))
    x = x * np.uint64(_MIX_A)
    x = x ^ (x >> np.uint64(27))
    x = x * np.uint64(_MIX_B)
    x = x ^ (x >> np.uint64(31))
    return x


def tensor_key(seed: int, layer: int, frame: int, tensor: int) -> int:
    """64-bit stream key of one (layer, frame, tensor)."""
    k = mix64_int(seed ^ _C0)
    k = mix64_int((k + layer * _C1 + frame) & _M64)
    k = mix64_int((k + tensor) & _M64)
    return k


def outlier_channels(seed: int, layer: int, n_heads: int, head_dim: int) -> np.ndarray:
    """int32[n_heads][4]: the outlier key channels of each head of one layer.

    Drawn without replacement from a hash sequence of (seed, layer, head);
    constant over the stream.
    """
    out = np.zeros((n_heads, N_OUTLIER_CHANNELS), dtype=np.int32)
    for h in range(n_heads):
        base = mix64_int((mix64_int(seed ^ _C1) + layer * _C0 + h) & _M64)
        chosen: list[int] = []
        ctr = 0
        while len(chosen) < N_OUTLIER_CHANNELS:
            c = mix64_int((base + ctr) & _M64) % head_dim
            ctr += 1
            if c not in chosen:
                chosen.append(c)
        out[h] = sorted(chosen)
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even; finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp32, exact."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def gen_tensor_bits(seed: int, layer: int, frame: int, tensor: int,
                    n_heads: int, n_tokens: int, head_dim: int) -> np.ndarray:
    """uint16[n_heads][n_tokens][head_dim]: bf16 bit patterns of one tensor."""
    key = np.uint64(tensor_key(seed, layer, frame, tensor))
    count = n_heads * n_tokens * head_dim
    e = np.arange(count, dtype=np.uint64) * np.uint64(3) + key
    u = np.zeros(count, dtype=np.int64)
    with np.errstate(over="ignore"):
        for i in range(3):
            w = _mix64_np(e + np.uint64(i))
            for s in (0, 16, 32, 48):
                u += ((w >> np.uint64(s)) & np.uint64(0xFFFF)).astype(np.int64)
    x = (u - 6 * 65535).astype(np.float32) * np.float32(2.0 ** -16)
    x = x.reshape(n_heads, n_tokens, head_dim)
    if tensor == TENSOR_K:
        oc = outlier_channels(seed, layer, n_heads, head_dim)
        for h in range(n_heads):
            x[h][:, oc[h]] *= np.float32(OUTLIER_GAIN)
    return f32_to_bf16_bits(x)


def gen_frame(seed: int, layer: int, frame: int, n_heads: int, n_tokens: int, head_dim: int):
    """(Q, K, V) bf16 bit patterns, each uint16[n_heads][n_tokens][head_dim]."""
    return tuple(gen_tensor_bits(seed, layer, frame, t, n_heads, n_tokens, head_dim)
                 for t in (TENSOR_Q, TENSOR_K, TENSOR_V))
