"""Seeded synthetic tensors shared by the tests, the benchmark and the CPU checker.

This module holds no arithmetic of the method itself: it only draws numbers.  A
counter-based generator (SplitMix64, Steele/Lea/Flood 2014: state = seed + (i+1)*golden
gamma, followed by the two xor-shift-multiply finalisers) gives element i of a stream
without any sequential state, so a tensor is the same whatever order or chunking it
is produced in.

Distributions follow the workload recipe: activations U(-1, 1); weights N(0, 1/fan_in)
(second argument is the variance); biases N(0, 0.01) kept in fp32.  Normals are made
with the Box-Muller transform in double precision.  Everything destined for fp16
storage is rounded once with numpy's round-to-nearest-even cast.
"""
from __future__ import annotations

import hashlib

import numpy as np

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _splitmix64(seed: int, start: int, count: int) -> np.ndarray:
    """Elements start .. start+count-1 of the SplitMix64 stream of `seed` (uint64)."""
    with np.errstate(over="ignore"):
        idx = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + idx * _GAMMA
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def stream_seed(*names) -> int:
    """64-bit seed derived from a tuple of names/ints (config id, tensor id, ...)."""
    h = hashlib.sha256("/".join(str(n) for n in names).encode()).digest()
    return int.from_bytes(h[:8], "little")


def unit_uniform(seed: int, count: int, start: int = 0) -> np.ndarray:
    """float64 uniforms strictly inside (0, 1): (top 24 bits + 0.5) / 2^24."""
    out = np.empty(count, dtype=np.float64)
    for o in range(0, count, _CHUNK):
        c = min(_CHUNK, count - o)
        bits = _splitmix64(seed, start + o, c) >> np.uint64(40)
        out[o:o + c] = (bits.astype(np.float64) + 0.5) * (1.0 / (1 << 24))
    return out


def uniform_pm1(seed: int, shape) -> np.ndarray:
    """U(-1, 1) rounded to fp16."""
    n = int(np.prod(shape))
    return (2.0 * unit_uniform(seed, n) - 1.0).astype(np.float16).reshape(shape)


def normal(seed: int, shape, std: float) -> np.ndarray:
    """N(0, std^2) in float64 (Box-Muller on consecutive pairs of the stream)."""
    n = int(np.prod(shape))
    out = np.empty(n + (n & 1), dtype=np.float64)
    half = out.size // 2
    for o in range(0, half, _CHUNK // 2):
        c = min(_CHUNK // 2, half - o)
        u = unit_uniform(seed, 2 * c, start=2 * o)
        r = np.sqrt(-2.0 * np.log(u[0::2]))
        t = 2.0 * np.pi * u[1::2]
        out[2 * o:2 * (o + c):2] = r * np.cos(t)
        out[2 * o + 1:2 * (o + c):2] = r * np.sin(t)
    return (out[:n] * std).reshape(shape)


def weight_f16(seed: int, shape, fan_in: int) -> np.ndarray:
    """N(0, 1/fan_in) rounded to fp16."""
    return normal(seed, shape, fan_in ** -0.5).astype(np.float16)


def bias_f32(seed: int, shape) -> np.ndarray:
    """N(0, 0.01) (std 0.1) in fp32."""
    return normal(seed, shape, 0.1).astype(np.float32)


def layer_params(tag: str, layers) -> list:
    """Weights and biases for every parametrised layer of a layer list.

    Returns a list with one entry per layer: (w_f16, bias_f32) or None.  Weight layout
    is [cout][kh][kw][cin/groups]; a fully connected layer is [cout][cin] with cin in
    NHWC-flatten order.  The stream of a tensor depends on (tag, layer index) only.
    """
    out = []
    for i, l in enumerate(layers):
        if l["op"] in ("conv", "dwconv"):
            cg = l["cin"] // l["groups"]
            shape = (l["cout"], l["kh"], l["kw"], cg)
            fan = l["kh"] * l["kw"] * cg
        elif l["op"] == "fc":
            shape = (l["cout"], l["cin"])
            fan = l["cin"]
        else:
            out.append(None)
            continue
        out.append((weight_f16(stream_seed(tag, i, "w"), shape, fan),
                    bias_f32(stream_seed(tag, i, "b"), (l["cout"],))))
    return out


def network_input(tag: str, n: int, h: int, w: int, c: int) -> np.ndarray:
    """NHWC fp16 input, U(-1, 1)."""
    return uniform_pm1(stream_seed(tag, "x"), (n, h, w, c))
