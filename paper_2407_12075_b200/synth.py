"""Seeded synthetic inputs shaped like the paper's workloads.

This module is the only code shared by the CUDA path's tests/benchmarks and the
CPU oracle: it produces *buffers* (numpy arrays) and contains none of the
method's arithmetic (no aggregation, no tiling, no contraction).

Generator: counter based.  Element ``i`` of stream ``s`` under seed ``d`` is a
function of (d, s, i) only, so any slice can be produced independently and the
result does not depend on a library's RNG version.  The 64-bit mixer is the
finaliser of the published SplitMix64 generator applied to
``(d * 0x9E3779B97F4A7C15 + s * 0xD1B54A32D192ED03 + i)``.  Uniforms use the top
53 bits; normals use Box-Muller on two independent uniforms, in fp64.

Streams: 0 = activations, 1 + l = weights W of layer l, 100 + l = the optional
separate tensor A of layer l, 200 + l = bias of layer l.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_STREAM = np.uint64(0xD1B54A32D192ED03)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _mix(z: np.ndarray) -> np.ndarray:
    z = z.copy()
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def _u01(seed: int, stream: int, start: int, count: int, lane: int) -> np.ndarray:
    """Uniform in (0,1): counter 2*i + lane of the (seed, stream) sequence."""
    with np.errstate(over="ignore"):
        base = np.uint64(seed) * _GOLDEN + np.uint64(stream) * _STREAM
        ctr = (np.arange(start, start + count, dtype=np.uint64) * np.uint64(2)
               + np.uint64(lane)) + base
        bits = _mix(ctr * _GOLDEN) >> np.uint64(11)
    return (bits.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def uniform(seed: int, stream: int, count: int, lo: float = 0.0, hi: float = 1.0,
            start: int = 0) -> np.ndarray:
    """fp32 uniforms in (lo, hi)."""
    out = np.empty(count, dtype=np.float32)
    for s in range(0, count, _CHUNK):
        c = min(_CHUNK, count - s)
        out[s:s + c] = (lo + (hi - lo) * _u01(seed, stream, start + s, c, 0)).astype(np.float32)
    return out


def normal(seed: int, stream: int, count: int, sigma: float = 1.0, start: int = 0) -> np.ndarray:
    """fp32 normals N(0, sigma^2) by Box-Muller (cosine branch)."""
    out = np.empty(count, dtype=np.float32)
    for s in range(0, count, _CHUNK):
        c = min(_CHUNK, count - s)
        u1 = _u01(seed, stream, start + s, c, 0)
        u2 = _u01(seed, stream, start + s, c, 1)
        out[s:s + c] = (sigma * np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)
    return out


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even.  Inputs are finite."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- #
# The benchmark configurations.  Each returns plain numpy buffers.             #
# --------------------------------------------------------------------------- #
def linear_layer(seed: int, T: int, n: int, m: int, x_bf16: bool, w_sigma: float = 0.02,
                 layer: int = 0):
    """Activations ~N(0,1) of shape [T, n] and full-precision weights ~N(0, w_sigma^2) [m, n]."""
    x = normal(seed, 0, T * n).reshape(T, n)
    W = normal(seed, 1 + layer, m * n, w_sigma).reshape(m, n)
    return (to_bf16_bits(x) if x_bf16 else x), W


def config_single_fc():
    """Single fully-connected layer 512 -> 512, k = 4, batch 64, fp32 activations, seed 0."""
    x, W = linear_layer(0, 64, 512, 512, x_bf16=False)
    return dict(x=x, W=W, k=4, T=64, n=512, m=512, per_tile=True)


MLP_DIMS = (1024, 2048, 2048, 10)
MLP_KS = (8, 8, 1)


def config_mlp(T: int = 4096, seed: int = 1):
    """3-layer MLP 1024 -> 2048 -> 2048 -> 10, k = 8 on the hidden layers, bf16 activations.
    The 20,480-weight classifier is below the paper's size threshold and stays untiled (k = 1)."""
    x = to_bf16_bits(normal(seed, 0, T * MLP_DIMS[0]).reshape(T, MLP_DIMS[0]))
    Ws = [normal(seed, 1 + l, MLP_DIMS[l + 1] * MLP_DIMS[l], 0.02).reshape(MLP_DIMS[l + 1], MLP_DIMS[l])
          for l in range(3)]
    return dict(x=x, Ws=Ws, ks=list(MLP_KS), dims=list(MLP_DIMS), T=T)


def conv_layer(seed: int, Nb: int, Cin: int, H: int, Wd: int, Cout: int, kh: int, kw: int,
               layer: int = 0, x_bf16: bool = True):
    """NCHW activations ~U(0,1) and Kaiming-normal (fan-in) weights (Cout,Cin,kh,kw)."""
    x = uniform(seed, 0, Nb * Cin * H * Wd).reshape(Nb, Cin, H, Wd)
    sigma = float(np.sqrt(2.0 / (Cin * kh * kw)))
    W = normal(seed, 1 + layer, Cout * Cin * kh * kw, sigma).reshape(Cout, Cin, kh, kw)
    return (to_bf16_bits(x) if x_bf16 else x), W


def config_large_linear(T: int, seed: int = 4, n: int = 8192, m: int = 8192):
    """Large linear sweep: in = out = 8192, bf16 activations ~N(0,1), W ~N(0, 0.02^2)."""
    x = to_bf16_bits(normal(seed, 0, T * n).reshape(T, n))
    W = normal(seed, 1, m * n, 0.02).reshape(m, n)
    return dict(x=x, W=W, T=T, n=n, m=m)
