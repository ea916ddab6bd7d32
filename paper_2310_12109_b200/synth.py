"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds NO arithmetic of the method: it only draws numbers.  A
counter-based generator (splitmix64 finaliser over ``seed, stream, counter``)
feeds Box-Muller in float64, so any element of any tensor can be regenerated
independently of how the tensor is chunked.  Values are scaled in float64 and
rounded once (round-to-nearest-even) to the storage type.

The tensors stand in for M2-BERT / M2-GPT activations and Hyena-style long
convolution filters: x ~ N(0,1); kernel k[h,t] = g[h,t] exp(-lambda t) / c with
g ~ N(0,1); Monarch weights ~ N(0, 1/fan_in).
"""
from __future__ import annotations

import numpy as np

SEED = 231012109

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    z = (z + np.uint64(0x9E3779B97F4A7C15)) & _M64
    z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
    z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
    return z ^ (z >> np.uint64(31))


def uniform01(stream: int, count: int, offset: int = 0, seed: int = SEED) -> np.ndarray:
    """`count` doubles in (0,1), element i depends only on (seed, stream, offset+i)."""
    with np.errstate(over="ignore"):
        base = _splitmix64(np.array([seed], dtype=np.uint64) ^ _splitmix64(np.array([stream], dtype=np.uint64)))
        ctr = np.arange(offset, offset + count, dtype=np.uint64)
        bits = _splitmix64(base + ctr * np.uint64(0xD1342543DE82EF95))
    return ((bits >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(stream: int, shape, seed: int = SEED) -> np.ndarray:
    """Standard normal float64 tensor (Box-Muller, two uniforms per value)."""
    count = int(np.prod(shape))
    u = uniform01(stream, 2 * count, 0, seed)
    r = np.sqrt(-2.0 * np.log(u[0::2]))
    return (r * np.cos(2.0 * np.pi * u[1::2])).reshape(shape)


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float64 -> bfloat16 (RNE) and return the values as float32."""
    f = np.asarray(a, dtype=np.float32)
    b = f.view(np.uint32).astype(np.uint64)
    rounded = (b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
    return rounded.astype(np.uint32).view(np.float32).reshape(f.shape)


def bf16_bits(a_f32: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    return (np.asarray(a_f32, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def stream_id(config: int, tensor: int) -> int:
    return config * 16 + tensor


def decay_kernel(config: int, H: int, n: int, lam: float, c: float) -> np.ndarray:
    """k[h,t] = g[h,t] exp(-lam t) / c as float32 (the library takes fp32 kernels)."""
    g = normal(stream_id(config, 1), (H, n))
    t = np.arange(n, dtype=np.float64)
    return (g * np.exp(-lam * t) / c).astype(np.float32)


# The five workloads -------------------------------------------------------------------

def config1():
    """Order-2 causal conv, fp32: B=1, H=4, n=256 -> N=512=32x16."""
    x = normal(stream_id(1, 0), (1, 4, 256)).astype(np.float32)
    k = decay_kernel(1, 4, 256, 0.01, 16.0)
    return dict(x=x, k=k, dims=(32, 16), causal=True)


def config2(B: int = 32, H: int = 768):
    """Bidirectional mixer: x[B,H,512] bf16, k[H,512] fp32, circular, N=512=32x16."""
    x = round_bf16(normal(stream_id(2, 0), (B, H, 512)))
    k = decay_kernel(2, H, 512, 0.005, float(np.sqrt(512.0)))
    return dict(x=x, k=k, dims=(32, 16), causal=False)


def config3(T: int = 16384, b: int = 64):
    """Order-2 Monarch matmul: X[T, b*b] bf16, L and R each b blocks of b x b ~ N(0,1/b)."""
    X = round_bf16(normal(stream_id(3, 0), (T, b * b)))
    L = round_bf16(normal(stream_id(3, 1), (b, b, b)) / np.sqrt(float(b)))
    R = round_bf16(normal(stream_id(3, 2), (b, b, b)) / np.sqrt(float(b)))
    return dict(X=X, L=L, R=R)


def config4(B: int = 4, H: int = 1024, n: int = 16384):
    """Long causal mixer: x[B,H,n] bf16, k[H,n] fp32, padded to 2n = 32^3 (order 3)."""
    x = round_bf16(normal(stream_id(4, 0), (B, H, n)))
    k = decay_kernel(4, H, n, 0.0005, 128.0)
    return dict(x=x, k=k, dims=(32, 32, 32), causal=True)


def config5(B: int = 32, T: int = 512, C: int = 768, nblk: int = 4, expand: int = 4):
    """M2 block: x[B,T,C] bf16, long kernel k[C,T], short conv w[C,3] ~ N(0,1/3),
    block-diagonal MLP weights ~ N(0, 1/fan_in) in bf16."""
    x = round_bf16(normal(stream_id(5, 0), (B, T, C)))
    k = decay_kernel(5, C, T, 0.005, float(np.sqrt(float(T))))
    w = (normal(stream_id(5, 2), (C, 3)) / np.sqrt(3.0)).astype(np.float32)
    ci, hi = C // nblk, expand * C // nblk
    W_up = round_bf16(normal(stream_id(5, 3), (nblk, hi, ci)) / np.sqrt(float(ci)))
    W_down = round_bf16(normal(stream_id(5, 4), (nblk, ci, hi)) / np.sqrt(float(hi)))
    return dict(x=x, k=k, w_short=w, W_up=W_up, W_down=W_down, dims=(32, 16))
