"""Seeded synthetic inputs for the SBP linear-layer path.

This module only manufactures input tensors (Gaussian activations, weights and
output gradients with the shapes and scales of ViT / ConvNeXt layers); it holds
none of the method's arithmetic and loads no native library.  Both the CUDA
tests / benchmark and the CPU oracle checks draw their inputs from here so the
two sides see bit-identical values.

Recipe: a splitmix64 counter stream per tensor -> Box-Muller in fp64 -> scale
-> round-to-nearest-even to the path's storage type (fp32, or bf16 kept as its
16-bit pattern in a uint16 array).
"""
from __future__ import annotations

import numpy as np

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_MIX1 = np.uint64(0xBF58476D1CE4E5B9)
_MIX2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _splitmix64(counters: np.ndarray) -> np.ndarray:
    """splitmix64 output for the given 64-bit states (vectorised, wraps mod 2^64)."""
    with np.errstate(over="ignore"):
        z = counters.copy()
        z ^= z >> np.uint64(30)
        z *= _MIX1
        z ^= z >> np.uint64(27)
        z *= _MIX2
        z ^= z >> np.uint64(31)
    return z


def tensor_seed(data_seed: int, tensor_id: int) -> int:
    """Independent stream seed for tensor ``tensor_id`` of data set ``data_seed``."""
    s = np.array([(data_seed * 0x100000001B3 + tensor_id * 0x9E3779B97F4A7C15 + 0x1234567)
                  & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    return int(_splitmix64(s)[0])


def gaussian_f64(n: int, seed: int, sigma: float = 1.0) -> np.ndarray:
    """``n`` draws of N(0, sigma^2) in fp64, a pure function of (seed, n-prefix)."""
    out = np.empty(n, dtype=np.float64)
    pairs_total = (n + 1) // 2
    done = 0
    with np.errstate(over="ignore"):
        base = np.uint64(seed & 0xFFFFFFFFFFFFFFFF)
        while done < pairs_total:
            cnt = min(_CHUNK, pairs_total - done)
            idx = np.arange(done, done + cnt, dtype=np.uint64)
            s1 = base + (np.uint64(2) * idx + np.uint64(1)) * _GAMMA
            s2 = base + (np.uint64(2) * idx + np.uint64(2)) * _GAMMA
            z1 = _splitmix64(s1)
            z2 = _splitmix64(s2)
            u1 = ((z1 >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
            u2 = (z2 >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
            rad = np.sqrt(-2.0 * np.log(u1)) * sigma
            ang = (2.0 * np.pi) * u2
            lo = 2 * done
            hi = min(n, 2 * (done + cnt))
            blk = np.empty(2 * cnt, dtype=np.float64)
            blk[0::2] = rad * np.cos(ang)
            blk[1::2] = rad * np.sin(ang)
            out[lo:hi] = blk[: hi - lo]
            done += cnt
    return out


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp64 -> fp32 -> bf16 (both round-to-nearest-even); returns uint16 bit patterns."""
    f32 = np.asarray(x, dtype=np.float32)
    bits = f32.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = bits + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp64."""
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def gaussian_tensor(shape, dtype: str, data_seed: int, tensor_id: int, sigma: float) -> np.ndarray:
    """Gaussian tensor in the path's storage type: ``"f32"`` -> float32, ``"bf16"`` -> uint16 bits."""
    n = int(np.prod(shape))
    g = gaussian_f64(n, tensor_seed(data_seed, tensor_id), sigma)
    if dtype == "f32":
        return g.astype(np.float32).reshape(shape)
    if dtype == "bf16":
        return f64_to_bf16_bits(g).reshape(shape)
    raise ValueError(dtype)


def to_f64(a: np.ndarray, dtype: str) -> np.ndarray:
    """Exact fp64 view of a stored tensor (what the oracle consumes)."""
    return a.astype(np.float64) if dtype == "f32" else bf16_bits_to_f64(a)


def layer_inputs(dtype: str, M: int, C_in: int, C_out: int, data_seed: int,
                 sigma_x: float = 1.0, sigma_w: float = 0.02, sigma_dy: float = 1e-2):
    """(X [M,C_in], W [C_in,C_out], dY [M,C_out]) for one linear layer."""
    X = gaussian_tensor((M, C_in), dtype, data_seed, 0, sigma_x)
    W = gaussian_tensor((C_in, C_out), dtype, data_seed, 1, sigma_w)
    dY = gaussian_tensor((M, C_out), dtype, data_seed, 2, sigma_dy)
    return X, W, dY


# Named workloads: (dtype, B, H, W, C_in, C_out, keep_ratio, mask mode, sigmas) ------------
def workload(name: str) -> dict:
    """Shapes of the benchmark / parity workloads.

    ``single_fp32``     tiny fp32 layer, B=2, N=16, 32->64, r=0.5 random
    ``vit_b16_fc1``     ViT-B/16 MLP fc1, bf16, B=64, 14x14 tokens, 768->3072, r=0.5 random
    """
    if name == "single_fp32":
        return dict(dtype="f32", B=2, H=16, W=1, C_in=32, C_out=64, keep_ratio=0.5, mode=0,
                    sigma_x=1.0, sigma_w=32 ** -0.5, sigma_dy=1.0, data_seed=1001)
    if name == "vit_b16_fc1":
        return dict(dtype="bf16", B=64, H=14, W=14, C_in=768, C_out=3072, keep_ratio=0.5, mode=0,
                    sigma_x=1.0, sigma_w=0.02, sigma_dy=1e-2, data_seed=1002)
    raise KeyError(name)
