"""Seeded synthetic inputs for the five fused-chain workloads.

This module serves the CPU oracle's tests and the CUDA path's tests/bench alike and
holds none of the chains' arithmetic: a counter-based generator (splitmix64 finaliser of
(seed, tensor id, element index)), uniform and Box-Muller normal draws, round-to-nearest-
even conversion to bf16 storage, and the shape/distribution table of the workloads.

Arrays are numpy: fp32 tensors as float32, bf16 tensors as uint16 bit patterns.
"""
from __future__ import annotations

import math
import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_CHUNK = 1 << 22


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function on uint64 arrays (wrapping arithmetic)."""
    z = (z + np.uint64(0x9E3779B97F4A7C15)) & _M64
    z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
    z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
    return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor_id: int) -> np.uint64:
    k = _mix(np.array([(seed * 0x632BE59BD9B4E019 + tensor_id * 0xD1342543DE82EF95 + 1)
                       & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))
    return k[0]


def _u01(key: np.uint64, idx: np.ndarray) -> np.ndarray:
    """Uniform in [0,1) with 53 bits, addressable by element index."""
    with np.errstate(over="ignore"):
        bits = _mix(key ^ _mix(idx))
    return (bits >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def _element_indices(shape, first):
    """Flat element indices (uint64) of the slices `first` along axis 0 of a tensor of `shape`."""
    inner = int(np.prod(shape[1:])) if len(shape) > 1 else 1
    first = np.asarray(first, dtype=np.uint64).reshape(-1, 1)
    return (first * np.uint64(inner) + np.arange(inner, dtype=np.uint64).reshape(1, -1)).reshape(-1)


def uniform(seed: int, tensor_id: int, shape, lo: float, hi: float, first=None) -> np.ndarray:
    """float64 array of U(lo, hi) draws; element i depends only on (seed, tensor_id, i).

    ``first`` (indices along axis 0) draws only those slices of the tensor of ``shape``: the
    values are the ones the full tensor holds there, without generating the rest."""
    key = _key(seed, tensor_id)
    if first is not None:
        u = _u01(key, _element_indices(shape, first))
        return (lo + (hi - lo) * u).reshape((len(first),) + tuple(shape[1:]))
    n = int(np.prod(shape))
    out = np.empty(n, np.float64)
    for s in range(0, n, _CHUNK):
        e = min(n, s + _CHUNK)
        u = _u01(key, np.arange(s, e, dtype=np.uint64))
        out[s:e] = lo + (hi - lo) * u
    return out.reshape(shape)


def normal(seed: int, tensor_id: int, shape, first=None) -> np.ndarray:
    """float64 array of N(0,1) draws (Box-Muller on two indexed uniforms per element).

    ``first``: as in uniform()."""
    key = _key(seed, tensor_id)
    if first is not None:
        i = _element_indices(shape, first)
        u1 = 1.0 - _u01(key, i * np.uint64(2))
        u2 = _u01(key, i * np.uint64(2) + np.uint64(1))
        return (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)).reshape(
            (len(first),) + tuple(shape[1:]))
    n = int(np.prod(shape))
    out = np.empty(n, np.float64)
    for s in range(0, n, _CHUNK):
        e = min(n, s + _CHUNK)
        i = np.arange(s, e, dtype=np.uint64)
        u1 = 1.0 - _u01(key, i * np.uint64(2))            # (0, 1]
        u2 = _u01(key, i * np.uint64(2) + np.uint64(1))
        out[s:e] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return out.reshape(shape)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float values to bf16 storage (round to nearest, ties to even); uint16 bits."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def store(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float64 draw to its storage dtype: 'f32' -> float32, 'bf16' -> uint16 bits."""
    if dtype == "f32":
        return np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "bf16":
        return to_bf16_bits(a)
    raise ValueError(dtype)


def widen(a: np.ndarray) -> np.ndarray:
    """Stored tensor -> float64 values."""
    if a.dtype == np.uint16:
        return bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


# ----------------------------------------------------------------------------------------
# Workload table.  Shapes and distributions are the five benchmark configurations:
# activations ~N(0,1); weights and biases ~U(+-1/sqrt(fan_in)) (the torch default for
# Linear/Conv parameters); residual ~N(0,1).  Tensor ids are fixed per role.
# ----------------------------------------------------------------------------------------
_X, _W, _B, _R = 1, 2, 3, 4

GEMM_CONFIGS = {
    # name: (dtype, M, N, K)
    "c1": ("f32", 128, 256, 512),
    "c2": ("bf16", 8192, 4096, 4096),
    "c3": ("bf16", 4096, 8192, 2048),
    "c4": ("bf16", 16384, 1024, 1024),
}
CONV_CONFIG = {"c5": ("bf16", 128, 64, 64, 64, 128, 32)}  # dtype, Nb, Cin, H, W, Cout, groups


def gemm_inputs(name: str, seed: int = 0, M=None, N=None, K=None, dtype=None, rows=None):
    """Inputs of a GEMM-chain workload; M/N/K/dtype override the table for reduced cases.

    ``rows`` (an index array) returns only those rows of X and R: every chain here is
    row-wise independent, so a row subset is a valid smaller problem with the same W, b.
    Note the element index of a draw is its index in the FULL tensor, so a row subset
    holds exactly the values the full tensor has there.
    """
    dt, M0, N0, K0 = GEMM_CONFIGS[name]
    dt = dtype or dt
    M, N, K = M or M0, N or N0, K or K0
    bound = 1.0 / math.sqrt(K)
    d = {"M": M, "N": N, "K": K, "dtype": dt, "seed": seed, "name": name}
    d["W"] = store(uniform(seed, _W, (N, K), -bound, bound), dt)
    d["b"] = store(uniform(seed, _B, (N,), -bound, bound), dt)
    if rows is not None:
        rows = np.asarray(rows)
        Xf = normal(seed, _X, (M, K), first=rows)
        Rf = normal(seed, _R, (M, N), first=rows) if name == "c2" else None
        d["M"] = len(rows)
    else:
        Xf = normal(seed, _X, (M, K))
        Rf = normal(seed, _R, (M, N)) if name == "c2" else None
    d["X"] = store(Xf, dt)
    d["R"] = store(Rf, dt) if Rf is not None else None
    return d


def conv_inputs(name: str = "c5", seed: int = 0, Nb=None, Cin=None, H=None, W=None, Cout=None,
                groups=None, dtype=None, images=None):
    """Inputs of the convolution workload.  ``images`` (an index array) returns only those
    images of x, holding exactly the values the full batch has there (images are independent)."""
    dt, Nb0, Cin0, H0, W0, Cout0, g0 = CONV_CONFIG[name]
    dt = dtype or dt
    Nb, Cin, H, W, Cout = Nb or Nb0, Cin or Cin0, H or H0, W or W0, Cout or Cout0
    groups = g0 if groups is None else groups
    bound = 1.0 / math.sqrt(Cin * 9)
    return {
        "Nb": Nb, "Cin": Cin, "H": H, "W": W, "Cout": Cout, "groups": groups, "eps": 1e-5,
        "dtype": dt, "seed": seed, "name": name,
        "x": store(normal(seed, _X, (Nb, Cin, H, W), first=images), dt),
        "w": store(uniform(seed, _W, (Cout, Cin, 3, 3), -bound, bound), dt),
        "bias": store(uniform(seed, _B, (Cout,), -bound, bound), dt),
    }
