"""fp64 CPU oracle for the fused operator chains -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Thin ctypes loader around ``kf_oracle.cpp`` (plain C++ loops, OpenMP over rows/images).
Only tests, the smoke check and the benchmark's cpu_baseline / reference arm may import
this package; the CUDA library and its Python binding never do.

Arrays are numpy: fp32 tensors as ``float32``, bf16 tensors as ``uint16`` bit patterns.
Outputs are ``float64`` and never rounded.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kf_oracle.cpp")
_LIB = os.path.join(_HERE, "libkf_oracle.so")

F32, BF16 = 0, 1
ACT = {"none": 0, "relu": 1, "gelu_tanh": 2, "sigmoid": 3, "gelu_erf": 4, "swish": 5,
       "tanh": 6, "hardtanh": 7, "chain95": 8, "leaky_relu": 9, "elu": 10, "mish": 11,
       "hardswish": 12, "softplus": 13, "relu6": 14, "hardsigmoid": 15}
RED = {"softmax": 0, "sum": 1, "max": 2, "mean": 3, "logsumexp": 4}


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (building the checker is not using it)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, vp, dbl, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_double, ctypes.c_int
        lib.oracle_act.restype = dbl
        lib.oracle_act.argtypes = [ci, dbl]
        lib.oracle_set_threads.argtypes = [ci]
        lib.oracle_get_threads.restype = ci
        lib.oracle_gemm_epilogue.restype = ci
        lib.oracle_gemm_epilogue.argtypes = [i64, i64, i64, ci, vp, i64, vp, i64, vp, ci, dbl,
                                             vp, i64, vp]
        lib.oracle_gemm_rowreduce.restype = ci
        lib.oracle_gemm_rowreduce.argtypes = [i64, i64, i64, ci, vp, i64, vp, i64, vp, ci, ci, vp]
        lib.oracle_conv3x3_gn.restype = ci
        lib.oracle_conv3x3_gn.argtypes = [i64, i64, i64, i64, i64, ci, vp, vp, vp, ci, ci, dbl,
                                          vp, vp, vp]
        lib.oracle_conv3x3_softmax_pool.restype = ci
        lib.oracle_conv3x3_softmax_pool.argtypes = [i64, i64, i64, i64, i64, ci, vp, vp, vp, i64, vp]
        lib.oracle_conv3x3_act_gap.restype = ci
        lib.oracle_conv3x3_act_gap.argtypes = [i64, i64, i64, i64, i64, ci, vp, vp, vp, ci, vp]
        lib.oracle_gemm_groupnorm.restype = ci
        lib.oracle_gemm_groupnorm.argtypes = [i64, i64, i64, ci, vp, i64, vp, i64, vp, i64, dbl, vp, vp, ci, vp]
        lib.oracle_conv3x3_act_pool.restype = ci
        lib.oracle_conv3x3_act_pool.argtypes = [i64, i64, i64, i64, i64, ci, vp, vp, vp, ci, ci, i64, vp]
        _lib = lib
    return _lib


def _dt(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("oracle takes float32 or uint16 (bf16 bits), got %s" % a.dtype)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dt=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if dt is not None and _dt(a) != dt:
        raise TypeError("mixed storage dtypes")
    return a


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def get_threads() -> int:
    return int(_load().oracle_get_threads())


def act(name: str, z: float) -> float:
    return float(_load().oracle_act(ACT[name], float(z)))


def gemm_epilogue(X, W, bias=None, act="none", scale=1.0, residual=None) -> np.ndarray:
    """Y = scale*act(X W^T + bias) + residual, fp64 [M,N]."""
    X = _c(X); dt = _dt(X); W = _c(W, dt); bias = _c(bias, dt); residual = _c(residual, dt)
    M, K = X.shape
    N, K2 = W.shape
    assert K == K2
    Y = np.empty((M, N), np.float64)
    rc = _load().oracle_gemm_epilogue(M, N, K, dt, _ptr(X), K, _ptr(W), K, _ptr(bias), ACT[act],
                                      float(scale), _ptr(residual), N, _ptr(Y))
    assert rc == 0
    return Y


def gemm_rowreduce(X, W, bias=None, pre_act="none", red="softmax") -> np.ndarray:
    """softmax: fp64 [M,N]; sum, max, mean, logsumexp: fp64 [M]."""
    X = _c(X); dt = _dt(X); W = _c(W, dt); bias = _c(bias, dt)
    M, K = X.shape
    N, K2 = W.shape
    assert K == K2
    out = np.empty((M, N) if red == "softmax" else (M,), np.float64)
    rc = _load().oracle_gemm_rowreduce(M, N, K, dt, _ptr(X), K, _ptr(W), K, _ptr(bias),
                                       ACT[pre_act], RED[red], _ptr(out))
    assert rc == 0
    return out


def conv3x3_gn(x, w, bias=None, act="none", groups=0, eps=1e-5, gamma=None, beta=None):
    """GroupNorm(act(conv3x3_pad1(x, w) + bias)), fp64 NCHW; groups=0 skips the norm."""
    x = _c(x); dt = _dt(x); w = _c(w, dt); bias = _c(bias, dt)
    gamma = _c(gamma, dt); beta = _c(beta, dt)
    Nb, Cin, H, Wd = x.shape
    Cout, Cin2, kh, kw = w.shape
    assert Cin == Cin2 and kh == 3 and kw == 3
    y = np.empty((Nb, Cout, H, Wd), np.float64)
    rc = _load().oracle_conv3x3_gn(Nb, Cin, H, Wd, Cout, dt, _ptr(x), _ptr(w), _ptr(bias),
                                   ACT[act], int(groups), float(eps), _ptr(gamma), _ptr(beta),
                                   _ptr(y))
    assert rc == 0
    return y


def conv3x3_softmax_pool(x, w, bias=None, pool=1):
    """max_pool(softmax over channels(conv3x3_pad1(x, w) + bias), pool), fp64 NCHW."""
    x = _c(x); dt = _dt(x); w = _c(w, dt); bias = _c(bias, dt)
    Nb, Cin, H, Wd = x.shape
    Cout = w.shape[0]
    y = np.empty((Nb, Cout, H // pool, Wd // pool), np.float64)
    rc = _load().oracle_conv3x3_softmax_pool(Nb, Cin, H, Wd, Cout, dt, _ptr(x), _ptr(w), _ptr(bias),
                                             int(pool), _ptr(y))
    assert rc == 0
    return y


def conv3x3_act_gap(x, w, bias=None, act="none"):
    """mean over H, W of act(conv3x3_pad1(x, w) + bias), fp64 [Nb, Cout]."""
    x = _c(x); dt = _dt(x); w = _c(w, dt); bias = _c(bias, dt)
    Nb, Cin, H, Wd = x.shape
    Cout = w.shape[0]
    y = np.empty((Nb, Cout), np.float64)
    rc = _load().oracle_conv3x3_act_gap(Nb, Cin, H, Wd, Cout, dt, _ptr(x), _ptr(w), _ptr(bias),
                                        ACT[act], _ptr(y))
    assert rc == 0
    return y


def gemm_groupnorm(X, W, bias=None, groups=1, eps=1e-5, gamma=None, beta=None, post_act="none"):
    """post_act(GroupNorm over column groups of (X W^T + bias)), fp64 [M,N]."""
    X = _c(X); dt = _dt(X); W = _c(W, dt); bias = _c(bias, dt)
    gamma = _c(gamma, dt); beta = _c(beta, dt)
    M, K = X.shape
    N = W.shape[0]
    Y = np.empty((M, N), np.float64)
    rc = _load().oracle_gemm_groupnorm(M, N, K, dt, _ptr(X), K, _ptr(W), K, _ptr(bias), int(groups),
                                       float(eps), _ptr(gamma), _ptr(beta), ACT[post_act], _ptr(Y))
    assert rc == 0
    return Y


POOL = {"max": 0, "avg": 1}


def conv3x3_act_pool(x, w, bias=None, act="none", kind="max", pool=2):
    """max / average pooling (kernel = stride = pool) of act(conv3x3_pad1(x, w) + bias), fp64 NCHW."""
    x = _c(x); dt = _dt(x); w = _c(w, dt); bias = _c(bias, dt)
    Nb, Cin, H, Wd = x.shape
    Cout = w.shape[0]
    y = np.empty((Nb, Cout, H // pool, Wd // pool), np.float64)
    rc = _load().oracle_conv3x3_act_pool(Nb, Cin, H, Wd, Cout, dt, _ptr(x), _ptr(w), _ptr(bias), ACT[act],
                                         POOL[kind], int(pool), _ptr(y))
    assert rc == 0
    return y
