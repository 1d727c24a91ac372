"""Fused operator chains for NVIDIA B200 (sm_100a): Python binding of the C-ABI library.

The binding only marshals arguments: every step of every chain runs in the library's own
CUDA kernels.  PyTorch is used for device memory and streams.  There is no CPU fallback;
importing works without a GPU, calling does not.

Raw entry points (same names and argument order as include/kf.h, pointers as ints):
    kf_gemm_epilogue, kf_gemm_rowreduce, kf_conv3x3_epilogue, kf_*_workspace_bytes,
    kf_device_status, kf_launch_count, kf_status_string, kf_version
Tensor-level helpers:
    gemm_epilogue(X, W, bias, act, scale, residual) -> Y
    gemm_rowreduce(X, W, bias, pre_act, red, out_dtype) -> out
    conv3x3_epilogue(x, w, bias, act, groups, eps, gamma, beta) -> y
"""
from __future__ import annotations

import ctypes
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkf.so")

KF_OK, KF_ERR_INVALID_ARG, KF_ERR_UNSUPPORTED, KF_ERR_WORKSPACE, KF_ERR_CUDA, KF_ERR_TIMEOUT = range(6)
KF_F32, KF_BF16 = 0, 1
ACT = {"none": 0, "relu": 1, "gelu_tanh": 2, "sigmoid": 3, "gelu_erf": 4, "swish": 5, "tanh": 6,
       "hardtanh": 7, "chain95": 8, "leaky_relu": 9, "elu": 10, "mish": 11, "hardswish": 12,
       "softplus": 13, "relu6": 14, "hardsigmoid": 15}
RED = {"softmax": 0, "sum": 1, "max": 2, "mean": 3, "logsumexp": 4}

EXPORTS = ["kf_gemm_epilogue", "kf_gemm_rowreduce", "kf_gemm_rowreduce_static",
           "kf_conv3x3_epilogue", "kf_conv3x3_softmax_pool",
           "kf_conv3x3_softmax_pool_workspace_bytes", "kf_selftest_bounded_wait",
           "kf_conv3x3_act_gap", "kf_conv3x3_act_gap_workspace_bytes",
           "kf_conv3x3_act_pool", "kf_conv3x3_act_pool_workspace_bytes",
           "kf_gemm_groupnorm", "kf_gemm_groupnorm_workspace_bytes",
           "kf_gemm_epilogue_workspace_bytes", "kf_gemm_rowreduce_workspace_bytes",
           "kf_conv3x3_workspace_bytes", "kf_device_status", "kf_launch_count",
           "kf_reload_tuning", "kf_tensor_map_cache_stats", "kf_status_string", "kf_version",
           "kf_gemm_epilogue_host", "kf_gemm_epilogue_host_staging_bytes", "kf_launch_noop",
           "kf_gemm_epilogue_workspace_bytes_for", "kf_gemm_rowreduce_workspace_bytes_for",
           "kf_gemm_groupnorm_workspace_bytes_for"]


class KfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (kf_status %d)" % (where, status_string(status), status))


_lib = None


def lib() -> ctypes.CDLL:
    """Load libkf.so; raises if it has not been built (python -m paper_2605_30359_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2605_30359_b200.build` "
                          "(there is no fallback path)" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    i64, vp, ci, f32, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    L.kf_gemm_epilogue.restype = ci
    L.kf_gemm_epilogue.argtypes = [i64, i64, i64, ci, vp, i64, vp, i64, vp, ci, f32, vp, i64, vp,
                                   i64, vp, sz, vp]
    L.kf_gemm_rowreduce.restype = ci
    L.kf_gemm_rowreduce.argtypes = [i64, i64, i64, ci, vp, i64, vp, i64, vp, ci, ci, vp, i64, ci,
                                    vp, sz, vp]
    L.kf_gemm_rowreduce_static.restype = ci
    L.kf_gemm_rowreduce_static.argtypes = [i64, i64, i64, ci, vp, i64, vp, i64, vp, ci, ci, vp, i64,
                                           ci, vp]
    L.kf_conv3x3_epilogue.restype = ci
    L.kf_conv3x3_epilogue.argtypes = [i64, i64, i64, i64, i64, ci, vp, vp, vp, ci, ci, f32, vp, vp,
                                      vp, vp, sz, vp]
    L.kf_conv3x3_softmax_pool.restype = ci
    L.kf_conv3x3_softmax_pool.argtypes = [i64, i64, i64, i64, i64, ci, vp, vp, vp, ci, vp, vp, sz, vp]
    L.kf_conv3x3_softmax_pool_workspace_bytes.restype = sz
    L.kf_conv3x3_softmax_pool_workspace_bytes.argtypes = [i64, i64, i64, i64, i64, ci]
    L.kf_gemm_groupnorm.restype = ci
    L.kf_gemm_groupnorm.argtypes = [i64, i64, i64, ci, vp, i64, vp, i64, vp, ci, ctypes.c_float, vp, vp, ci,
                                    vp, i64, vp, sz, vp]
    L.kf_gemm_groupnorm_workspace_bytes.restype = sz
    L.kf_gemm_groupnorm_workspace_bytes.argtypes = [i64, i64, i64, ci, ci]
    L.kf_conv3x3_act_gap.restype = ci
    L.kf_conv3x3_act_gap.argtypes = [i64, i64, i64, i64, i64, ci, vp, vp, vp, ci, vp, vp, sz, vp]
    L.kf_conv3x3_act_gap_workspace_bytes.restype = sz
    L.kf_conv3x3_act_gap_workspace_bytes.argtypes = [i64, i64, i64, i64, i64, ci]
    L.kf_conv3x3_act_pool.restype = ci
    L.kf_conv3x3_act_pool.argtypes = [i64, i64, i64, i64, i64, ci, vp, vp, vp, ci, ci, ci, vp, vp, sz, vp]
    L.kf_conv3x3_act_pool_workspace_bytes.restype = sz
    L.kf_conv3x3_act_pool_workspace_bytes.argtypes = [i64, i64, i64, i64, i64, ci, ci]
    L.kf_selftest_bounded_wait.restype = ci
    L.kf_selftest_bounded_wait.argtypes = [ctypes.c_uint64, ctypes.POINTER(ctypes.c_uint64), vp]
    L.kf_gemm_epilogue_workspace_bytes.restype = sz
    L.kf_gemm_epilogue_workspace_bytes.argtypes = [i64, i64, i64, ci]
    L.kf_gemm_rowreduce_workspace_bytes.restype = sz
    L.kf_gemm_rowreduce_workspace_bytes.argtypes = [i64, i64, i64, ci, ci]
    L.kf_conv3x3_workspace_bytes.restype = sz
    L.kf_conv3x3_workspace_bytes.argtypes = [i64, i64, i64, i64, i64, ci, ci]
    L.kf_device_status.restype = ci
    L.kf_device_status.argtypes = []
    L.kf_launch_count.restype = i64
    L.kf_launch_count.argtypes = []
    L.kf_gemm_epilogue_host_staging_bytes.restype = sz
    L.kf_gemm_epilogue_host_staging_bytes.argtypes = [i64, i64, i64, ci, ci, ci]
    L.kf_gemm_epilogue_host.restype = ci
    L.kf_gemm_epilogue_host.argtypes = [i64, i64, i64, ci, vp, i64, vp, i64, vp, ci, f32, vp, i64, vp, i64,
                                        vp, sz, ci, vp]
    L.kf_gemm_epilogue_workspace_bytes_for.restype = sz
    L.kf_gemm_epilogue_workspace_bytes_for.argtypes = [i64, i64, i64, ci, vp, i64, vp, i64]
    L.kf_gemm_rowreduce_workspace_bytes_for.restype = sz
    L.kf_gemm_rowreduce_workspace_bytes_for.argtypes = [i64, i64, i64, ci, ci, vp, i64, vp, i64]
    L.kf_gemm_groupnorm_workspace_bytes_for.restype = sz
    L.kf_gemm_groupnorm_workspace_bytes_for.argtypes = [i64, i64, i64, ci, ci, vp, i64, vp, i64, vp, i64]
    L.kf_launch_noop.restype = ci
    L.kf_launch_noop.argtypes = [vp]
    L.kf_reload_tuning.restype = None
    L.kf_reload_tuning.argtypes = []
    L.kf_tensor_map_cache_stats.restype = None
    L.kf_tensor_map_cache_stats.argtypes = [ctypes.POINTER(i64), ctypes.POINTER(i64)]
    L.kf_status_string.restype = ctypes.c_char_p
    L.kf_status_string.argtypes = [ci]
    L.kf_version.restype = ci
    L.kf_version.argtypes = []
    _lib = L
    return L


# ------------------------------------------------------------------ raw entry points
def kf_gemm_epilogue(M, N, K, io_dtype, X, ldx, W, ldw, bias, act, scale, residual, ldr, Y, ldy,
                     workspace, workspace_bytes, stream) -> int:
    return lib().kf_gemm_epilogue(M, N, K, io_dtype, X, ldx, W, ldw, bias, act, scale, residual,
                                  ldr, Y, ldy, workspace, workspace_bytes, stream)


def kf_gemm_rowreduce(M, N, K, in_dtype, X, ldx, W, ldw, bias, pre_act, red, out, ldo, out_dtype,
                      workspace, workspace_bytes, stream) -> int:
    return lib().kf_gemm_rowreduce(M, N, K, in_dtype, X, ldx, W, ldw, bias, pre_act, red, out, ldo,
                                   out_dtype, workspace, workspace_bytes, stream)


KF_STATIC_SCRATCH_BYTES = 2 << 20


def kf_gemm_rowreduce_static(M, N, K, in_dtype, X, ldx, W, ldw, bias, pre_act, red, out, ldo,
                             out_dtype, stream) -> int:
    """kf_gemm_rowreduce for callers that cannot allocate: no workspace argument, the partial
    statistics go to a fixed array inside the library (at most KF_STATIC_SCRATCH_BYTES)."""
    return lib().kf_gemm_rowreduce_static(M, N, K, in_dtype, X, ldx, W, ldw, bias, pre_act, red,
                                          out, ldo, out_dtype, stream)


def kf_conv3x3_epilogue(Nb, Cin, H, Wd, Cout, io_dtype, x, w, bias, act, groups, eps, gamma, beta,
                        y, workspace, workspace_bytes, stream) -> int:
    return lib().kf_conv3x3_epilogue(Nb, Cin, H, Wd, Cout, io_dtype, x, w, bias, act, groups, eps,
                                     gamma, beta, y, workspace, workspace_bytes, stream)


def kf_conv3x3_softmax_pool(Nb, Cin, H, Wd, Cout, io_dtype, x, w, bias, pool, y, workspace,
                            workspace_bytes, stream) -> int:
    return lib().kf_conv3x3_softmax_pool(Nb, Cin, H, Wd, Cout, io_dtype, x, w, bias, pool, y,
                                         workspace, workspace_bytes, stream)


def kf_conv3x3_softmax_pool_workspace_bytes(Nb, Cin, H, Wd, Cout, io_dtype) -> int:
    return lib().kf_conv3x3_softmax_pool_workspace_bytes(Nb, Cin, H, Wd, Cout, io_dtype)


def kf_gemm_groupnorm(M, N, K, io_dtype, X, ldx, W, ldw, bias, groups, eps, gamma, beta, post_act, Y, ldy,
                      workspace, workspace_bytes, stream) -> int:
    return lib().kf_gemm_groupnorm(M, N, K, io_dtype, X, ldx, W, ldw, bias, groups, eps, gamma, beta,
                                   post_act, Y, ldy, workspace, workspace_bytes, stream)


def kf_gemm_groupnorm_workspace_bytes(M, N, K, io_dtype, groups) -> int:
    return lib().kf_gemm_groupnorm_workspace_bytes(M, N, K, io_dtype, groups)


def kf_conv3x3_act_gap(Nb, Cin, H, Wd, Cout, io_dtype, x, w, bias, act, out, workspace,
                       workspace_bytes, stream) -> int:
    return lib().kf_conv3x3_act_gap(Nb, Cin, H, Wd, Cout, io_dtype, x, w, bias, act, out, workspace,
                                    workspace_bytes, stream)


def kf_conv3x3_act_gap_workspace_bytes(Nb, Cin, H, Wd, Cout, io_dtype) -> int:
    return lib().kf_conv3x3_act_gap_workspace_bytes(Nb, Cin, H, Wd, Cout, io_dtype)


def kf_conv3x3_act_pool(Nb, Cin, H, Wd, Cout, io_dtype, x, w, bias, act, pool_kind, pool, y,
                        workspace, workspace_bytes, stream) -> int:
    return lib().kf_conv3x3_act_pool(Nb, Cin, H, Wd, Cout, io_dtype, x, w, bias, act, pool_kind,
                                     pool, y, workspace, workspace_bytes, stream)


def kf_conv3x3_act_pool_workspace_bytes(Nb, Cin, H, Wd, Cout, io_dtype, pool) -> int:
    return lib().kf_conv3x3_act_pool_workspace_bytes(Nb, Cin, H, Wd, Cout, io_dtype, pool)


def kf_selftest_bounded_wait(limit_ns, stream=None):
    """Returns (status, nanoseconds waited)."""
    waited = ctypes.c_uint64(0)
    st = lib().kf_selftest_bounded_wait(int(limit_ns), ctypes.byref(waited), stream)
    return st, int(waited.value)


def kf_gemm_epilogue_workspace_bytes(M, N, K, io_dtype) -> int:
    return lib().kf_gemm_epilogue_workspace_bytes(M, N, K, io_dtype)


def kf_gemm_rowreduce_workspace_bytes(M, N, K, in_dtype, red) -> int:
    return lib().kf_gemm_rowreduce_workspace_bytes(M, N, K, in_dtype, red)


def kf_conv3x3_workspace_bytes(Nb, Cin, H, Wd, Cout, io_dtype, groups) -> int:
    return lib().kf_conv3x3_workspace_bytes(Nb, Cin, H, Wd, Cout, io_dtype, groups)


def kf_device_status() -> int:
    return lib().kf_device_status()


def kf_launch_count() -> int:
    return lib().kf_launch_count()


def kf_reload_tuning() -> None:
    """Re-read the KF_* dispatch switches from the environment (they are read once otherwise)."""
    lib().kf_reload_tuning()


def kf_tensor_map_cache_stats():
    """(hits, misses) of the encoded-tensor-map cache since load."""
    h, m = ctypes.c_int64(0), ctypes.c_int64(0)
    lib().kf_tensor_map_cache_stats(ctypes.byref(h), ctypes.byref(m))
    return int(h.value), int(m.value)


def status_string(status: int) -> str:
    return lib().kf_status_string(status).decode()


def kf_version() -> int:
    return lib().kf_version()


# ------------------------------------------------------------------ tensor-level helpers
def _torch():
    import torch
    return torch


def _kf_dtype(t) -> int:
    torch = _torch()
    if t.dtype == torch.float32:
        return KF_F32
    if t.dtype == torch.bfloat16:
        return KF_BF16
    raise TypeError("kf chains take float32 or bfloat16 tensors, got %s" % t.dtype)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _check_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise ValueError("kf chains run on CUDA tensors only (no CPU fallback)")


_workspaces = {}


def workspace(nbytes: int, device, slot: str = "ws"):
    """A cached, 256-byte aligned device scratch buffer of at least nbytes (None for 0); buffers
    of different `slot` names are distinct."""
    if nbytes == 0:
        return None
    torch = _torch()
    key = (device.type, device.index, slot)
    buf = _workspaces.get(key)
    if buf is None or buf.numel() < nbytes:
        buf = torch.empty(max(nbytes, 1 << 20), dtype=torch.uint8, device=device)
        _workspaces[key] = buf
    return buf


def _stream_ptr(stream):
    torch = _torch()
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def gemm_epilogue(X, W, bias=None, act="none", scale=1.0, residual=None, out=None, stream=None):
    """Y = scale*act(X @ W.T + bias) + residual in one kernel.  X [M,K], W [N,K], row-major."""
    torch = _torch()
    _check_cuda(X, W, bias, residual, out)
    M, K = X.shape
    N = W.shape[0]
    dt = _kf_dtype(X)
    if out is None:
        out = torch.empty((M, N), dtype=X.dtype, device=X.device)
    nb = lib().kf_gemm_epilogue_workspace_bytes_for(M, N, K, dt, _ptr(X), X.stride(0), _ptr(W), W.stride(0))
    ws = workspace(nb, X.device)
    st = kf_gemm_epilogue(M, N, K, dt, _ptr(X), X.stride(0), _ptr(W), W.stride(0), _ptr(bias),
                          ACT[act], float(scale), _ptr(residual),
                          residual.stride(0) if residual is not None else 0, _ptr(out),
                          out.stride(0), _ptr(ws), nb, _stream_ptr(stream))
    if st != KF_OK:
        raise KfError(st, "kf_gemm_epilogue")
    return out


def gemm_rowreduce(X, W, bias=None, pre_act="none", red="softmax", out_dtype=None, out=None,
                   stream=None):
    """softmax: out[M,N] = softmax_n(pre_act(X @ W.T + bias)); sum / max / mean / logsumexp:
    out[M] fp32 = that reduction of every row."""
    torch = _torch()
    _check_cuda(X, W, bias, out)
    M, K = X.shape
    N = W.shape[0]
    dt = _kf_dtype(X)
    if red != "softmax":
        if out is None:
            out = torch.empty((M,), dtype=torch.float32, device=X.device)
        odt, ldo = KF_F32, 1
    else:
        if out is None:
            out = torch.empty((M, N), dtype=out_dtype or X.dtype, device=X.device)
        odt, ldo = _kf_dtype(out), out.stride(0)
    nb = lib().kf_gemm_rowreduce_workspace_bytes_for(M, N, K, dt, RED[red], _ptr(X), X.stride(0), _ptr(W),
                                                     W.stride(0))
    ws = workspace(nb, X.device)
    st = kf_gemm_rowreduce(M, N, K, dt, _ptr(X), X.stride(0), _ptr(W), W.stride(0), _ptr(bias),
                           ACT[pre_act], RED[red], _ptr(out), ldo, odt, _ptr(ws), nb,
                           _stream_ptr(stream))
    if st != KF_OK:
        raise KfError(st, "kf_gemm_rowreduce")
    return out


def conv3x3_epilogue(x, w, bias=None, act="none", groups=0, eps=1e-5, gamma=None, beta=None,
                     out=None, stream=None):
    """y = GroupNorm(act(conv3x3_pad1(x, w) + bias)); x NCHW, w OIHW, contiguous."""
    torch = _torch()
    _check_cuda(x, w, bias, gamma, beta, out)
    if not (x.is_contiguous() and w.is_contiguous()):
        raise ValueError("conv3x3_epilogue takes contiguous NCHW / OIHW tensors")
    Nb, Cin, H, Wd = x.shape
    Cout = w.shape[0]
    dt = _kf_dtype(x)
    if out is None:
        out = torch.empty((Nb, Cout, H, Wd), dtype=x.dtype, device=x.device)
    nb = kf_conv3x3_workspace_bytes(Nb, Cin, H, Wd, Cout, dt, groups)
    ws = workspace(nb, x.device)
    st = kf_conv3x3_epilogue(Nb, Cin, H, Wd, Cout, dt, _ptr(x), _ptr(w), _ptr(bias), ACT[act],
                             int(groups), float(eps), _ptr(gamma), _ptr(beta), _ptr(out), _ptr(ws),
                             nb, _stream_ptr(stream))
    if st != KF_OK:
        raise KfError(st, "kf_conv3x3_epilogue")
    return out


def conv3x3_softmax_pool(x, w, bias=None, pool=1, out=None, stream=None):
    """y = max_pool(softmax over channels(conv3x3_pad1(x, w) + bias), pool); NCHW / OIHW."""
    torch = _torch()
    _check_cuda(x, w, bias, out)
    if not (x.is_contiguous() and w.is_contiguous()):
        raise ValueError("conv3x3_softmax_pool takes contiguous NCHW / OIHW tensors")
    Nb, Cin, H, Wd = x.shape
    Cout = w.shape[0]
    dt = _kf_dtype(x)
    if out is None:
        div = max(int(pool), 1)        # a bad pool is rejected by the library, not here
        out = torch.empty((Nb, Cout, H // div, Wd // div), dtype=x.dtype, device=x.device)
    nb = kf_conv3x3_softmax_pool_workspace_bytes(Nb, Cin, H, Wd, Cout, dt)
    ws = workspace(nb, x.device)
    st = kf_conv3x3_softmax_pool(Nb, Cin, H, Wd, Cout, dt, _ptr(x), _ptr(w), _ptr(bias), int(pool),
                                 _ptr(out), _ptr(ws), nb, _stream_ptr(stream))
    if st != KF_OK:
        raise KfError(st, "kf_conv3x3_softmax_pool")
    return out


def gemm_groupnorm(X, W, bias=None, groups=1, eps=1e-5, gamma=None, beta=None, post_act="none", out=None,
                   stream=None):
    """Y = post_act(GroupNorm over groups of N/groups consecutive columns of (X @ W.T + bias))."""
    torch = _torch()
    _check_cuda(X, W, bias, gamma, beta, out)
    M, K = X.shape
    N = W.shape[0]
    dt = _kf_dtype(X)
    if out is None:
        out = torch.empty((M, N), dtype=X.dtype, device=X.device)
    nb = lib().kf_gemm_groupnorm_workspace_bytes_for(M, N, K, dt, int(groups), _ptr(X), X.stride(0), _ptr(W),
                                                     W.stride(0), _ptr(out), out.stride(0))
    ws = workspace(nb, X.device)
    st = kf_gemm_groupnorm(M, N, K, dt, _ptr(X), X.stride(0), _ptr(W), W.stride(0), _ptr(bias), int(groups),
                           float(eps), _ptr(gamma), _ptr(beta), ACT[post_act], _ptr(out), out.stride(0),
                           _ptr(ws), nb, _stream_ptr(stream))
    if st != KF_OK:
        raise KfError(st, "kf_gemm_groupnorm")
    return out


def conv3x3_act_gap(x, w, bias=None, act="none", out=None, stream=None):
    """out[Nb, Cout] fp32 = mean over H, W of act(conv3x3_pad1(x, w) + bias); NCHW / OIHW."""
    torch = _torch()
    _check_cuda(x, w, bias, out)
    if not (x.is_contiguous() and w.is_contiguous()):
        raise ValueError("conv3x3_act_gap takes contiguous NCHW / OIHW tensors")
    Nb, Cin, H, Wd = x.shape
    Cout = w.shape[0]
    dt = _kf_dtype(x)
    if out is None:
        out = torch.empty((Nb, Cout), dtype=torch.float32, device=x.device)
    nb = kf_conv3x3_act_gap_workspace_bytes(Nb, Cin, H, Wd, Cout, dt)
    ws = workspace(nb, x.device)
    st = kf_conv3x3_act_gap(Nb, Cin, H, Wd, Cout, dt, _ptr(x), _ptr(w), _ptr(bias), ACT[act],
                            _ptr(out), _ptr(ws), nb, _stream_ptr(stream))
    if st != KF_OK:
        raise KfError(st, "kf_conv3x3_act_gap")
    return out


POOL = {"max": 0, "avg": 1}


def conv3x3_act_pool(x, w, bias=None, act="none", kind="max", pool=2, out=None, stream=None):
    """out[Nb, Cout, H//pool, W//pool] = max / average pooling of act(conv3x3_pad1(x, w) + bias)."""
    torch = _torch()
    _check_cuda(x, w, bias, out)
    if not (x.is_contiguous() and w.is_contiguous()):
        raise ValueError("conv3x3_act_pool takes contiguous NCHW / OIHW tensors")
    Nb, Cin, H, Wd = x.shape
    Cout = w.shape[0]
    dt = _kf_dtype(x)
    if out is None:
        out = torch.empty((Nb, Cout, H // max(pool, 1), Wd // max(pool, 1)), dtype=x.dtype, device=x.device)
    nb = kf_conv3x3_act_pool_workspace_bytes(Nb, Cin, H, Wd, Cout, dt, pool)
    ws = workspace(nb, x.device)
    st = kf_conv3x3_act_pool(Nb, Cin, H, Wd, Cout, dt, _ptr(x), _ptr(w), _ptr(bias), ACT[act],
                             POOL[kind], pool, _ptr(out), _ptr(ws), nb, _stream_ptr(stream))
    if st != KF_OK:
        raise KfError(st, "kf_conv3x3_act_pool")
    return out


# ------------------------------------------------------------------ host-buffer front end
def kf_launch_noop(stream=None):
    st = lib().kf_launch_noop(_stream_ptr(stream))
    if st != KF_OK:
        raise KfError(st, "kf_launch_noop")


def gemm_epilogue_host(X, W, bias=None, act="none", scale=1.0, residual=None, out_host=None,
                       device=None, stream=None, chunks=4):
    """gemm_epilogue for HOST tensors (pinned memory recommended): marshals the arguments of
    kf_gemm_epilogue_host, which pipelines uploads, kernels and downloads over `chunks` row
    blocks.  The work is enqueued on `stream` (default: the current stream); synchronise it
    before reading out_host.  The device staging buffer is the binding's cached workspace."""
    torch = _torch()
    device = device or torch.device("cuda", torch.cuda.current_device())
    for t in (X, W, bias, residual, out_host):
        if t is not None and t.is_cuda:
            raise ValueError("gemm_epilogue_host takes host tensors")
    M, K = X.shape
    N = W.shape[0]
    dt = _kf_dtype(X)
    if out_host is None:
        out_host = torch.empty((M, N), dtype=X.dtype).pin_memory()
    nb = lib().kf_gemm_epilogue_host_staging_bytes(M, N, K, dt, int(bias is not None), int(residual is not None))
    ws = workspace(nb, device, slot="host_staging")
    with torch.cuda.device(device):
        st = lib().kf_gemm_epilogue_host(M, N, K, dt, X.data_ptr(), X.stride(0), W.data_ptr(), W.stride(0),
                                         bias.data_ptr() if bias is not None else None, ACT[act], float(scale),
                                         residual.data_ptr() if residual is not None else None,
                                         residual.stride(0) if residual is not None else 0,
                                         out_host.data_ptr(), out_host.stride(0), _ptr(ws), nb, int(chunks),
                                         _stream_ptr(stream))
    if st != KF_OK:
        raise KfError(st, "kf_gemm_epilogue_host")
    return out_host
