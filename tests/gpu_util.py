"""Helpers for the GPU parity tests: numpy <-> device tensors and the elementwise comparison
against the fp64 oracle with a diagnostic that locates mismatches by position."""
import numpy as np

import kf_inputs as ki

F32_TOL = (1e-4, 1e-4)     # max |gpu-ref| <= atol + rtol*|ref| for fp32 chains
BF16_TOL = (2e-2, 2e-2)    # ... for bf16 chains


def to_dev(a):
    """numpy float32 / uint16-bf16-bits array -> CUDA tensor (float32 / bfloat16)."""
    import torch
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).cuda()
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def to_f64(t):
    """CUDA tensor -> float64 numpy (exact widening)."""
    return t.detach().float().cpu().numpy().astype(np.float64)


def tol_for(dtype):
    return F32_TOL if dtype == "f32" else BF16_TOL


def assert_close(got, ref, atol, rtol, what=""):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    err = np.abs(got - ref)
    lim = atol + rtol * np.abs(ref)
    bad = ~(err <= lim)          # also catches NaN
    if not bad.any():
        return float((err / lim).max()) if err.size else 0.0
    idx = np.argwhere(bad)
    lines = ["%s: %d of %d elements out of tolerance (atol %g rtol %g); worst err/limit %.3g"
             % (what, bad.sum(), bad.size, atol, rtol, float(np.nanmax(err / lim)))]
    for d in range(idx.shape[1]):
        u = np.unique(idx[:, d])
        lines.append("  dim %d: %d distinct indices, first %s last %s" % (d, len(u), u[:12].tolist(), u[-4:].tolist()))
    for i in idx[:8]:
        t = tuple(i.tolist())
        lines.append("  at %s got %.8g ref %.8g" % (t, got[t], ref[t]))
    raise AssertionError("\n".join(lines))


def check_status():
    import paper_2605_30359_b200 as kf
    st = kf.kf_device_status()
    assert st == kf.KF_OK, "device status: %s" % kf.status_string(st)
