"""kf_gemm_rowreduce_static: the row-reduction entry point for callers that cannot allocate.

Such callers (an inference runtime's enqueue hook, a process whose allocator already owns the
whole device, a serving loop that must not allocate after start-up) have no workspace to pass,
so the library keeps the per-tile partial statistics in a fixed array of its own.  The test
calls the entry point through the C ABI twice in a row -- the second time on a different,
smaller problem, so that whatever the first call left in the shared array would show up if it
were ever read -- and checks each result against kf_gemm_rowreduce with a caller-owned
workspace (bit for bit) and against the fp64 CPU oracle on the same seeded inputs.  This file sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest

import kf_inputs as ki
import oracle
import paper_2605_30359_b200 as kf
from gpu_util import assert_close, check_status, to_dev, to_f64


def _call_static(M, N, K, X, W, b, act, red, out, ldo, odt):
    import torch
    return kf.kf_gemm_rowreduce_static(M, N, K, kf.KF_BF16, X.data_ptr(), K, W.data_ptr(), K,
                                       b.data_ptr(), kf.ACT[act], kf.RED[red], out.data_ptr(), ldo,
                                       odt, torch.cuda.current_stream().cuda_stream)


@pytest.mark.gpu
def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    import torch
    kf.lib()
    cases = [("c3", 640, 2048, 256, "none", "softmax"),     # 5 x 8 tiles: 40 KB of partials
             ("c4", 384, 1024, 128, "sigmoid", "sum"),      # smaller: reuses the array's front
             ("c3", 200, 1000, 136, "none", "softmax")]     # ragged tiles over stale contents
    for (name, M, N, K, act, red) in cases:
        d = ki.gemm_inputs(name, seed=5, M=M, N=N, K=K)
        X, W, b = to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"])
        ref = kf.gemm_rowreduce(X, W, b, act, red)          # caller-owned workspace
        if red == "softmax":
            out = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
            st = _call_static(M, N, K, X, W, b, act, red, out, N, kf.KF_BF16)
        else:
            out = torch.zeros(M, dtype=torch.float32, device="cuda")
            st = _call_static(M, N, K, X, W, b, act, red, out, 1, kf.KF_F32)
        assert st == kf.KF_OK, kf.status_string(st)
        check_status()
        assert_close(to_f64(out), to_f64(ref), 2e-2, 2e-2, "%s %s static vs workspace" % (name, red))
        assert torch.equal(out, ref)                        # same kernels, same order: same bits
        # and against the definition itself: the fp64 oracle, with the gates the row reductions use
        want = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], act, red).reshape(to_f64(out).shape)
        assert_close(to_f64(out), want, 2e-2, 2e-2, "%s %s static vs oracle" % (name, red))
        if red == "softmax":
            assert_close(to_f64(out), want, 1e-7, 2e-2, "%s static vs oracle, relative" % name)
        else:
            assert_close(to_f64(out), want, 0.0, 1e-3, "%s static vs oracle, relative" % name)


def test_static_scratch_rejects_oversized_problems():
    """The size check comes before any CUDA call, so it needs no GPU and launches nothing."""
    kf.lib()
    before = kf.kf_launch_count()
    p = 0x10000
    # softmax partials for 16384 x 8192: 16384 rows * 32 tiles * 16 bytes (two float2 per tile) = 8 MiB > the 2 MiB array
    assert kf.kf_gemm_rowreduce_workspace_bytes(16384, 8192, 1024, kf.KF_BF16, 0) > kf.KF_STATIC_SCRATCH_BYTES
    st = kf.kf_gemm_rowreduce_static(16384, 8192, 1024, kf.KF_BF16, p, 1024, p, 1024, None, 0, 0,
                                     p + 4096, 8192, kf.KF_BF16, None)
    assert st == kf.KF_ERR_WORKSPACE
    # fp32 chains stage M*N floats: 1024 x 1024 x 4 = 4 MiB
    st = kf.kf_gemm_rowreduce_static(1024, 1024, 64, kf.KF_F32, p, 64, p, 64, None, 0, 1,
                                     p + 4096, 1, kf.KF_F32, None)
    assert st == kf.KF_ERR_WORKSPACE
    assert kf.kf_launch_count() == before
