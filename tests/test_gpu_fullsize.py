"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The fp64 oracle cannot recompute 137 G multiply-adds per test, but every chain here is
independent per row (per image for the convolution), so the oracle recomputes sampled rows /
images exactly -- first and last rows, both sides of tile boundaries, random interior rows --
and whole-output properties cover the rest."""
import numpy as np
import pytest

import kf_inputs as ki
import oracle
from gpu_util import assert_close, check_status, to_dev, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kf():
    import paper_2605_30359_b200 as kf
    kf.lib()
    return kf


def sample_rows(M, n_random, seed):
    fixed = [0, 1, 127, 128, 129, 255, 256, M // 2 - 1, M // 2, M - 129, M - 128, M - 2, M - 1]
    r = np.random.default_rng(seed).integers(0, M, size=n_random).tolist()
    return np.array(sorted(set(fixed + r)))


def test_c2_full_size_sampled_rows(kf):
    d = ki.gemm_inputs("c2", seed=0)
    Y = kf.gemm_epilogue(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "gelu_tanh", 0.5, to_dev(d["R"]))
    check_status()
    rows = sample_rows(d["M"], 32, 2)
    ref = oracle.gemm_epilogue(d["X"][rows], d["W"], d["b"], "gelu_tanh", 0.5, d["R"][rows])
    assert_close(to_f64(Y[rows]), ref, 2e-2, 2e-2, "c2 sampled rows")
    # whole output: finite, and Y - R = 0.5*gelu(z) >= -0.085 (GELU's minimum is -0.17)
    import torch
    assert torch.isfinite(Y).all()
    diff = Y.float() - to_dev(d["R"]).float()
    assert float(diff.min()) > -0.12


def test_c3_full_size_sampled_rows(kf):
    d = ki.gemm_inputs("c3", seed=0)
    P = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "none", "softmax")
    check_status()
    rows = sample_rows(d["M"], 16, 3)
    ref = oracle.gemm_rowreduce(d["X"][rows], d["W"], d["b"], "none", "softmax")
    got = to_f64(P[rows])
    assert_close(got, ref, 2e-2, 2e-2, "c3 sampled rows")
    assert_close(got, ref, 1e-7, 2e-2, "c3 sampled rows, relative")
    sums = P.float().sum(dim=1)
    assert float((sums - 1).abs().max()) < 4e-3                  # every row of the output
    assert float(P.float().min()) > 0


def test_c4_full_size_sampled_rows(kf):
    d = ki.gemm_inputs("c4", seed=0)
    S = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "sigmoid", "sum")
    check_status()
    rows = sample_rows(d["M"], 100, 4)
    ref = oracle.gemm_rowreduce(d["X"][rows], d["W"], d["b"], "sigmoid", "sum")
    assert_close(to_f64(S[rows]), ref, 2e-2, 2e-2, "c4 sampled rows")
    assert_close(to_f64(S[rows]), ref, 0.0, 1e-3, "c4 sampled rows, relative")
    s = to_f64(S)
    assert ((s > 0) & (s < d["N"])).all() and abs(s.mean() - d["N"] / 2) < 2.0


def test_c5_full_size_sampled_images(kf):
    d = ki.conv_inputs("c5", seed=0)
    y = kf.conv3x3_epilogue(to_dev(d["x"]), to_dev(d["w"]), to_dev(d["bias"]), "relu", d["groups"], d["eps"])
    check_status()
    for n in (0, 77, d["Nb"] - 1):
        ref = oracle.conv3x3_gn(d["x"][n:n + 1], d["w"], d["bias"], "relu", d["groups"], d["eps"])
        assert_close(to_f64(y[n:n + 1]), ref, 2e-2, 2e-2, "c5 image %d" % n)
    blk = y.float().reshape(d["Nb"], d["groups"], -1)                # every (image, group) block
    assert float(blk.mean(dim=2).abs().max()) < 3e-3
    assert float((blk.var(dim=2, unbiased=False) - 1).abs().max()) < 1e-2


# ------------------------------------------------------------------ the widened paths at bench sizes
def test_split_k_skinny_full_size(kf):
    """bench.py --workload skinny: 64 x 8192 x 8192 through the split-K cluster kernel; the oracle
    recomputes sampled output columns (a column of Y needs one row of W)."""
    M, N, K = 64, 8192, 8192
    d = ki.gemm_inputs("c2", seed=5, M=M, N=N, K=K)
    Y = kf.gemm_epilogue(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "gelu_tanh", 0.5, to_dev(d["R"]))
    check_status()
    cols = sample_rows(N, 48, 6)          # both sides of the 64-column slices and 256-column tiles
    ref = oracle.gemm_epilogue(d["X"], d["W"][cols], d["b"][cols], "gelu_tanh", 0.5,
                               np.ascontiguousarray(d["R"][:, cols]))
    assert_close(to_f64(Y[:, cols]), ref, 2e-2, 2e-2, "split-K sampled columns")
    import torch
    assert torch.isfinite(Y).all()


def test_fp32_tensor_core_full_size_sampled_rows(kf):
    """bench.py --workload f32: 2048^3 fp32 through the 3xTF32 kernel, sampled rows."""
    M = N = K = 2048
    d = ki.gemm_inputs("c2", seed=7, M=M, N=N, K=K, dtype="f32")
    Y = kf.gemm_epilogue(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "gelu_tanh", 0.5, to_dev(d["R"]))
    check_status()
    rows = sample_rows(M, 24, 8)
    ref = oracle.gemm_epilogue(d["X"][rows], d["W"], d["b"], "gelu_tanh", 0.5, d["R"][rows])
    assert_close(to_f64(Y[rows]), ref, 1e-4, 1e-4, "fp32 3xTF32 sampled rows")
    import torch
    assert torch.isfinite(Y).all()
    diff = Y - to_dev(d["R"])
    assert float(diff.min()) > -0.0851           # 0.5 * min GELU = -0.08498...


def test_conv_softmax_pool_full_size_sampled_images(kf):
    """bench.py --workload pool: config 5's tensors, pool 4; the oracle recomputes three images."""
    d = ki.conv_inputs("c5", seed=0)
    y = kf.conv3x3_softmax_pool(to_dev(d["x"]), to_dev(d["w"]), to_dev(d["bias"]), 4)
    check_status()
    imgs = [0, 63, 127]
    ref = oracle.conv3x3_softmax_pool(d["x"][imgs], d["w"], d["bias"], 4)
    got = to_f64(y[imgs])
    assert_close(got, ref, 2e-2, 2e-2, "conv softmax pool sampled images")
    assert_close(got, ref, 1e-6, 2e-2, "conv softmax pool sampled images, relative")
    yy = y.float()
    assert float(yy.min()) > 0 and float(yy.max()) <= 1.0


def test_short_k_chain_full_size_sampled_rows(kf):
    """4096x4096x512 + bias + GELU*0.5 + residual: the single-CTA kernel with two epilogue groups
    and per-warp slabs, several waves, epilogue-bound."""
    d = ki.gemm_inputs("c2", seed=5, M=4096, N=4096, K=512)
    Y = kf.gemm_epilogue(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "gelu_tanh", 0.5, to_dev(d["R"]))
    check_status()
    rows = sample_rows(4096, 48, 6)
    ref = oracle.gemm_epilogue(d["X"][rows], d["W"], d["b"], "gelu_tanh", 0.5, d["R"][rows])
    assert_close(to_f64(Y[rows]), ref, 2e-2, 2e-2, "short-K chain sampled rows")
    import torch
    assert torch.isfinite(Y).all()
    assert float((Y.float() - to_dev(d["R"]).float()).min()) > -0.12


def test_conv_act_pool_full_size_sampled_images(kf):
    """conv + ReLU + max-pool 2 on config 5's tensors: pooled inside the convolution epilogue."""
    d = ki.conv_inputs("c5", seed=0)
    y = kf.conv3x3_act_pool(to_dev(d["x"]), to_dev(d["w"]), to_dev(d["bias"]), "relu", "max", 2)
    check_status()
    assert tuple(y.shape) == (128, 128, 32, 32)
    imgs = [0, 63, 127]
    ref = oracle.conv3x3_act_pool(d["x"][imgs], d["w"], d["bias"], "relu", "max", 2)
    assert_close(to_f64(y[imgs]), ref, 2e-2, 2e-2, "conv relu max-pool sampled images")
    assert float(y.float().min()) >= 0.0


def test_c5_two_kernel_route_full_size_sampled_images(kf, tuning):
    """Config 5 through the convolution + separate normalisation kernels (the route shapes take
    that do not qualify for the cluster form)."""
    tuning.setenv("KF_NO_FUSED_GN", "1")
    d = ki.conv_inputs("c5", seed=0)
    y = kf.conv3x3_epilogue(to_dev(d["x"]), to_dev(d["w"]), to_dev(d["bias"]), "relu", d["groups"], d["eps"])
    check_status()
    imgs = [0, 77, 127]
    ref = oracle.conv3x3_gn(d["x"][imgs], d["w"], d["bias"], "relu", d["groups"], d["eps"], None, None)
    assert_close(to_f64(y[imgs]), ref, 2e-2, 2e-2, "c5 two-kernel route sampled images")
