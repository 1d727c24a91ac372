"""GPU parity: the CUDA chains (called through the C ABI) against the fp64 CPU oracle, element by
element on the same seeded inputs.  Sizes span several tiles and ragged tails; the full-size
benchmark configurations are checked on sampled rows / images in test_gpu_fullsize.py."""
import math

import numpy as np
import pytest

import kf_inputs as ki
import oracle
from gpu_util import assert_close, check_status, to_dev, to_f64, tol_for

pytestmark = pytest.mark.gpu

ACTS = ["none", "relu", "gelu_tanh", "sigmoid", "gelu_erf", "swish", "tanh", "hardtanh", "chain95",
        "leaky_relu", "elu", "mish", "hardswish", "softplus", "relu6", "hardsigmoid"]
RUNTIME_ACTS = ACTS[9:]       # selected by a switch inside one kernel instantiation


@pytest.fixture(scope="module")
def kf():
    import paper_2605_30359_b200 as kf
    kf.lib()
    return kf


def run_gemm(kf, d, act, scale=1.0, use_bias=True, use_res=True):
    X, W = to_dev(d["X"]), to_dev(d["W"])
    b = to_dev(d["b"]) if use_bias else None
    R = to_dev(d["R"]) if (use_res and d["R"] is not None) else None
    Y = kf.gemm_epilogue(X, W, b, act, scale, R)
    check_status()
    ref = oracle.gemm_epilogue(d["X"], d["W"], d["b"] if use_bias else None, act, scale,
                               d["R"] if (use_res and d["R"] is not None) else None)
    return to_f64(Y), ref


# ------------------------------------------------------------------ config 1 (fp32), full size
def test_c1_fp32_linear_bias_relu(kf):
    d = ki.gemm_inputs("c1", seed=0)
    got, ref = run_gemm(kf, d, "relu")
    assert_close(got, ref, 1e-4, 1e-4, "c1")
    assert ((got == 0) == (ref <= 0)).mean() > 0.999


@pytest.mark.parametrize("shape", [(1, 1, 1), (3, 5, 7), (33, 65, 31), (100, 37, 129), (64, 64, 64)])
@pytest.mark.parametrize("act", ["none", "gelu_tanh", "sigmoid", "chain95"])
def test_fp32_ragged_shapes(kf, shape, act):
    M, N, K = shape
    d = ki.gemm_inputs("c2", seed=3, M=M, N=N, K=K, dtype="f32")
    got, ref = run_gemm(kf, d, act, 0.5)
    assert_close(got, ref, 1e-4, 1e-4, "fp32 %s %s" % (shape, act))


def test_fp32_gelu_variant_is_the_tanh_one(kf):
    # X = 0, b = -3: the two GELUs differ by 4.1e-4 there, four times the fp32 tolerance
    X = np.zeros((4, 8), np.float32); W = np.zeros((8, 8), np.float32)
    b = np.full(8, -3.0, np.float32)
    Y = kf.gemm_epilogue(to_dev(X), to_dev(W), to_dev(b), "gelu_tanh")
    assert_close(to_f64(Y), np.full((4, 8), oracle.act("gelu_tanh", -3.0)), 1e-4, 1e-4, "gelu fixed point")
    assert abs(to_f64(Y)[0, 0] - oracle.act("gelu_erf", -3.0)) > 3e-4


# ------------------------------------------------------------------ fp32 on the tensor cores (3xTF32)
# M*N*K >= 2^29 takes the split-operand tensor-core kernel; the result must stay within the
# fp32 tolerance whatever K is (accumulation is folded into an fp32 running sum every 512).
@pytest.mark.parametrize("shape", [(1024, 1024, 512),      # aligned: vector epilogue, one chunk
                                   (768, 640, 1100),       # three chunks, ragged last K block
                                   (1000, 999, 600),       # unaligned rows: scalar epilogue
                                   (256, 512, 4100)])      # nine chunks on two row tiles
def test_fp32_tensor_core_chain(kf, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c2", seed=41, M=M, N=N, K=K, dtype="f32")
    got, ref = run_gemm(kf, d, "gelu_tanh", 0.5)
    assert_close(got, ref, 1e-4, 1e-4, "fp32 3xTF32 %s" % (shape,))
    got, ref = run_gemm(kf, d, "none", 1.0, use_bias=False, use_res=False)
    assert_close(got, ref, 1e-4, 1e-4, "fp32 3xTF32 bare %s" % (shape,))
    assert np.abs(got - ref).max() < 3e-5       # an order of magnitude better than one-pass TF32


def test_fp32_tensor_core_chain_narrow_n(kf):
    """N <= 128 takes the 128-column instance of the fp32 tensor-core kernel."""
    d = ki.gemm_inputs("c2", seed=42, M=4096, N=128, K=1024, dtype="f32")
    got, ref = run_gemm(kf, d, "sigmoid", 1.0)
    assert_close(got, ref, 1e-4, 1e-4, "fp32 3xTF32 N=128")
    d = ki.gemm_inputs("c2", seed=43, M=8192, N=100, K=700, dtype="f32")      # ragged everywhere
    got, ref = run_gemm(kf, d, "tanh", 2.0)
    assert_close(got, ref, 1e-4, 1e-4, "fp32 3xTF32 N=100")


def test_fp32_tensor_core_layout_and_split_pins(kf):
    """One-hot X rows return W's entries: exact whenever an entry fits hi + lo (22 significant
    bits), so a wrong K block, swizzle or operand (hi/lo mixed up) shows as a mismatch."""
    M, N, K = 1024, 1024, 512
    r = np.random.default_rng(7)
    Wv = r.integers(-(1 << 21), 1 << 21, size=(N, K)).astype(np.float64) / (1 << 12)
    ks = r.integers(0, K, size=M)
    Xf = np.zeros((M, K)); Xf[np.arange(M), ks] = 1.0
    Y = kf.gemm_epilogue(to_dev(Xf.astype(np.float32)), to_dev(Wv.astype(np.float32)))
    check_status()
    assert_close(to_f64(Y), Wv[:, ks].T, 0.0, 0.0, "one-hot X rows, 3xTF32")
    # x = 1 + 2^-12 needs the lo part: (1 + 2^-12) * 1 summed over K
    Xs = np.full((M, K), 1.0 + 2.0 ** -12, np.float32)
    Y = kf.gemm_epilogue(to_dev(Xs), to_dev(np.ones((N, K), np.float32)))
    assert (to_f64(Y) == K * (1.0 + 2.0 ** -12)).all()


def test_fp32_tensor_core_workspace_is_checked(kf):
    import torch
    M, N, K = 1024, 1024, 512
    need = kf.kf_gemm_epilogue_workspace_bytes(M, N, K, kf.KF_F32)
    assert need == 2 * M * K * 4 + 2 * N * K * 4
    X = torch.zeros((M, K), device="cuda"); W = torch.zeros((N, K), device="cuda")
    Y = torch.empty((M, N), device="cuda")
    ws = torch.empty(need // 2, dtype=torch.uint8, device="cuda")
    st = kf.kf_gemm_epilogue(M, N, K, kf.KF_F32, X.data_ptr(), K, W.data_ptr(), K, None, 0, 1.0, None, 0,
                             Y.data_ptr(), N, ws.data_ptr(), need // 2, None)
    assert st == kf.KF_ERR_WORKSPACE
    assert kf.kf_gemm_epilogue_workspace_bytes(128, 256, 512, kf.KF_F32) == 0


# ------------------------------------------------------------------ run-time selected activations
@pytest.mark.parametrize("act", RUNTIME_ACTS)
def test_runtime_activations_every_kernel_family(kf, act):
    """Each further activation through every kernel family: fp32 FMA kernel, split-K cluster
    kernel, row reductions (softmax pre-activation and row sum), both convolution kernels."""
    d = ki.gemm_inputs("c2", seed=81, M=70, N=50, K=40, dtype="f32")                 # fp32 FMA
    got, ref = run_gemm(kf, d, act, 0.5)
    assert_close(got, ref, 1e-4, 1e-4, "fp32 %s" % act)
    d = ki.gemm_inputs("c2", seed=82, M=128, N=512, K=2048)                           # split-K cluster
    got, ref = run_gemm(kf, d, act, 2.0)
    assert_close(got, ref, 2e-2, 2e-2, "split-K %s" % act)
    d = ki.gemm_inputs("c3", seed=83, M=150, N=600, K=136)
    for red in ("softmax", "sum"):
        out = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), act, red)
        ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], act, red)
        assert_close(to_f64(out), ref, 2e-2, 2e-2, "%s of %s" % (red, act))
        if red == "sum":
            assert_close(to_f64(out), ref, 1e-3, 3e-3, "row sum of %s, relative" % act)
    # tensor-core conv; no GroupNorm here: after a squashing activation (hardsigmoid's outputs
    # have a standard deviation of 0.05) the normalisation multiplies the bf16 rounding of the
    # stored activations by 20, which says nothing about the activation itself
    dc = ki.conv_inputs(seed=84, Nb=2, Cin=64, H=8, W=64, Cout=96, groups=0)
    got, ref = run_conv(kf, dc, act=act)
    assert_close(got, ref, 2e-2, 2e-2, "conv %s" % act)
    if act == "mish":
        dc = ki.conv_inputs(seed=84, Nb=2, Cin=64, H=8, W=64, Cout=96, groups=3)
        got, ref = run_conv(kf, dc, act=act)
        assert_close(got, ref, 2e-2, 2e-2, "conv %s + GroupNorm" % act)
    dc = ki.conv_inputs(seed=85, Nb=1, Cin=3, H=5, W=7, Cout=4, groups=0, dtype="f32")  # direct conv
    got, ref = run_conv(kf, dc, act=act)
    assert_close(got, ref, 1e-4, 1e-4, "direct conv %s" % act)
    check_status()


@pytest.mark.parametrize("act", ["mish", "elu", "softplus"])
def test_runtime_activations_fp32_tensor_core(kf, act):
    d = ki.gemm_inputs("c2", seed=86, M=1024, N=1024, K=512, dtype="f32")
    got, ref = run_gemm(kf, d, act, 1.0)
    assert_close(got, ref, 1e-4, 1e-4, "fp32 3xTF32 %s" % act)


# ------------------------------------------------------------------ bf16 tensor-core GEMM
def test_bf16_layout_pins_onehot_and_permutation(kf):
    """Products by 0/1 are exact, so any mismatch is a layout / swizzle / descriptor bug."""
    M, N, K = 256, 512, 192
    r = np.random.default_rng(5)
    Wv = (r.integers(-64, 65, size=(N, K)) / 64.0)
    ks = r.integers(0, K, size=M)
    Xf = np.zeros((M, K)); Xf[np.arange(M), ks] = 1.0
    Y = kf.gemm_epilogue(to_dev(ki.store(Xf, "bf16")), to_dev(ki.store(Wv, "bf16")))
    check_status()
    assert_close(to_f64(Y), Wv[:, ks].T, 0.0, 0.0, "one-hot X rows")
    K2 = 512
    Xv = (r.integers(-64, 65, size=(M, K2)) / 64.0)
    perm = r.permutation(K2)
    Wp = np.zeros((K2, K2)); Wp[np.arange(K2), perm] = 1.0
    Y = kf.gemm_epilogue(to_dev(ki.store(Xv, "bf16")), to_dev(ki.store(Wp, "bf16")))
    check_status()
    assert_close(to_f64(Y), Xv[:, perm], 0.0, 0.0, "permutation W")


@pytest.mark.parametrize("act", ACTS)
def test_bf16_gemm_epilogue_all_activations(kf, act):
    d = ki.gemm_inputs("c2", seed=1, M=300, N=520, K=200)       # 3x3 tiles, ragged in M, N and K
    got, ref = run_gemm(kf, d, act, 0.5)
    assert_close(got, ref, 2e-2, 2e-2, "bf16 %s" % act)


@pytest.mark.parametrize("shape", [(128, 256, 64), (1, 8, 8), (129, 264, 72), (640, 128, 1024),
                                   (257, 1000, 136), (130, 100, 64)])
def test_bf16_gemm_shapes(kf, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c2", seed=2, M=M, N=N, K=K)
    got, ref = run_gemm(kf, d, "gelu_tanh", 0.5)
    assert_close(got, ref, 2e-2, 2e-2, "bf16 %s" % (shape,))


# One-wave problems take the narrowest tile that keeps them in one wave (32, 64, 128 or 256
# columns); rows of Y / R that do not start on 16 bytes take the epilogue without TMA.
@pytest.mark.parametrize("shape", [(1024, 1000, 64),      # 64-column tiles
                                   (2048, 777, 72),       # 128-column tiles, unaligned rows
                                   (2304, 1030, 64),      # 256-column tiles, unaligned rows
                                   (333, 777, 520),       # 32-column tiles, unaligned rows
                                   (128, 33, 8)])         # one tile, one ragged piece + 1 column
def test_bf16_gemm_tile_widths_and_unaligned_rows(kf, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c2", seed=21, M=M, N=N, K=K)
    got, ref = run_gemm(kf, d, "swish", 2.0)
    assert_close(got, ref, 2e-2, 2e-2, "bf16 %s" % (shape,))
    got, ref = run_gemm(kf, d, "none", 1.0, use_bias=False, use_res=False)
    assert_close(got, ref, 2e-2, 2e-2, "bf16 bare %s" % (shape,))


# Few tiles and a long K take the split-K cluster kernel: 4 or 8 CTAs per tile, partial tiles
# exchanged through distributed shared memory, slices of 64 or 32 columns finished per CTA.
@pytest.mark.parametrize("shape", [(128, 1024, 2048),     # 4 tiles x 8 CTAs, 256-column tiles
                                   (200, 300, 1800),      # 4 tiles x 4 CTAs, ragged M, N, K (28.1 K blocks)
                                   (100, 128, 4096),      # 128-column tile x 4 CTAs
                                   (64, 2000, 2048),      # 8 tiles x 8 CTAs, last tile ragged in N
                                   (130, 777, 1848),      # unaligned rows: scalar stores
                                   (16, 5000, 2048),      # 40 tiles x 4 CTAs, two CTAs per SM, 32 live rows
                                   (40, 4800, 8192),      # ... long K shares, 64 live rows
                                   (97, 2048, 1920)])     # 128 live rows, one CTA per SM
def test_bf16_gemm_split_k_cluster_kernel(kf, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c2", seed=31, M=M, N=N, K=K)
    for act, scale, res in [("gelu_tanh", 0.5, True), ("none", 1.0, False), ("chain95", 1.0, True)]:
        got, ref = run_gemm(kf, d, act, scale, use_res=res)
        assert_close(got, ref, 2e-2, 2e-2, "bf16 split-K %s %s" % (shape, act))
    # the same call again gives the same bits (fixed summation order across the cluster)
    X, W, b = to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"])
    y1 = kf.gemm_epilogue(X, W, b, "swish")
    y2 = kf.gemm_epilogue(X, W, b, "swish")
    assert (y1.view(__import__("torch").int16) == y2.view(__import__("torch").int16)).all()


def test_bf16_split_k_layout_pins(kf):
    """One-hot X rows through the split-K kernel: every K share and column slice lands in place."""
    M, N, K = 128, 512, 4096
    r = np.random.default_rng(6)
    Wv = (r.integers(-64, 65, size=(N, K)) / 64.0)
    ks = r.integers(0, K, size=M)
    Xf = np.zeros((M, K)); Xf[np.arange(M), ks] = 1.0
    Y = kf.gemm_epilogue(to_dev(ki.store(Xf, "bf16")), to_dev(ki.store(Wv, "bf16")))
    check_status()
    assert_close(to_f64(Y), Wv[:, ks].T, 0.0, 0.0, "one-hot X rows, split-K")
    # all-ones: each of the 8 K shares contributes K/8; the exact sum needs all of them once
    Y = kf.gemm_epilogue(to_dev(ki.store(np.ones((M, K)), "bf16")), to_dev(ki.store(np.ones((N, K)) / 64, "bf16")))
    assert (to_f64(Y) == K / 64).all()


# bf16 operands whose K is not a multiple of 8 cannot be loaded by TMA as they are; problems large
# enough are repacked (zero-padded rows) into the workspace and take the tensor cores anyway.
@pytest.mark.parametrize("shape", [(512, 520, 1001), (300, 257, 4099)])
def test_bf16_gemm_repacked_operands(kf, shape):
    M, N, K = shape
    assert kf.kf_gemm_epilogue_workspace_bytes(M, N, K, kf.KF_BF16) > 0
    d = ki.gemm_inputs("c2", seed=51, M=M, N=N, K=K)
    got, ref = run_gemm(kf, d, "gelu_tanh", 0.5)
    assert_close(got, ref, 2e-2, 2e-2, "bf16 repacked %s" % (shape,))
    d3 = ki.gemm_inputs("c3", seed=52, M=M, N=N, K=K)
    P = kf.gemm_rowreduce(to_dev(d3["X"]), to_dev(d3["W"]), to_dev(d3["b"]), "none", "softmax")
    check_status()
    ref = oracle.gemm_rowreduce(d3["X"], d3["W"], d3["b"], "none", "softmax")
    assert_close(to_f64(P), ref, 2e-2, 2e-2, "bf16 repacked softmax %s" % (shape,))
    assert_close(to_f64(P), ref, 1e-7, 2e-2, "bf16 repacked softmax, relative %s" % (shape,))


# Softmax output rows that do not start on 16 bytes (odd N): numerators leave through shared
# memory along rows, the second pass works in aligned vectors between a scalar head and tail.
@pytest.mark.parametrize("shape", [(300, 4101, 136),      # 34 slices: block-per-row second pass
                                   (260, 1001, 72),       # 64-column tiles, warp-per-row second pass
                                   (129, 50257, 64)])     # vocabulary-sized odd N
def test_bf16_softmax_unaligned_rows(kf, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=61, M=M, N=N, K=K)
    P = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "none", "softmax")
    check_status()
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", "softmax")
    got = to_f64(P)
    assert_close(got, ref, 2e-2, 2e-2, "softmax odd N %s" % (shape,))
    assert_close(got, ref, 1e-7, 2e-2, "softmax odd N, relative %s" % (shape,))
    assert np.abs(got.sum(axis=1) - 1).max() < 4e-3


# K >= 2048 with more than 256 rows and enough K blocks per CTA takes the CTA-pair kernel (256-row
# tiles over two SMs); these small shapes reach it with the work threshold switched off
@pytest.mark.parametrize("shape", [(384, 520, 2048), (257, 256, 2112), (1000, 264, 2048)])
def test_bf16_gemm_cta_pair_kernel(kf, shape, tuning):
    tuning.setenv("KF_PAIR_MIN_KB_PER_CTA", "0")
    M, N, K = shape
    d = ki.gemm_inputs("c2", seed=12, M=M, N=N, K=K)
    got, ref = run_gemm(kf, d, "gelu_tanh", 0.5)
    assert_close(got, ref, 2e-2, 2e-2, "bf16 pair %s" % (shape,))


def test_bf16_cta_pair_layout_pins(kf, tuning):
    """One-hot rows through the pair kernel: each CTA's A half and B half must land where the
    256-row MMA expects them."""
    tuning.setenv("KF_PAIR_MIN_KB_PER_CTA", "0")
    M, N, K = 640, 512, 2048
    r = np.random.default_rng(6)
    Wv = (r.integers(-64, 65, size=(N, K)) / 64.0)
    ks = r.integers(0, K, size=M)
    Xf = np.zeros((M, K)); Xf[np.arange(M), ks] = 1.0
    Y = kf.gemm_epilogue(to_dev(ki.store(Xf, "bf16")), to_dev(ki.store(Wv, "bf16")))
    check_status()
    assert_close(to_f64(Y), Wv[:, ks].T, 0.0, 0.0, "one-hot X rows, pair kernel")


@pytest.mark.parametrize("red,act,shape", [("softmax", "none", (300, 1000, 2048)),
                                           ("sum", "sigmoid", (520, 512, 2048))])
def test_bf16_row_reductions_cta_pair_kernel(kf, red, act, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=13, M=M, N=N, K=K)
    out = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), act, red)
    check_status()
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], act, red)
    if red == "softmax":
        softmax_gates(to_f64(out), ref, "softmax pair %s" % (shape,))
    else:
        assert_close(to_f64(out), ref, 0.0, 1e-3, "rowsum pair %s" % (shape,))


@pytest.mark.parametrize("shape", [(5, 7, 3), (17, 9, 13), (40, 33, 20)])
def test_bf16_unaligned_shapes_take_the_scalar_kernel(kf, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c2", seed=4, M=M, N=N, K=K)
    got, ref = run_gemm(kf, d, "gelu_tanh", 0.5)
    assert_close(got, ref, 2e-2, 2e-2, "bf16 scalar %s" % (shape,))


def test_bf16_zero_inputs_return_residual_bit_exact(kf):
    d = ki.gemm_inputs("c2", seed=6, M=256, N=256, K=128)
    Z = np.zeros_like(d["X"])
    zb = np.zeros_like(d["b"])
    Y = kf.gemm_epilogue(to_dev(Z), to_dev(d["W"]), to_dev(zb), "gelu_tanh", 0.5, to_dev(d["R"]))
    assert np.array_equal(to_f64(Y), ki.widen(d["R"]))
    # X = 0, b = value: every row equals scale*act(b) + R
    Y = kf.gemm_epilogue(to_dev(Z), to_dev(d["W"]), to_dev(d["b"]), "relu", 2.0, None)
    want = 2.0 * np.maximum(ki.widen(d["b"]), 0.0)
    assert_close(to_f64(Y), np.broadcast_to(want, (256, 256)), 2e-2, 2e-2, "X=0")


def test_bf16_no_bias_no_residual_and_strided_operands(kf):
    import torch
    d = ki.gemm_inputs("c2", seed=7, M=200, N=264, K=128)
    got, ref = run_gemm(kf, d, "relu", 1.0, use_bias=False, use_res=False)
    assert_close(got, ref, 2e-2, 2e-2, "no bias")
    # leading dimensions larger than the row length
    Xp = torch.zeros(200, 160, dtype=torch.bfloat16, device="cuda"); Xp[:, :128] = to_dev(d["X"])
    Yp = torch.full((200, 272), 7.0, dtype=torch.bfloat16, device="cuda")
    kf.gemm_epilogue(Xp[:, :128], to_dev(d["W"]), to_dev(d["b"]), "relu", 1.0, None, out=Yp[:, :264])
    check_status()
    ref = oracle.gemm_epilogue(d["X"], d["W"], d["b"], "relu")
    assert_close(to_f64(Yp[:, :264]), ref, 2e-2, 2e-2, "strided")
    assert (Yp[:, 264:] == 7.0).all()                          # padding columns untouched


def test_repeat_runs_are_bit_identical(kf):
    d = ki.gemm_inputs("c3", seed=8, M=300, N=1100, K=256)
    X, W, b = to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"])
    a1 = kf.gemm_rowreduce(X, W, b, "none", "softmax").clone()
    s1 = kf.gemm_rowreduce(X, W, b, "sigmoid", "sum").clone()
    for _ in range(3):
        assert (kf.gemm_rowreduce(X, W, b, "none", "softmax") == a1).all()
        assert (kf.gemm_rowreduce(X, W, b, "sigmoid", "sum") == s1).all()


# ------------------------------------------------------------------ row reductions
def softmax_gates(got, ref, what):
    assert_close(got, ref, 2e-2, 2e-2, what)                     # the official (weak) tolerance
    assert_close(got, ref, 1e-7, 2e-2, what + " relative")       # elementwise relative error
    assert np.abs(got.sum(axis=1) - 1.0).max() < 4e-3, what


@pytest.mark.parametrize("shape", [(200, 1000, 136), (128, 256, 64), (300, 2056, 512), (1, 8, 8)])
def test_bf16_softmax(kf, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=1, M=M, N=N, K=K)
    P = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "none", "softmax")
    check_status()
    softmax_gates(to_f64(P), oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", "softmax"),
                  "softmax %s" % (shape,))


def test_bf16_softmax_fp32_output_and_closed_forms(kf):
    import torch
    N, K = 1024, 64
    X = np.zeros((130, K)); W = ki.normal(1, 2, (N, K))
    b = np.full(N, 0.75)
    P = kf.gemm_rowreduce(to_dev(ki.store(X, "bf16")), to_dev(ki.store(W, "bf16")),
                          to_dev(ki.store(b, "bf16")), "none", "softmax", out_dtype=torch.float32)
    check_status()
    assert_close(to_f64(P), np.full((130, N), 1.0 / N), 0.0, 1e-6, "constant row")
    # one logit far above the rest: one-hot, no overflow
    b2 = np.zeros(N); b2[700] = 120.0
    P = kf.gemm_rowreduce(to_dev(ki.store(X, "bf16")), to_dev(ki.store(W, "bf16")),
                          to_dev(ki.store(b2, "bf16")), "none", "softmax", out_dtype=torch.float32)
    got = to_f64(P)
    assert not np.isnan(got).any() and (got[:, 700] == 1.0).all() and got.sum() == 130.0
    d = ki.gemm_inputs("c3", seed=2, M=150, N=1024, K=128)
    P = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "none", "softmax",
                          out_dtype=torch.float32)
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", "softmax")
    assert_close(to_f64(P), ref, 1e-7, 1e-3, "softmax fp32 out")


@pytest.mark.parametrize("shape", [(200, 1000, 136), (128, 256, 64), (513, 1024, 256)])
def test_bf16_sigmoid_rowsum(kf, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c4", seed=1, M=M, N=N, K=K)
    S = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "sigmoid", "sum")
    check_status()
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "sigmoid", "sum")
    assert_close(to_f64(S), ref, 2e-2, 2e-2, "rowsum %s" % (shape,))
    assert_close(to_f64(S), ref, 0.0, 1e-3, "rowsum relative %s" % (shape,))


def test_bf16_rowsum_row_owner_schedule(kf):
    """148 row blocks x 2 column tiles: each CTA owns whole row blocks, carries the sum across
    its tiles and writes out[m] itself (no partial buffer, one kernel)."""
    M, N, K = 18900, 512, 64
    d = ki.gemm_inputs("c4", seed=2, M=M, N=N, K=K)
    before = kf.kf_launch_count()
    S = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "sigmoid", "sum")
    check_status()
    assert kf.kf_launch_count() - before == 1
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "sigmoid", "sum")
    assert_close(to_f64(S), ref, 0.0, 1e-3, "rowsum row-owner")


def test_rowsum_closed_forms(kf):
    N, K = 1024, 128
    d = ki.gemm_inputs("c4", seed=3, M=256, N=N, K=K)
    zX = np.zeros_like(d["X"]); zb = np.zeros_like(d["b"])
    S = kf.gemm_rowreduce(to_dev(zX), to_dev(d["W"]), to_dev(zb), "sigmoid", "sum")
    assert_close(to_f64(S), np.full(256, N / 2), 0.0, 1e-6, "X=0,b=0")
    # sigmoid(z)+sigmoid(-z)=1: stacking W with -W and b with -b gives N per row for any X
    W2 = np.concatenate([ki.widen(d["W"])[:512], -ki.widen(d["W"])[:512]])
    b2 = np.concatenate([ki.widen(d["b"])[:512], -ki.widen(d["b"])[:512]])
    S = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(ki.store(W2, "bf16")), to_dev(ki.store(b2, "bf16")),
                          "sigmoid", "sum")
    assert_close(to_f64(S), np.full(256, 512.0), 0.0, 1e-4, "antisymmetry")


@pytest.mark.parametrize("red,act", [("softmax", "none"), ("sum", "sigmoid"), ("softmax", "relu")])
@pytest.mark.parametrize("dtype,shape", [("f32", (33, 70, 31)), ("f32", (128, 256, 512)), ("bf16", (9, 21, 13)),
                                         ("f32", (1024, 1000, 600))])   # GEMM on the tensor cores (3xTF32)
def test_scalar_path_row_reductions(kf, red, act, dtype, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=4, M=M, N=N, K=K, dtype=dtype)
    out = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), act, red)
    check_status()
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], act, red)
    atol, rtol = tol_for(dtype)
    assert_close(to_f64(out), ref, atol, rtol, "scalar %s %s %s" % (red, dtype, shape))
    if red == "softmax":
        assert_close(to_f64(out), ref, 1e-7, 2e-4 if dtype == "f32" else 2e-2, "relative")


# ------------------------------------------------------------------ row max / mean / log-sum-exp
@pytest.mark.parametrize("red", ["max", "mean", "logsumexp"])
@pytest.mark.parametrize("dtype,shape", [("bf16", (300, 1000, 136)),      # 64-column tiles, ragged
                                         ("bf16", (2500, 2056, 264)),     # 256-column tiles, several waves
                                         ("bf16", (9, 21, 13)),           # scalar path
                                         ("f32", (130, 70, 33)),          # fp32 scalar path
                                         ("f32", (1024, 1000, 600))])     # fp32 GEMM on the tensor cores
def test_row_max_mean_logsumexp(kf, red, dtype, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=91, M=M, N=N, K=K, dtype=dtype)
    out = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "gelu_tanh", red)
    check_status()
    assert tuple(out.shape) == (M,)
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "gelu_tanh", red)
    atol, rtol = tol_for(dtype)
    assert_close(to_f64(out), ref, atol, rtol, "%s %s %s" % (red, dtype, shape))
    # tighter: a mean averages the rounding of N terms, max and log-sum-exp are dominated by few
    tight = {"max": 5e-3, "mean": 2e-3, "logsumexp": 5e-3}[red] if dtype == "bf16" else 1e-4
    assert np.abs(to_f64(out) - ref).max() < tight


def test_row_reductions_reject_bad_arguments(kf):
    import torch
    X = torch.zeros((8, 8), device="cuda", dtype=torch.bfloat16)
    out = torch.zeros((8,), device="cuda", dtype=torch.bfloat16)
    for red in (2, 3, 4):        # a scalar-valued reduction needs an fp32 output
        st = kf.kf_gemm_rowreduce(8, 8, 8, kf.KF_BF16, X.data_ptr(), 8, X.data_ptr(), 8, None, 0, red,
                                  out.data_ptr(), 1, kf.KF_BF16, None, 0, None)
        assert st == kf.KF_ERR_INVALID_ARG
    st = kf.kf_gemm_rowreduce(8, 8, 8, kf.KF_BF16, X.data_ptr(), 8, X.data_ptr(), 8, None, 0, 5,
                              out.data_ptr(), 1, kf.KF_F32, None, 0, None)
    assert st == kf.KF_ERR_INVALID_ARG


# ------------------------------------------------------------------ GEMM + GroupNorm over column groups
@pytest.mark.parametrize("dtype,shape,groups", [
    ("bf16", (300, 1024, 136), 32),      # groups of 32 columns: one piece each, in the epilogue
    ("bf16", (257, 512, 72), 2),         # groups of 256: a whole tile
    ("bf16", (1000, 640, 2048), 5),      # groups of 128, CTA pairs, ragged last tile (640 = 2.5 tiles)
    ("bf16", (130, 192, 64), 3),         # groups of 64
    ("bf16", (64, 96, 40), 4),           # groups of 24: FMA kernel + row kernel
    ("bf16", (512, 960, 264), 8),        # groups of 120 on a larger problem: fused GEMM + in-place row kernel
    ("bf16", (64, 1024, 64), 1),         # one group of 1024 (LayerNorm): tile statistics + row pass
    ("bf16", (300, 2048, 136), 4),       # groups of 512 = two tiles each, ragged M
    ("bf16", (512, 1024, 2048), 1),      # the same through the CTA-pair kernel
    ("f32", (70, 60, 33), 5),            # fp32 scalar path
    ("f32", (1024, 1024, 512), 16),      # fp32 GEMM on the tensor cores, then the row kernel
])
def test_gemm_groupnorm(kf, dtype, shape, groups, tuning):
    M, N, K = shape
    if K >= 2048:
        tuning.setenv("KF_PAIR_MIN_KB_PER_CTA", "0")    # small shapes through the CTA-pair kernel
    d = ki.gemm_inputs("c3", seed=95, M=M, N=N, K=K, dtype=dtype)
    gamma = ki.store(ki.uniform(95, 7, (N,), 0.5, 1.5), dtype)
    beta = ki.store(ki.uniform(95, 8, (N,), -1.0, 1.0), dtype)
    atol, rtol = tol_for(dtype)          # fp32: 1e-4 / 1e-4 (measured worst err/limit 0.09 on the 3xTF32 route)
    for post, g_, b_ in (("none", None, None), ("swish", gamma, beta)):
        Y = kf.gemm_groupnorm(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), groups, 1e-5,
                              to_dev(g_), to_dev(b_), post)
        check_status()
        ref = oracle.gemm_groupnorm(d["X"], d["W"], d["b"], groups, 1e-5, g_, b_, post)
        assert_close(to_f64(Y), ref, atol, rtol, "gemm groupnorm %s %s g=%d %s" % (dtype, shape, groups, post))
    # unit moments of every (row, group) of the plain normalisation
    Y = to_f64(kf.gemm_groupnorm(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), groups, 1e-5))
    blk = Y.reshape(M, groups, N // groups)
    assert np.abs(blk.mean(axis=2)).max() < (2e-2 if dtype == "bf16" else 1e-4)
    assert np.abs(blk.var(axis=2) - 1.0).max() < (5e-2 if dtype == "bf16" else 1e-3)


# Rows of several whole 256-column tiles in ONE kernel on every SM: the tiles of a row block sit on
# neighbouring CTAs of a cooperative grid, exchange per-row (maximum, sum) through global memory and
# write final probabilities; the numerators wait in registers.  Normally taken from K = 2048 on
# problems of two waves; the knob forces it on small ones (single-CTA form below K = 2048, CTA pairs
# from there).
@pytest.mark.parametrize("shape,act", [
    ((1000, 1024, 256), "none"),        # 8 row blocks x 4 tiles, ragged last row block
    ((640, 2048, 128), "gelu_tanh"),    # a pre-activation; 5 x 8 tiles
    ((256, 16384, 64), "none"),         # 64 tiles per row: two rounds of the schedule per row block
    ((40000, 512, 64), "none"),         # 313 row blocks x 2 tiles: many rounds, exchange rows of many blocks
    ((1536, 1024, 2048), "none"),       # CTA pairs (K = 2048): 256-row tiles, both CTAs publish their own rows
    ((700, 768, 2112), "relu"),         # CTA pairs, ragged last pair (rows 512..699), 33 K blocks
])
def test_bf16_softmax_wide_rows_one_kernel(kf, shape, act, tuning):
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=17, M=M, N=N, K=K)
    tuning.setenv("KF_SOFTMAX_GX_MIN_TILES", "1")
    before = kf.kf_launch_count()
    P = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), act, "softmax")
    check_status()
    assert kf.kf_launch_count() - before == 1                # the one-kernel route was taken
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], act, "softmax")
    got = to_f64(P)
    assert_close(got, ref, 2e-2, 2e-2, "softmax one kernel %s" % (shape,))
    assert_close(got, ref, 1e-7, 2e-2, "softmax one kernel, relative %s" % (shape,))
    assert np.abs(got.sum(axis=1) - 1.0).max() < 4e-3
    P2 = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), act, "softmax")
    assert (to_f64(P2) == got).all()                          # fixed order of the exchange: bit-identical repeats
    tuning.setenv("KF_NO_WIDE_STORE", "1")                    # whole pieces behind group barriers instead of per-warp slabs
    P3 = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), act, "softmax")
    assert (to_f64(P3) == got).all()


def _softmax_gx_fuzz_cases():
    rng = np.random.default_rng(20261126)
    cases = []
    while len(cases) < 6:
        M = int(rng.integers(100, 9000))
        N = 256 * int(rng.integers(2, 11))
        K = 8 * int(rng.integers(8, 280))                  # 64..2232: both the single-CTA form and CTA pairs
        # (problems of one wave of 256-column tiles take 64-column tiles and another route)
        if M * N * K > 6e9 or ((M + 127) // 128) * (N // 256) <= 160:
            continue
        cases.append((M, N, K))
    return cases


@pytest.mark.parametrize("shape", _softmax_gx_fuzz_cases())
def test_bf16_softmax_wide_rows_one_kernel_seeded_shapes(kf, shape, tuning):
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=29, M=M, N=N, K=K)
    tuning.setenv("KF_SOFTMAX_GX_MIN_TILES", "1")
    before = kf.kf_launch_count()
    P = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "none", "softmax")
    check_status()
    assert kf.kf_launch_count() - before == 1                # the one-kernel route was taken
    got = to_f64(P)
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", "softmax")
    assert_close(got, ref, 2e-2, 2e-2, "softmax one kernel, seeded shape %s" % (shape,))
    assert_close(got, ref, 1e-7, 2e-2, "softmax one kernel, seeded shape, relative %s" % (shape,))
    # the two-kernel route on the same inputs
    tuning.setenv("KF_NO_SOFTMAX_GX", "1")
    P2 = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "none", "softmax")
    assert_close(to_f64(P2), got, 1e-7, 2e-2, "softmax one kernel against two kernels %s" % (shape,))


# Rows that lie in one tile (N <= 256, or <= 64 on the narrow-tile kernel): the softmax is finished
# inside the GEMM epilogue (maxima and sums exchanged between the two epilogue groups), no second
# kernel runs.
@pytest.mark.parametrize("shape", [(20000, 256, 64), (19000, 200, 264), (4096, 136, 64), (129, 64, 128),
                                   (77, 40, 72), (5120, 256, 2048), (19500, 250, 72), (128, 8, 64),
                                   (300, 256, 512),          # clusters of 4 column tiles
                                   (1000, 1000, 304),        # clusters of 16, ragged last tile (1000 = 15.6 x 64)
                                   (2500, 136, 1024),        # clusters of 3, twenty row blocks
                                   (128, 1024, 2048),        # clusters of 16 x 32 K blocks
                                   (1024, 1024, 1024),       # 128-column tiles, clusters of 8
                                   (1100, 1000, 64),         # ... ragged last tile and row block
                                   (1700, 600, 520),         # ... fourteen row blocks, clusters of 5
                                   (1024, 768, 512)])        # 96 narrow CTAs: the 128-column form, clusters of 6
def test_bf16_softmax_one_kernel(kf, shape, tuning):
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=41, M=M, N=N, K=K)
    args = (to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]))
    before = kf.kf_launch_count()
    P = kf.gemm_rowreduce(*args, "relu", "softmax")
    launches = kf.kf_launch_count() - before
    check_status()
    ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "relu", "softmax")
    got = to_f64(P)
    assert_close(got, ref, 2e-2, 2e-2, "softmax in one tile %s" % (shape,))
    assert np.abs(got.sum(axis=1) - 1.0).max() < 1e-2
    # 64-column tiles when they fit in one wave, else 256-column tiles.  One kernel when a row
    # lies in one tile, or in 2..16 narrow tiles (their CTAs form a cluster); else two.
    bn = 64 if ((M + 127) // 128) * ((N + 63) // 64) <= 148 else 256
    tiles = ((M + 127) // 128) * ((N + 63) // 64)
    # Narrow-tile clusters of more than 80 CTAs (or that would not all be resident, more than
    # 112): 128-column tiles in clusters of at most 8, while those are at most 120 CTAs.
    cl128 = bn == 64 and 2 <= (N + 127) // 128 <= 8 and ((M + 127) // 128) * ((N + 127) // 128) <= 120
    cl64 = bn == 64 and (N + 63) // 64 <= 16 and tiles <= (80 if cl128 else 112)
    assert launches == (1 if (N <= bn or cl64 or cl128) else 2)
    # the two-kernel route gives the same probabilities up to the rounding of the numerators
    tuning.setenv("KF_NO_FUSED_SOFTMAX", "1")
    tuning.setenv("KF_NO_CLUSTER_SOFTMAX", "1")
    P2 = to_f64(kf.gemm_rowreduce(*args, "relu", "softmax"))
    assert np.abs(P2 - got).max() <= 2.0 ** -7 * max(1e-30, got.max())
    # fp32 probabilities from the same kernel family
    tuning.delenv("KF_NO_FUSED_SOFTMAX")
    tuning.delenv("KF_NO_CLUSTER_SOFTMAX")
    import torch
    P32 = kf.gemm_rowreduce(*args, "relu", "softmax", out_dtype=torch.float32)
    check_status()
    assert_close(to_f64(P32), ref, 2e-2, 2e-2, "softmax in one tile, fp32 out %s" % (shape,))


# ------------------------------------------------------------------ seeded shape fuzz across the dispatch rules
def _fuzz_shapes(seed, count):
    """bf16 GEMM shapes around the dispatch boundaries: tile widths 32..256, one or two epilogue
    groups, CTA pairs (M > 256, K >= 2048), split-K (few tiles, K >= 1792), rows that TMA cannot
    store (odd N), operands that TMA cannot load (K not a multiple of 8: repacked or scalar)."""
    r = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        M = int(r.choice([1, 31, 64, 100, 128, 129, 257, 300, 512, 640]))
        N = int(r.choice([8, 40, 64, 96, 136, 256, 264, 333, 512, 776, 1024]))
        K = int(r.choice([8, 64, 72, 200, 512, 1000, 1027, 1536, 1800, 2048, 2304]))
        out.append((M, N, K))
    return out


@pytest.mark.parametrize("shape", _fuzz_shapes(2024, 28))
def test_fuzz_bf16_gemm_chain(kf, shape, tuning):
    M, N, K = shape
    d = ki.gemm_inputs("c2", seed=M + 3 * N + 7 * K, M=M, N=N, K=K)
    opts = [("gelu_tanh", 0.5, True, True), ("relu", 1.0, True, False), ("none", 1.0, False, False),
            ("mish", 2.0, False, True)]
    act, scale, use_bias, use_res = opts[(M + N + K) % 4]
    got, ref = run_gemm(kf, d, act, scale, use_bias=use_bias, use_res=use_res)
    assert_close(got, ref, 2e-2, 2e-2, "fuzz chain %s %s" % (shape, act))
    if M > 256 and K >= 2048:         # the same through the CTA-pair kernel (work threshold off)
        tuning.setenv("KF_PAIR_MIN_KB_PER_CTA", "0")
        got, ref = run_gemm(kf, d, act, scale, use_bias=use_bias, use_res=use_res)
        assert_close(got, ref, 2e-2, 2e-2, "fuzz chain, pairs %s %s" % (shape, act))


@pytest.mark.parametrize("shape", _fuzz_shapes(77, 16))
def test_fuzz_bf16_gemm_rowreduce(kf, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=M + 5 * N + K, M=M, N=N, K=K)
    for act, red in (("none", "softmax"), ("sigmoid", "sum"), ("relu", "logsumexp")):
        out = kf.gemm_rowreduce(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), act, red)
        check_status()
        ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], act, red)
        if red == "softmax":
            assert_close(to_f64(out), ref, 2e-2, 2e-2, "fuzz softmax %s" % (shape,))
            assert np.abs(to_f64(out).sum(axis=1) - 1.0).max() < 2e-2
        else:
            # a sum of N terms, each within the bf16-input tolerance: compare relative to N
            err = np.abs(to_f64(out) - ref).max()
            assert err <= 2e-2 * max(1.0, np.abs(ref).max()), "fuzz %s %s: %g" % (red, shape, err)


@pytest.mark.parametrize("shape,groups", [((300, 256, 512), 8), ((129, 512, 1000), 4), ((64, 1024, 2048), 8),
                                          ((640, 768, 256), 3), ((257, 384, 72), 12), ((100, 512, 2304), 2),
                                          ((512, 256, 64), 1)])
def test_fuzz_bf16_gemm_groupnorm(kf, shape, groups):
    """Group widths 32, 64, 128 (inside one epilogue group's half tile), 256 (per-slice statistics
    + second pass, single-CTA and pair kernels), 1024 and an odd width (row kernel)."""
    M, N, K = shape
    d = ki.gemm_inputs("c3", seed=N + K, M=M, N=N, K=K)
    gamma = ki.store(ki.uniform(5, 7, (N,), 0.5, 1.5), "bf16")
    beta = ki.store(ki.uniform(5, 8, (N,), -1.0, 1.0), "bf16")
    Y = kf.gemm_groupnorm(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), groups, 1e-5, to_dev(gamma),
                          to_dev(beta), "swish")
    check_status()
    ref = oracle.gemm_groupnorm(d["X"], d["W"], d["b"], groups, 1e-5, gamma, beta, "swish")
    assert_close(to_f64(Y), ref, 2e-2, 2e-2, "fuzz gemm groupnorm %s g=%d" % (shape, groups))


# ------------------------------------------------------------------ convolution + GroupNorm
def run_conv(kf, d, act="relu", groups=None, gamma=None, beta=None, use_bias=True):
    groups = d["groups"] if groups is None else groups
    y = kf.conv3x3_epilogue(to_dev(d["x"]), to_dev(d["w"]), to_dev(d["bias"]) if use_bias else None,
                            act, groups, d["eps"], to_dev(gamma), to_dev(beta))
    check_status()
    ref = oracle.conv3x3_gn(d["x"], d["w"], d["bias"] if use_bias else None, act, groups, d["eps"],
                            gamma, beta)
    return to_f64(y), ref


@pytest.mark.parametrize("cfg", [
    dict(Nb=2, Cin=64, H=8, W=64, Cout=128, groups=32),      # benchmark geometry, small
    dict(Nb=3, Cin=128, H=16, W=32, Cout=64, groups=4),      # two channel blocks per tap, 4 rows per tile
    dict(Nb=1, Cin=64, H=16, W=8, Cout=256, groups=0),       # 16 rows per tile, widest N tile, no norm
    dict(Nb=2, Cin=64, H=2, W=128, Cout=48, groups=3),       # one row per tile, Cout below the tile width
    dict(Nb=3, Cin=64, H=13, W=64, Cout=96, groups=3),       # NCHW-direct kernel, ragged row units
    dict(Nb=1, Cin=64, H=1, W=64, Cout=128, groups=0),       # NCHW-direct kernel, single row
])
def test_bf16_conv_tensor_core_path(kf, cfg):
    d = ki.conv_inputs(seed=1, **cfg)
    got, ref = run_conv(kf, d)
    assert_close(got, ref, 2e-2, 2e-2, "conv %s" % cfg)


# Any width up to 256 whose rows tile into multiples of 32 pixels, any Cin (padded to 64) and any
# H (the last tile of an image may hang over its end) take the tensor-core convolution too.
@pytest.mark.parametrize("cfg", [
    dict(Nb=2, Cin=64, H=56, W=56, Cout=64, groups=8),       # 4 rows x 56 = 224-pixel tiles
    dict(Nb=2, Cin=128, H=28, W=28, Cout=32, groups=4),      # 8 rows per tile, last tile 4 rows
    dict(Nb=2, Cin=256, H=14, W=14, Cout=256, groups=8),     # planes of 196 pixels: no TMA store
    dict(Nb=1, Cin=3, H=32, W=32, Cout=16, groups=4),        # 3 channels padded to 64
    dict(Nb=2, Cin=32, H=7, W=7, Cout=64, groups=8),         # 32-row box on a 7-row image
    dict(Nb=1, Cin=64, H=5, W=96, Cout=40, groups=5),        # 2 rows per tile, ragged last tile
    dict(Nb=1, Cin=20, H=9, W=24, Cout=24, groups=3),        # padded channels, ragged rows
    dict(Nb=1, Cin=8, H=3, W=224, Cout=8, groups=0),         # one row per tile
    dict(Nb=1, Cin=8, H=4, W=320, Cout=16, groups=2),        # rows cut into two 160-pixel segments
])
def test_bf16_conv_tensor_core_general_shapes(kf, cfg):
    d = ki.conv_inputs(seed=6, **cfg)
    got, ref = run_conv(kf, d)
    assert_close(got, ref, 2e-2, 2e-2, "conv general %s" % cfg)
    got, ref = run_conv(kf, d, act="none", groups=0, use_bias=False)
    assert_close(got, ref, 2e-2, 2e-2, "conv general bare %s" % cfg)


def test_bf16_conv_position_pins(kf):
    """Delta kernels and all-ones inputs: exact results that pin tap orientation and padding."""
    Nb, C, H, W = 2, 64, 8, 64
    r = np.random.default_rng(2)
    xv = r.integers(-32, 33, size=(Nb, C, H, W)) / 32.0
    for (rr, ss) in [(1, 1), (0, 0), (2, 1), (1, 2), (0, 2)]:
        wt = np.zeros((C, C, 3, 3)); wt[np.arange(C), np.arange(C), rr, ss] = 1.0
        d = dict(x=ki.store(xv, "bf16"), w=ki.store(wt, "bf16"), bias=None, groups=0, eps=1e-5)
        got, ref = run_conv(kf, d, act="none", use_bias=False)
        assert_close(got, ref, 0.0, 0.0, "delta tap (%d,%d)" % (rr, ss))
    d = dict(x=ki.store(np.ones((1, C, H, W)), "bf16"), w=ki.store(np.ones((16, C, 3, 3)), "bf16"),
             bias=None, groups=0, eps=1e-5)
    got, _ = run_conv(kf, d, act="none", use_bias=False)
    assert got[0, 0, 3, 5] == 9 * C and got[0, 3, 0, 5] == 6 * C and got[0, 15, H - 1, W - 1] == 4 * C


def test_bf16_conv_groupnorm_moments_and_affine(kf):
    d = ki.conv_inputs(seed=3, Nb=2, Cin=64, H=16, W=64, Cout=128, groups=32)
    got, ref = run_conv(kf, d)
    blk = got.reshape(2, 32, -1)
    assert np.abs(blk.mean(axis=2)).max() < 2e-3
    assert np.abs(blk.var(axis=2) - 1.0).max() < 1e-2
    gamma = ki.store(ki.uniform(3, 7, (128,), 0.5, 1.5), "bf16")
    beta = ki.store(ki.uniform(3, 8, (128,), -1.0, 1.0), "bf16")
    got, ref = run_conv(kf, d, gamma=gamma, beta=beta)
    assert_close(got, ref, 2e-2, 2e-2, "affine")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("cfg", [dict(Nb=1, Cin=2, H=1, W=1, Cout=4, groups=2),
                                 dict(Nb=2, Cin=3, H=5, W=7, Cout=6, groups=3),
                                 dict(Nb=2, Cin=4, H=9, W=4, Cout=8, groups=0)])
def test_conv_scalar_path(kf, dtype, cfg):
    d = ki.conv_inputs(seed=4, dtype=dtype, **cfg)
    got, ref = run_conv(kf, d)
    atol, rtol = tol_for(dtype)      # fp32 with GroupNorm: measured worst err/limit 0.003
    assert_close(got, ref, atol, rtol, "conv scalar %s %s" % (dtype, cfg))


# fp32 convolutions of at least 2^24 multiply-adds per tap take the tensor cores (3xTF32 implicit
# GEMM, chunked accumulation), GroupNorm by the two-pass kernel afterwards.
@pytest.mark.parametrize("cfg", [
    dict(Nb=8, Cin=32, H=32, W=32, Cout=64, groups=8),        # 8 rows x 32 pixels per tile
    dict(Nb=16, Cin=20, H=28, W=28, Cout=72, groups=4),       # channels padded to 32, ragged last tile
    dict(Nb=32, Cin=64, H=14, W=14, Cout=48, groups=0),       # 16-row box on a 14-row image
    dict(Nb=8, Cin=256, H=7, W=7, Cout=256, groups=8),        # planes of 49 pixels: scalar stores; K = 2304, five chunks
    dict(Nb=2, Cin=64, H=64, W=64, Cout=130, groups=0),       # two channel tiles, the second nearly empty
])
def test_fp32_conv_tensor_core_path(kf, cfg):
    d = ki.conv_inputs(seed=8, dtype="f32", **cfg)
    assert kf.kf_conv3x3_workspace_bytes(cfg["Nb"], cfg["Cin"], cfg["H"], cfg["W"], cfg["Cout"], kf.KF_F32,
                                         cfg["groups"]) > 0
    got, ref = run_conv(kf, d)
    assert_close(got, ref, 1e-4, 1e-4, "fp32 conv %s" % cfg)     # with GroupNorm: measured worst err/limit 0.14
    got, ref = run_conv(kf, d, act="none", groups=0, use_bias=False)
    assert_close(got, ref, 1e-4, 1e-4, "fp32 conv bare %s" % cfg)
    assert np.abs(got - ref).max() < 3e-5


def test_groupnorm_biased_variance_on_gpu(kf):
    # 1x1 image, four channels per group, x = 0 so the activations are the biases {1,2,3,4}/4
    bias = np.array([0.25, 0.5, 0.75, 1.0, 2.0, 2.0, 2.0, 2.0], np.float32)
    d = dict(x=np.zeros((1, 2, 1, 1), np.float32), w=np.zeros((8, 2, 3, 3), np.float32), bias=bias,
             groups=2, eps=0.0)
    got, ref = run_conv(kf, d)
    v = np.array([0.25, 0.5, 0.75, 1.0])
    assert_close(got[0, :4, 0, 0], (v - 0.625) / math.sqrt(5.0 / 64), 1e-5, 1e-5, "biased variance")
    d["eps"] = 1e-5
    got, _ = run_conv(kf, d)
    assert (got[0, 4:, 0, 0] == 0).all()


# GroupNorm finished inside the convolution kernel: the CTAs holding one image's 2, 4, 8 or 16 pixel
# tiles form a cluster and exchange the group statistics through distributed shared memory
# (bf16, Cout <= 128, groups of 4..32 channels).
@pytest.mark.parametrize("cfg", [
    dict(Nb=3, Cin=64, H=8, W=64, Cout=128, groups=32),      # clusters of 2, groups of 4 channels
    dict(Nb=2, Cin=32, H=28, W=28, Cout=96, groups=12),      # clusters of 4, ragged last tile, 96 of 128 channel rows
    dict(Nb=2, Cin=16, H=32, W=64, Cout=64, groups=2),       # clusters of 8, groups of 32 channels
    dict(Nb=9, Cin=64, H=64, W=64, Cout=128, groups=8),      # clusters of 16, more images than resident clusters
    dict(Nb=4, Cin=64, H=16, W=16, Cout=256, groups=32),     # one tile per image and channel tile: no peers, two channel tiles
    dict(Nb=3, Cin=32, H=14, W=14, Cout=160, groups=5),      # the same with a ragged second channel tile, groups of 32
    dict(Nb=3, Cin=16, H=28, W=40, Cout=64, groups=8),       # clusters of 7 (four rows of 40 pixels per tile)
    dict(Nb=4, Cin=16, H=6, W=96, Cout=32, groups=8),        # clusters of 3
])
def test_conv_groupnorm_cluster_kernel(kf, cfg, tuning):
    d = ki.conv_inputs(seed=21, dtype="bf16", **cfg)
    gamma = ki.store(ki.uniform(21, 7, (cfg["Cout"],), 0.5, 1.5), "bf16")
    beta = ki.store(ki.uniform(21, 8, (cfg["Cout"],), -1.0, 1.0), "bf16")
    for act, g_, b_ in (("relu", None, None), ("mish", gamma, beta)):
        got, ref = run_conv(kf, d, act=act, gamma=g_, beta=b_)
        assert_close(got, ref, 2e-2, 2e-2, "conv GN cluster %s %s" % (cfg, act))
    # the two-kernel route on the same inputs: same statistics, activations rounded to bf16
    # before instead of after the normalisation
    fused, _ = run_conv(kf, d)
    tuning.setenv("KF_NO_FUSED_GN", "1")
    two, ref = run_conv(kf, d)
    assert_close(two, ref, 2e-2, 2e-2, "conv GN two kernels %s" % (cfg,))
    assert (np.abs(fused - two) <= 2.0 ** -7 * np.maximum(1.0, np.abs(two))).all()      # two bf16 ulps


# The same chain on every SM (no clusters): the tiles of an image sit on neighbouring CTAs of a
# cooperative grid, the group statistics travel through global memory, the epilogue is pipelined
# one tile ahead.  Normally taken for 9..64 tiles per image on multi-wave problems; the knobs
# force it here on small problems, including images that straddle two rounds of the schedule.
@pytest.mark.parametrize("cfg", [
    dict(Nb=3, Cin=64, H=64, W=64, Cout=128, groups=32),     # 16 tiles per image, benchmark geometry
    dict(Nb=11, Cin=32, H=56, W=56, Cout=64, groups=8),      # 14 tiles of 224 pixels, ragged channel rows, 154 tiles: 2 rounds
    dict(Nb=2, Cin=16, H=128, W=128, Cout=64, groups=4),     # 64 tiles per image
    dict(Nb=40, Cin=16, H=16, W=16, Cout=160, groups=5),     # one tile per image, two channel tiles (the second ragged)
    dict(Nb=5, Cin=16, H=30, W=40, Cout=32, groups=8),       # 8 tiles, the last one hangs over the image's end
    dict(Nb=2, Cin=64, H=8, W=64, Cout=128, groups=32),      # fewer tiles than CTAs: one tile each
])
def test_conv_groupnorm_all_sm_kernel(kf, cfg, tuning):
    d = ki.conv_inputs(seed=23, dtype="bf16", **cfg)
    gamma = ki.store(ki.uniform(23, 7, (cfg["Cout"],), 0.5, 1.5), "bf16")
    beta = ki.store(ki.uniform(23, 8, (cfg["Cout"],), -1.0, 1.0), "bf16")
    tuning.setenv("KF_GNX_MIN_TILES", "1")
    tuning.setenv("KF_GNX_MIN_TPI", "1")
    before = kf.kf_launch_count()
    for act, g_, b_ in (("relu", None, None), ("mish", gamma, beta)):
        got, ref = run_conv(kf, d, act=act, gamma=g_, beta=b_)
        assert_close(got, ref, 2e-2, 2e-2, "conv GN all SMs %s %s" % (cfg, act))
    assert kf.kf_launch_count() - before == 4               # prepass + one kernel per call: the route was taken
    again, _ = run_conv(kf, d, act="mish", gamma=gamma, beta=beta)
    assert (again == got).all()                              # fixed summation order: repeat runs are bit-identical
    # whole shares leave in 64-pixel slabs where the mainloop's mode frees a tensor map for them;
    # the 32-pixel form stores the same bits
    tuning.setenv("KF_NO_WIDE_STORE", "1")
    narrow, _ = run_conv(kf, d, act="mish", gamma=gamma, beta=beta)
    assert (narrow == got).all()
    tuning.delenv("KF_NO_WIDE_STORE")
    # the two-kernel route on the same inputs: same statistics, activations rounded to bf16
    # before instead of after the normalisation
    fused, _ = run_conv(kf, d)
    tuning.setenv("KF_NO_FUSED_GN", "1")
    two, ref = run_conv(kf, d)
    assert (np.abs(fused - two) <= 2.0 ** -7 * np.maximum(1.0, np.abs(two))).all()      # two bf16 ulps


def _gnx_fuzz_cases():
    # seeded shapes the all-SM kernel accepts when forced: widths whose tiles are whole 32-pixel
    # pieces, groups of 4 / 8 / 16 / 32 channels, any number of rows, images and channel tiles
    rng = np.random.default_rng(20261125)
    cases = []
    while len(cases) < 10:
        W = int(rng.choice([16, 32, 64, 128, 8, 24, 40, 56]))
        H = int(rng.integers(3, 41))
        Cin = int(rng.choice([16, 32, 64, 128]))
        cpg = int(rng.choice([4, 8, 16, 32]))
        groups = int(rng.integers(1, 9))
        Cout = cpg * groups
        Nb = int(rng.integers(1, 8))
        if Nb * H * W * Cout * Cin * 9 > 3e8:
            continue
        cases.append(dict(Nb=Nb, Cin=Cin, H=H, W=W, Cout=Cout, groups=groups))
    return cases


@pytest.mark.parametrize("cfg", _gnx_fuzz_cases())
def test_conv_groupnorm_all_sm_kernel_seeded_shapes(kf, cfg, tuning):
    d = ki.conv_inputs(seed=41, dtype="bf16", **cfg)
    tuning.setenv("KF_GNX_MIN_TILES", "1")
    tuning.setenv("KF_GNX_MIN_TPI", "1")
    got, ref = run_conv(kf, d, act="swish")
    assert_close(got, ref, 2e-2, 2e-2, "conv GN all SMs, seeded shape %s" % (cfg,))
    # the other routes (cluster or two kernels) on the same inputs agree to two bf16 ulps
    tuning.setenv("KF_NO_GNX", "1")
    other, _ = run_conv(kf, d, act="swish")
    assert (np.abs(got - other) <= 2.0 ** -7 * np.maximum(1.0, np.abs(other))).all()


# ------------------------------------------------------------------ conv -> activation -> global average pool
@pytest.mark.parametrize("dtype,cfg", [
    ("bf16", dict(Nb=2, Cin=64, H=8, W=64, Cout=128)),      # means from the tensor-core epilogue
    ("bf16", dict(Nb=3, Cin=64, H=13, W=64, Cout=96)),      # ragged last tile: its empty rows must not count
    ("bf16", dict(Nb=2, Cin=128, H=28, W=28, Cout=32)),     # 8-row tiles, padded box
    ("bf16", dict(Nb=2, Cin=8, H=6, W=30, Cout=16)),        # width without a tiling: direct conv + plane means
    ("f32", dict(Nb=8, Cin=32, H=32, W=32, Cout=64)),       # fp32 tensor-core conv + plane means
    ("f32", dict(Nb=2, Cin=3, H=5, W=7, Cout=6)),           # fp32 direct conv
])
@pytest.mark.parametrize("act", ["relu", "mish"])
def test_conv_act_global_average_pool(kf, dtype, cfg, act):
    d = ki.conv_inputs(seed=14, dtype=dtype, groups=0, **cfg)
    out = kf.conv3x3_act_gap(to_dev(d["x"]), to_dev(d["w"]), to_dev(d["bias"]), act)
    check_status()
    assert tuple(out.shape) == (cfg["Nb"], cfg["Cout"]) and str(out.dtype) == "torch.float32"
    ref = oracle.conv3x3_act_gap(d["x"], d["w"], d["bias"], act)
    atol, rtol = tol_for(dtype)
    assert_close(to_f64(out), ref, atol, rtol, "conv gap %s %s %s" % (dtype, cfg, act))
    # a mean of hundreds of terms: far tighter than the elementwise tolerance (bf16 planes that
    # are stored first carry their rounding, 2^-9 relative per term, averaged)
    assert np.abs(to_f64(out) - ref).max() < (2e-3 if dtype == "bf16" else 2e-5)


# ------------------------------------------------------------------ conv -> channel softmax -> max-pool
def run_conv_softmax_pool(kf, d, pool, use_bias=True):
    bias = d["bias"] if use_bias else None
    y = kf.conv3x3_softmax_pool(to_dev(d["x"]), to_dev(d["w"]), to_dev(bias), pool)
    check_status()
    return to_f64(y), oracle.conv3x3_softmax_pool(d["x"], d["w"], bias, pool)


@pytest.mark.parametrize("pool", [1, 2, 4])
@pytest.mark.parametrize("cfg", [
    dict(Nb=2, Cin=64, H=8, W=64, Cout=128),       # tensor-core convolution, benchmark geometry
    dict(Nb=1, Cin=64, H=13, W=64, Cout=96),       # ragged rows: 13 = 3*4 + 1, the rim is dropped
    dict(Nb=3, Cin=128, H=16, W=32, Cout=16),      # the case study's 16 output channels
])
def test_bf16_conv_softmax_pool(kf, cfg, pool):
    d = ki.conv_inputs(seed=11, groups=0, **cfg)
    got, ref = run_conv_softmax_pool(kf, d, pool)
    assert got.shape == (cfg["Nb"], cfg["Cout"], cfg["H"] // pool, cfg["W"] // pool)
    assert_close(got, ref, 2e-2, 2e-2, "conv softmax pool %s pool %d" % (cfg, pool))
    # probabilities are ~1/Cout, far below the absolute tolerance: gate them relatively as well
    # (bf16 staging of the logits and of the result, 2^-9 each)
    assert_close(got, ref, 1e-6, 2e-2, "relative gate %s pool %d" % (cfg, pool))


def test_bf16_conv_softmax_pool_peaked(kf):
    """Weights x16 make the softmax peaked: winners near 1 and losers near 0 in one image."""
    d = ki.conv_inputs(seed=12, Nb=2, Cin=64, H=8, W=64, Cout=32, groups=0)
    d["w"] = ki.store(ki.widen(d["w"]) * 16.0, "bf16")        # exact: a power of two
    got, ref = run_conv_softmax_pool(kf, d, 2)
    assert ref.max() > 0.9 and ref.min() < 1e-3
    assert_close(got, ref, 2e-2, 2e-2, "peaked softmax, official tolerance")
    # The logits are staged in bf16: each carries a relative rounding of 2^-9, so a probability
    # (a ratio of exponentials of two logits) moves by up to 2 * 2^-9 * max|logit| relatively,
    # plus 2^-9 for its own rounding.
    zmax = np.abs(oracle.conv3x3_gn(d["x"], d["w"], d["bias"], "none", 0)).max()
    assert_close(got, ref, 1e-6, 2.0 ** -8 * (zmax + 1.0), "peaked softmax, derived relative gate")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("cfg,pool", [(dict(Nb=2, Cin=3, H=5, W=7, Cout=6), 2),
                                      (dict(Nb=1, Cin=2, H=4, W=9, Cout=1), 3),
                                      (dict(Nb=2, Cin=4, H=9, W=4, Cout=8), 1),
                                      (dict(Nb=1, Cin=2, H=3, W=3, Cout=5), 4),    # empty result
                                      (dict(Nb=1, Cin=2, H=4, W=200, Cout=64), 2),  # two column tiles, ragged
                                      (dict(Nb=1, Cin=1, H=4, W=8, Cout=2100), 4)])  # strip too big for smem
def test_conv_softmax_pool_scalar_path(kf, dtype, cfg, pool):
    d = ki.conv_inputs(seed=13, dtype=dtype, groups=0, **cfg)
    got, ref = run_conv_softmax_pool(kf, d, pool, use_bias=(cfg["Cout"] != 8))
    atol, rtol = tol_for(dtype)
    assert_close(got, ref, atol, rtol, "scalar conv softmax pool %s %s" % (dtype, cfg))
    if dtype == "f32":
        assert_close(got, ref, 1e-7, 1e-4, "relative gate")
    if cfg["Cout"] == 1 and got.size:
        assert (got == 1.0).all()          # one channel: every probability is exactly 1


def test_conv_softmax_pool_errors(kf):
    import torch
    x = torch.zeros((1, 2, 8, 8), device="cuda"); w = torch.zeros((2, 2, 3, 3), device="cuda")
    with pytest.raises(kf.KfError) as e:
        kf.conv3x3_softmax_pool(x, w, None, 5)
    assert e.value.status == kf.KF_ERR_UNSUPPORTED
    with pytest.raises(kf.KfError) as e:
        kf.conv3x3_softmax_pool(x, w, None, 0)
    assert e.value.status == kf.KF_ERR_INVALID_ARG


# ------------------------------------------------------------------ bounded waits
def test_bounded_wait_gives_up_and_is_reported(kf):
    """A wait nothing satisfies returns after its limit, raises the device status word, and the
    context stays usable (no trap, no fault, no unbounded loop)."""
    assert kf.kf_device_status() == kf.KF_OK
    st, waited = kf.kf_selftest_bounded_wait(2_000_000)          # 2 ms
    assert st == kf.KF_OK
    assert 2_000_000 <= waited < 200_000_000
    assert kf.kf_device_status() == kf.KF_ERR_TIMEOUT            # reported once ...
    assert kf.kf_device_status() == kf.KF_OK                     # ... and cleared
    assert kf.kf_selftest_bounded_wait(10)[0] == kf.KF_ERR_INVALID_ARG
    assert kf.kf_selftest_bounded_wait(2_000_000_000)[0] == kf.KF_ERR_INVALID_ARG
    # the library still computes afterwards
    d = ki.gemm_inputs("c2", seed=71, M=128, N=64, K=64)
    got, ref = run_gemm(kf, d, "relu")
    assert_close(got, ref, 2e-2, 2e-2, "after the self-test")


# ------------------------------------------------------------------ error handling on the device box
def test_workspace_errors(kf):
    import torch
    d = ki.gemm_inputs("c3", seed=1, M=128, N=512, K=64)
    X, W = to_dev(d["X"]), to_dev(d["W"])
    out = torch.empty(128, 512, dtype=torch.bfloat16, device="cuda")
    before = kf.kf_launch_count()
    st = kf.kf_gemm_rowreduce(128, 512, 64, kf.KF_BF16, X.data_ptr(), 64, W.data_ptr(), 64, None, 0, 0,
                              out.data_ptr(), 512, kf.KF_BF16, None, 0, None)
    assert st == kf.KF_ERR_WORKSPACE
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    st = kf.kf_gemm_rowreduce(128, 512, 64, kf.KF_BF16, X.data_ptr(), 64, W.data_ptr(), 64, None, 0, 0,
                              out.data_ptr(), 512, kf.KF_BF16, ws.data_ptr() + 8, 4088, None)
    assert st == kf.KF_ERR_WORKSPACE
    assert kf.kf_launch_count() == before
    with pytest.raises(kf.KfError):
        kf.gemm_epilogue(X, W, act="none", out=X)


def test_calls_on_a_side_stream(kf):
    import torch
    d = ki.gemm_inputs("c2", seed=9, M=256, N=256, K=128)
    s = torch.cuda.Stream()
    X, W, b, R = to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), to_dev(d["R"])
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        Y = kf.gemm_epilogue(X, W, b, "gelu_tanh", 0.5, R, stream=s)
    s.synchronize()
    ref = oracle.gemm_epilogue(d["X"], d["W"], d["b"], "gelu_tanh", 0.5, d["R"])
    assert_close(to_f64(Y), ref, 2e-2, 2e-2, "side stream")


# ------------------------------------------------------------------ conv -> activation -> max / average pool
@pytest.mark.parametrize("dtype,cfg,pool", [
    ("bf16", dict(Nb=2, Cin=64, H=8, W=64, Cout=128), 2),     # pooled in the epilogue: 4-row tiles
    ("bf16", dict(Nb=3, Cin=32, H=14, W=32, Cout=72), 2),     # 8-row tiles, last tile holds 6 rows; ragged channels
    ("bf16", dict(Nb=2, Cin=16, H=6, W=96, Cout=130), 2),     # 2-row tiles of 192 pixels; second channel tile nearly empty
    ("bf16", dict(Nb=2, Cin=64, H=4, W=128, Cout=64), 2),     # 2-row tiles of 256 pixels
    ("bf16", dict(Nb=2, Cin=64, H=4, W=256, Cout=64), 2),     # one row per tile: conv, then the pooling kernel
    ("bf16", dict(Nb=2, Cin=64, H=9, W=64, Cout=32), 2),      # odd H: last row dropped; two passes
    ("bf16", dict(Nb=2, Cin=64, H=8, W=64, Cout=32), 3),      # pool 3 with a ragged rim
    ("bf16", dict(Nb=2, Cin=8, H=7, W=30, Cout=16), 2),       # direct convolution + pooling kernel
    ("bf16", dict(Nb=1, Cin=8, H=8, W=32, Cout=16), 4),
    ("f32", dict(Nb=8, Cin=32, H=32, W=32, Cout=64), 2),      # fp32 tensor-core conv + pooling kernel
    ("f32", dict(Nb=2, Cin=3, H=5, W=7, Cout=6), 2),          # fp32 direct conv
    ("f32", dict(Nb=2, Cin=3, H=5, W=7, Cout=6), 1),          # pool 1: the activations themselves
])
@pytest.mark.parametrize("kind", ["max", "avg"])
def test_conv_act_pool(kf, dtype, cfg, pool, kind):
    d = ki.conv_inputs(seed=16, dtype=dtype, groups=0, **cfg)
    for act in ("relu", "tanh"):          # tanh is not monotone-free of sign: pooling after, not before
        out = kf.conv3x3_act_pool(to_dev(d["x"]), to_dev(d["w"]), to_dev(d["bias"]), act, kind, pool)
        check_status()
        assert tuple(out.shape) == (cfg["Nb"], cfg["Cout"], cfg["H"] // pool, cfg["W"] // pool)
        ref = oracle.conv3x3_act_pool(d["x"], d["w"], d["bias"], act, kind, pool)
        atol, rtol = tol_for(dtype)
        assert_close(to_f64(out), ref, atol, rtol, "conv pool %s %s %s %d %s" % (dtype, cfg, kind, pool, act))


def test_conv_act_pool_fused_and_two_pass_agree(kf, tuning):
    """The pooling in the convolution's epilogue and the two-kernel route see the same fp32
    activations; the two-kernel route rounds them to bf16 before pooling, so max pooling (which
    commutes with the monotone rounding) must agree bit for bit."""
    import torch
    cfg = dict(Nb=2, Cin=64, H=16, W=64, Cout=96)
    d = ki.conv_inputs(seed=17, dtype="bf16", groups=0, **cfg)
    args = (to_dev(d["x"]), to_dev(d["w"]), to_dev(d["bias"]), "swish", "max", 2)
    assert kf.kf_conv3x3_act_pool_workspace_bytes(2, 64, 16, 64, 96, kf.KF_BF16, 2) == \
        kf.kf_conv3x3_workspace_bytes(2, 64, 16, 64, 96, kf.KF_BF16, 0)
    fused = kf.conv3x3_act_pool(*args).clone()
    tuning.setenv("KF_NO_FUSED_POOL", "1")
    two = kf.conv3x3_act_pool(*args)
    torch.cuda.synchronize()
    assert torch.equal(fused, two)
    check_status()


def test_conv_act_pool_unaligned_output_and_empty(kf):
    import torch
    cfg = dict(Nb=1, Cin=16, H=4, W=32, Cout=8)
    d = ki.conv_inputs(seed=18, dtype="bf16", groups=0, **cfg)
    buf = torch.zeros(1 + 8 * 2 * 16 + 1, dtype=torch.bfloat16, device="cuda")
    out = buf[1:-1].view(1, 8, 2, 16)                     # 2-byte aligned only
    kf.conv3x3_act_pool(to_dev(d["x"]), to_dev(d["w"]), to_dev(d["bias"]), "relu", "avg", 2, out=out)
    check_status()
    ref = oracle.conv3x3_act_pool(d["x"], d["w"], d["bias"], "relu", "avg", 2)
    assert_close(to_f64(out), ref, 2e-2, 2e-2, "unaligned pooled output")
    assert float(buf[0]) == 0.0 and float(buf[-1]) == 0.0
    empty = kf.conv3x3_act_pool(to_dev(d["x"]), to_dev(d["w"]), None, "relu", "max", 5)
    assert tuple(empty.shape) == (1, 8, 0, 6)
    with pytest.raises(kf.KfError):
        kf.conv3x3_act_pool(to_dev(d["x"]), to_dev(d["w"]), None, "relu", "max", 0)


def test_host_front_end_matches_device_call(kf):
    """gemm_epilogue_host (chunked copies on side streams) gives the same bits as one device call."""
    import torch
    d = ki.gemm_inputs("c2", seed=10, M=1300, N=264, K=128)
    pin = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    hX, hW, hb, hR = pin(d["X"]), pin(d["W"]), pin(d["b"]), pin(d["R"])
    out = torch.zeros(1300, 264, dtype=torch.bfloat16).pin_memory()
    kf.gemm_epilogue_host(hX, hW, hb, "gelu_tanh", 0.5, hR, out_host=out)
    torch.cuda.synchronize()
    ref = kf.gemm_epilogue(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "gelu_tanh", 0.5, to_dev(d["R"]))
    assert torch.equal(out, ref.cpu())
    check_status()


def test_host_front_end_back_to_back_calls(kf):
    """Consecutive host calls share staging buffers and overlap (the next call's uploads run
    while the previous call's downloads finish): every call must still see its own inputs."""
    import torch
    M, N, K = 2048, 512, 256
    pin = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    sets, outs = [], []
    for seed in (20, 21, 22, 23):
        d = ki.gemm_inputs("c2", seed=seed, M=M, N=N, K=K)
        sets.append((d, pin(d["X"]), pin(d["W"]), pin(d["b"]), pin(d["R"])))
        outs.append(torch.zeros(M, N, dtype=torch.bfloat16).pin_memory())
    for (d, hX, hW, hb, hR), out in zip(sets, outs):            # no synchronisation in between
        kf.gemm_epilogue_host(hX, hW, hb, "gelu_tanh", 0.5, hR, out_host=out)
    torch.cuda.synchronize()
    for (d, hX, hW, hb, hR), out in zip(sets, outs):
        ref = kf.gemm_epilogue(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "gelu_tanh", 0.5, to_dev(d["R"]))
        assert torch.equal(out, ref.cpu())
    check_status()


# ------------------------------------------------------------------ host-buffer entry point
@pytest.mark.parametrize("blocks", [1, 4])
def test_gemm_epilogue_host_buffers_through_the_c_abi(kf, blocks):
    """kf_gemm_epilogue_host: pinned host tensors in, host tensor out, pitched rows, two calls in a
    row on the same staging buffer (the second call's uploads must wait for the first call's
    kernels); against the oracle and bit for bit against the device-buffer entry point."""
    import torch
    M, N, K = 1024, 320, 136
    d = ki.gemm_inputs("c2", seed=21, M=M, N=N, K=K)
    hX = torch.zeros(M, K + 8, dtype=torch.bfloat16).pin_memory()
    hX[:, :K] = torch.from_numpy(d["X"].view(np.int16)).view(torch.bfloat16)
    hW = torch.from_numpy(d["W"].view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    hb = torch.from_numpy(d["b"].view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    hR = torch.from_numpy(d["R"].view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    ref = oracle.gemm_epilogue(d["X"], d["W"], d["b"], "gelu_tanh", 0.5, d["R"])
    dev = kf.gemm_epilogue(to_dev(d["X"]), to_dev(d["W"]), to_dev(d["b"]), "gelu_tanh", 0.5, to_dev(d["R"]))
    for rep in range(2):
        hY = torch.zeros(M, N, dtype=torch.bfloat16).pin_memory()
        kf.gemm_epilogue_host(hX[:, :K], hW, hb, "gelu_tanh", 0.5, hR, out_host=hY, chunks=blocks)
        torch.cuda.synchronize()
        check_status()
        assert_close(hY.float().numpy().astype(np.float64), ref, 2e-2, 2e-2, "host buffers, call %d" % rep)
        assert torch.equal(hY, dev.cpu())


# ------------------------------------------------------------------ workspace queries for any operands
def test_workspace_queries_for_unaligned_operands_cover_the_call(kf):
    """Operands TMA cannot load (an odd pitch, a base off 16 bytes) take other routes with other
    workspace needs: the *_for queries, given the call's own pointers and pitches, must return
    enough for the call to succeed, through the raw C ABI."""
    import torch
    M, N, K = 96, 80, 72
    d = ki.gemm_inputs("c3", seed=31, M=M, N=N, K=K)
    Xb = torch.zeros(M * (K + 3) + 1, dtype=torch.bfloat16, device="cuda")
    X = Xb[1:].view(M, K + 3)[:, :K]                     # base off 16 bytes, pitch 75
    X.copy_(to_dev(d["X"]))
    W, b = to_dev(d["W"]), to_dev(d["b"])
    Y = torch.empty(M, N + 1, dtype=torch.bfloat16, device="cuda")[:, :N]     # pitch 81
    stream = torch.cuda.current_stream().cuda_stream
    L = kf.lib()

    def ws_for(nbytes):
        return (torch.empty(max(nbytes, 1), dtype=torch.uint8, device="cuda"), nbytes)

    nb = L.kf_gemm_epilogue_workspace_bytes_for(M, N, K, kf.KF_BF16, X.data_ptr(), X.stride(0), W.data_ptr(), K)
    ws, nb = ws_for(nb)
    st = kf.kf_gemm_epilogue(M, N, K, kf.KF_BF16, X.data_ptr(), X.stride(0), W.data_ptr(), K, b.data_ptr(),
                             kf.ACT["relu"], 1.0, None, 0, Y.data_ptr(), Y.stride(0), ws.data_ptr() if nb else None,
                             nb, stream)
    assert st == kf.KF_OK, kf.status_string(st)
    assert_close(to_f64(Y), oracle.gemm_epilogue(d["X"], d["W"], d["b"], "relu"), 2e-2, 2e-2, "epilogue, odd pitch")

    for red, name in ((kf.RED["softmax"], "softmax"), (kf.RED["sum"], "sum")):
        assert kf.kf_gemm_rowreduce_workspace_bytes(M, N, K, kf.KF_BF16, red) < M * N * 4     # the short form is not enough
        nb = L.kf_gemm_rowreduce_workspace_bytes_for(M, N, K, kf.KF_BF16, red, X.data_ptr(), X.stride(0),
                                                     W.data_ptr(), K)
        assert nb >= M * N * 4
        ws, nb = ws_for(nb)
        out = (torch.empty(M, N, dtype=torch.bfloat16, device="cuda") if name == "softmax"
               else torch.empty(M, dtype=torch.float32, device="cuda"))
        st = kf.kf_gemm_rowreduce(M, N, K, kf.KF_BF16, X.data_ptr(), X.stride(0), W.data_ptr(), K, b.data_ptr(),
                                  kf.ACT["none"], red, out.data_ptr(), N if name == "softmax" else 1,
                                  kf.KF_BF16 if name == "softmax" else kf.KF_F32, ws.data_ptr(), nb, stream)
        assert st == kf.KF_OK, kf.status_string(st)
        ref = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", name).reshape(to_f64(out).shape)
        assert_close(to_f64(out), ref, 2e-2, 2e-2, "rowreduce %s, odd pitch" % name)

    groups = 5                                           # 16 columns per group: the scalar route in any case
    assert kf.kf_gemm_groupnorm_workspace_bytes(M, N, K, kf.KF_BF16, 2) >= 0
    nb = L.kf_gemm_groupnorm_workspace_bytes_for(M, N, K, kf.KF_BF16, groups, X.data_ptr(), X.stride(0),
                                                 W.data_ptr(), K, Y.data_ptr(), Y.stride(0))
    ws, nb = ws_for(nb)
    st = kf.kf_gemm_groupnorm(M, N, K, kf.KF_BF16, X.data_ptr(), X.stride(0), W.data_ptr(), K, b.data_ptr(), groups,
                              1e-5, None, None, kf.ACT["none"], Y.data_ptr(), Y.stride(0),
                              ws.data_ptr() if nb else None, nb, stream)
    assert st == kf.KF_OK, kf.status_string(st)
    check_status()
    assert_close(to_f64(Y), oracle.gemm_groupnorm(d["X"], d["W"], d["b"], groups, 1e-5, None, None, "none"),
                 2e-2, 2e-2, "groupnorm, odd pitch")
    # a 64-column group with a Y that TMA cannot store to: the short query says 0, the call needs M*N floats
    assert kf.kf_gemm_groupnorm_workspace_bytes(128, 128, 64, kf.KF_BF16, 2) == 0
    Xa = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    Wa = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    Ya = torch.empty(128, 129, dtype=torch.bfloat16, device="cuda")[:, :128]
    nb = L.kf_gemm_groupnorm_workspace_bytes_for(128, 128, 64, kf.KF_BF16, 2, Xa.data_ptr(), 64, Wa.data_ptr(), 64,
                                                 Ya.data_ptr(), 129)
    assert nb >= 128 * 128 * 4
