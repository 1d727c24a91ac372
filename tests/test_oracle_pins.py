"""Pins for the fp64 CPU oracle: closed forms, invariants, library special cases and exact
brute force.  None of these re-types the oracle's own loops: each expected value comes from
mathematics (an identity, a closed form), from a library routine the oracle does not call
(numpy matmul, scipy softmax / correlate2d / normal CDF), or from exact rational arithmetic.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.signal
import scipy.special
import scipy.stats

import kf_inputs as ki
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


def f32(a):
    return np.asarray(a, dtype=np.float32)


def bf(a):
    return ki.to_bf16_bits(np.asarray(a, dtype=np.float64))


def rng_small(shape, seed, dtype):
    """Small-integer-over-power-of-two values: exactly representable in bf16 and fp32."""
    r = np.random.default_rng(seed)
    v = r.integers(-8, 9, size=shape).astype(np.float64) / 8.0
    return ki.store(v, dtype)


# ------------------------------------------------------------------ activations
def test_activation_fixed_points():
    a = oracle.act
    assert a("relu", -1.0) == 0.0 and a("relu", 2.0) == 2.0 and a("relu", 0.0) == 0.0
    assert a("none", -3.25) == -3.25
    assert a("sigmoid", 0.0) == 0.5
    assert abs(a("sigmoid", math.log(3.0)) - 0.75) < 1e-15
    assert abs(a("sigmoid", -math.log(3.0)) - 0.25) < 1e-15
    assert a("sigmoid", 40.0) <= 1.0 and a("sigmoid", -40.0) >= 0.0
    assert not math.isnan(a("sigmoid", 800.0)) and not math.isnan(a("sigmoid", -800.0))
    assert a("gelu_tanh", 0.0) == 0.0 and a("gelu_erf", 0.0) == 0.0
    assert abs(a("gelu_tanh", 10.0) - 10.0) < 1e-12 and abs(a("gelu_tanh", -10.0)) < 1e-12
    assert a("hardtanh", 3.0) == 1.0 and a("hardtanh", -3.0) == -1.0 and a("hardtanh", 0.3) == 0.3
    assert a("tanh", 0.0) == 0.0 and abs(a("tanh", 0.5) - math.tanh(0.5)) < 1e-16
    assert a("swish", 0.0) == 0.0 and abs(a("swish", math.log(3.0)) - 0.75 * math.log(3.0)) < 1e-15


@pytest.mark.parametrize("z", [-6.0, -3.0, -1.0, -0.3, 0.2, 1.0, 2.0, 4.5])
def test_gelu_identities(z):
    gt, ge = oracle.act("gelu_tanh", z), oracle.act("gelu_erf", z)
    # erf-GELU is z * Phi(z): the normal CDF from a library the oracle does not use.
    assert abs(ge - z * scipy.stats.norm.cdf(z)) < 1e-14
    # tanh is odd, so gelu_tanh(z) - gelu_tanh(-z) = z exactly.
    assert abs(gt - oracle.act("gelu_tanh", -z) - z) < 1e-14
    # (1+tanh u)/2 = sigmoid(2u): the same function through a different elementary route.
    u = math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)
    assert abs(gt - z / (1.0 + math.exp(-2.0 * u))) < 1e-14
    # the tanh form approximates the erf form to within 5e-4 everywhere.
    assert abs(gt - ge) < 5e-4


def test_gelu_variants_are_distinguishable():
    # at z = -3 the two GELUs differ by ~4.1e-4: enough for the fp32 tolerance to tell them apart
    d = abs(oracle.act("gelu_tanh", -3.0) - oracle.act("gelu_erf", -3.0))
    assert 3.5e-4 < d < 4.7e-4


def test_further_activations_against_closed_forms_and_torch():
    """The seven further activations: closed-form values, then torch's own fp64 routines on a
    grid (an independent implementation of the same definitions)."""
    import torch
    import torch.nn.functional as F
    e = math.e
    closed = [("leaky_relu", -2.0, -0.02), ("leaky_relu", 3.0, 3.0), ("elu", -1.0, 1.0 / e - 1.0), ("elu", 2.0, 2.0),
              ("mish", 0.0, 0.0), ("mish", 1.0, 0.86509838826731), ("mish", -1.0, -0.30340146137411),
              ("hardswish", 1.0, 2.0 / 3.0), ("hardswish", -3.0, 0.0), ("hardswish", 3.0, 3.0), ("hardswish", -4.0, 0.0),
              ("softplus", 0.0, math.log(2.0)), ("softplus", 800.0, 800.0), ("softplus", -800.0, 0.0),
              ("relu6", 7.0, 6.0), ("relu6", -1.0, 0.0), ("relu6", 2.5, 2.5),
              ("hardsigmoid", 0.0, 0.5), ("hardsigmoid", 3.0, 1.0), ("hardsigmoid", -3.0, 0.0), ("hardsigmoid", 1.5, 0.75)]
    for name, z, want in closed:
        assert abs(oracle.act(name, z) - want) < (1e-13 if name == "mish" else 1e-14), (name, z)   # mish: 14 printed digits
    lib = {"leaky_relu": F.leaky_relu, "elu": F.elu, "mish": F.mish, "hardswish": F.hardswish,
           "softplus": lambda t: F.softplus(t, threshold=1e9), "relu6": F.relu6, "hardsigmoid": F.hardsigmoid}
    zs = np.linspace(-12.0, 12.0, 481)
    t = torch.from_numpy(zs)
    for name, fn in lib.items():
        want = fn(t).numpy()
        got = np.array([oracle.act(name, float(z)) for z in zs])
        assert np.abs(got - want).max() < 1e-13, name


def test_row_max_mean_logsumexp():
    """The further row reductions against independent routes: the pre-reduction matrix from the
    separately pinned elementwise oracle, reduced by numpy / scipy; and softmax = exp(A - lse)."""
    import scipy.special
    d = ki.gemm_inputs("c3", seed=9, M=7, N=33, K=20, dtype="f32")
    A = oracle.gemm_epilogue(d["X"], d["W"], d["b"], "gelu_tanh")
    mx = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "gelu_tanh", "max")
    mean = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "gelu_tanh", "mean")
    lse = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "gelu_tanh", "logsumexp")
    sm = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "gelu_tanh", "softmax")
    assert mx.shape == mean.shape == lse.shape == (7,)
    assert np.array_equal(mx, A.max(axis=1))
    assert np.abs(mean - A.mean(axis=1)).max() < 1e-15
    assert np.abs(lse - scipy.special.logsumexp(A, axis=1)).max() < 1e-14
    assert np.abs(sm - np.exp(A - lse[:, None])).max() < 1e-15
    # one column: max = mean = logsumexp = the value itself; large values do not overflow
    X = np.zeros((3, 4), np.float32); W = np.zeros((1, 4), np.float32); b = np.array([900.0], np.float32)
    for red in ("max", "mean", "logsumexp"):
        assert np.array_equal(oracle.gemm_rowreduce(X, W, b, "none", red), np.full(3, 900.0))


def test_conv_act_global_average_pool():
    """Global average pooling after the convolution: against the separately pinned convolution
    averaged by numpy, and a closed form (all-ones image and kernel: each output pixel counts
    its in-image taps, 9 inside, 6 on an edge, 4 in a corner)."""
    d = ki.conv_inputs(seed=5, Nb=2, Cin=3, H=5, W=6, Cout=4, groups=0, dtype="f32")
    for act in ("none", "relu", "mish"):
        full = oracle.conv3x3_gn(d["x"], d["w"], d["bias"], act, 0)
        got = oracle.conv3x3_act_gap(d["x"], d["w"], d["bias"], act)
        assert got.shape == (2, 4)
        assert np.abs(got - full.mean(axis=(2, 3))).max() < 1e-15
    H, W, C = 4, 7, 2
    ones = oracle.conv3x3_act_gap(np.ones((1, C, H, W), np.float32), np.ones((3, C, 3, 3), np.float32), None, "none")
    taps = 9 * (H - 2) * (W - 2) + 6 * (2 * (H - 2) + 2 * (W - 2)) + 4 * 4
    assert np.abs(ones - C * taps / (H * W)).max() < 1e-13


def test_gemm_groupnorm_against_torch_and_moments():
    """GroupNorm over column groups of a GEMM output: torch's own fp64 group_norm applied to the
    separately pinned pre-normalisation matrix; unit moments per (row, group); a 2-element group
    closed form ((-1, +1) whatever the two values, as long as they differ)."""
    import torch
    import torch.nn.functional as F
    d = ki.gemm_inputs("c3", seed=11, M=6, N=48, K=20, dtype="f32")
    Z = oracle.gemm_epilogue(d["X"], d["W"], d["b"], "none")
    gamma = ki.store(ki.uniform(11, 7, (48,), 0.5, 1.5), "f32")
    beta = ki.store(ki.uniform(11, 8, (48,), -1.0, 1.0), "f32")
    for groups in (1, 3, 12, 48 // 2):
        want = F.group_norm(torch.from_numpy(Z), groups, torch.from_numpy(gamma.astype(np.float64)),
                            torch.from_numpy(beta.astype(np.float64)), 1e-5).numpy()
        got = oracle.gemm_groupnorm(d["X"], d["W"], d["b"], groups, 1e-5, gamma, beta)
        assert np.abs(got - want).max() < 1e-12, groups
        swish = oracle.gemm_groupnorm(d["X"], d["W"], d["b"], groups, 1e-5, gamma, beta, "swish")
        assert np.abs(swish - want / (1.0 + np.exp(-want))).max() < 1e-12
    plain = oracle.gemm_groupnorm(d["X"], d["W"], d["b"], 4, 0.0).reshape(6, 4, 12)
    assert np.abs(plain.mean(axis=2)).max() < 1e-14
    assert np.abs(plain.var(axis=2) - 1.0).max() < 1e-13
    two = oracle.gemm_groupnorm(d["X"], d["W"], d["b"], 24, 0.0).reshape(6, 24, 2)
    assert np.abs(np.sort(two, axis=2) - np.array([-1.0, 1.0])).max() < 1e-9


def test_conv_act_pool_against_torch_pooling():
    """Spatial pooling after conv + activation: torch's own max_pool2d / avg_pool2d (fp64) applied
    to the separately pinned convolution, ragged rims included; pool 1 is the identity."""
    import torch
    import torch.nn.functional as F
    d = ki.conv_inputs(seed=6, Nb=2, Cin=3, H=7, W=9, Cout=4, groups=0, dtype="f32")
    for act in ("relu", "swish"):
        full = oracle.conv3x3_gn(d["x"], d["w"], d["bias"], act, 0)
        t = torch.from_numpy(full)
        for pool in (1, 2, 3, 4):
            mx = oracle.conv3x3_act_pool(d["x"], d["w"], d["bias"], act, "max", pool)
            av = oracle.conv3x3_act_pool(d["x"], d["w"], d["bias"], act, "avg", pool)
            assert mx.shape == (2, 4, 7 // pool, 9 // pool)
            assert np.array_equal(mx, F.max_pool2d(t, pool).numpy())
            assert np.abs(av - F.avg_pool2d(t, pool).numpy()).max() < 1e-15
        assert np.array_equal(oracle.conv3x3_act_pool(d["x"], d["w"], d["bias"], act, "max", 1), full)


def test_paper_constants_and_chain95():
    g = golden()
    assert abs(g["erf_gelu_inner_scale"] - 1.0 / math.sqrt(2.0)) < 1e-15
    for z in [-5.0, -1.2, -0.1, 0.0, 0.4, 1.7, 6.0, 400.0]:
        s = oracle.act("swish", z)
        t = oracle.act("tanh", s)
        ge = oracle.act("gelu_erf", t)
        want = oracle.act("hardtanh", ge)
        assert abs(oracle.act("chain95", z) - want) < 1e-14
        assert g["hardtanh_lo"] <= oracle.act("chain95", z) <= g["hardtanh_hi"]
    # tanh through exponentials, as the paper's listing writes it
    s = 0.37
    e = math.exp(g["tanh_exp_factor"] * s)
    assert abs((e - 1) / (e + 1) - oracle.act("tanh", s)) < 1e-15


# ------------------------------------------------------------------ GEMM + epilogue
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_onehot_rows_pick_weight_columns(dtype):
    M, N, K = 7, 5, 11
    W = rng_small((N, K), 1, dtype)
    ks = [(3 * m + 2) % K for m in range(M)]
    Xf = np.zeros((M, K)); Xf[np.arange(M), ks] = 1.0
    Y = oracle.gemm_epilogue(ki.store(Xf, dtype), W)
    assert np.array_equal(Y, ki.widen(W)[:, ks].T)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_permutation_weight_permutes_columns(dtype):
    M, N = 6, 9
    X = rng_small((M, N), 2, dtype)
    perm = np.random.default_rng(3).permutation(N)
    Wf = np.zeros((N, N)); Wf[np.arange(N), perm] = 1.0
    Y = oracle.gemm_epilogue(X, ki.store(Wf, dtype))
    assert np.array_equal(Y, ki.widen(X)[:, perm])


def test_identity_weight_and_zero_inputs():
    n = 8
    X = rng_small((5, n), 4, "f32"); b = rng_small((n,), 5, "f32"); R = rng_small((5, n), 6, "f32")
    eye = f32(np.eye(n))
    Y = oracle.gemm_epilogue(X, eye, b, "relu")
    assert np.array_equal(Y, np.maximum(ki.widen(X) + ki.widen(b), 0.0))
    zero = f32(np.zeros((5, n)))
    # X = 0: every row is scale*act(b) + R
    Y = oracle.gemm_epilogue(zero, rng_small((n, n), 7, "f32"), b, "sigmoid", 0.5, R)
    want = 0.5 * scipy.special.expit(ki.widen(b))[None, :] + ki.widen(R)
    assert np.abs(Y - want).max() < 1e-15
    # X = 0, b = 0 with GELU or ReLU: Y = R exactly
    for act in ("gelu_tanh", "relu", "gelu_erf"):
        Y = oracle.gemm_epilogue(zero, eye, f32(np.zeros(n)), act, 0.5, R)
        assert np.array_equal(Y, ki.widen(R))


def test_epilogue_order_bias_act_scale_residual():
    # 1x1x1 problem: z = x*w + b; Y = s*relu(z) + r.  Values chosen so every other order differs.
    x, w, b, s, r = 2.0, -1.5, 1.0, 0.5, 0.25
    Y = oracle.gemm_epilogue(f32([[x]]), f32([[w]]), f32([b]), "relu", s, f32([[r]]))
    assert Y[0, 0] == s * max(x * w + b, 0.0) + r == 0.25
    x = 3.0
    w = 1.0
    Y = oracle.gemm_epilogue(f32([[x]]), f32([[w]]), f32([b]), "relu", s, f32([[r]]))
    assert Y[0, 0] == 0.5 * 4.0 + 0.25


def _exact_z(X, W, b, m, n):
    z = Fraction(0)
    for k in reversed(range(X.shape[1])):          # different order from the oracle on purpose
        z += Fraction(float(X[m, k])) * Fraction(float(W[n, k]))
    if b is not None:
        z += Fraction(float(b[n]))
    return z


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(1, 1, 1), (3, 2, 5), (4, 7, 3), (17, 5, 9), (2, 13, 17)])
def test_gemm_brute_force_exact(dtype, shape):
    M, N, K = shape
    d = ki.gemm_inputs("c1", seed=11, M=M, N=N, K=K, dtype=dtype)
    Xw, Ww, bw = ki.widen(d["X"]), ki.widen(d["W"]), ki.widen(d["b"])
    R = ki.store(ki.normal(11, 9, (M, N)), dtype)
    Y = oracle.gemm_epilogue(d["X"], d["W"], d["b"], "gelu_tanh", 0.5, R)
    Z = oracle.gemm_epilogue(d["X"], d["W"], d["b"])
    for m in range(M):
        for n in range(N):
            z = float(_exact_z(Xw, Ww, bw, m, n))
            assert abs(Z[m, n] - z) <= 1e-13 * (1 + abs(z))
            u = math.sqrt(2 / math.pi) * (z + 0.044715 * z ** 3)
            want = 0.5 * (z / (1.0 + math.exp(-2.0 * u))) + float(ki.widen(R)[m, n])
            assert abs(Y[m, n] - want) <= 1e-13 * (1 + abs(want))


def test_gemm_matches_library_matmul():
    d = ki.gemm_inputs("c1", seed=0)
    Y = oracle.gemm_epilogue(d["X"], d["W"], d["b"], "relu")
    want = np.maximum(ki.widen(d["X"]) @ ki.widen(d["W"]).T + ki.widen(d["b"]), 0.0)
    assert np.abs(Y - want).max() < 1e-12
    assert 0.45 < (Y == 0).mean() < 0.55            # ReLU zeroes about half of N(0, 1/3) values


def test_threads_do_not_change_results():
    d = ki.gemm_inputs("c3", M=16, N=64, K=128)
    oracle.set_threads(1)
    a = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", "softmax")
    oracle.set_threads(0)
    b = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", "softmax")
    assert np.array_equal(a, b)


# ------------------------------------------------------------------ row reductions
def test_softmax_invariants():
    d = ki.gemm_inputs("c3", M=9, N=200, K=64)
    P = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", "softmax")
    assert np.abs(P.sum(axis=1) - 1.0).max() < 1e-14 and (P > 0).all()
    Z = ki.widen(d["X"]) @ ki.widen(d["W"]).T + ki.widen(d["b"])
    assert np.abs(P - scipy.special.softmax(Z, axis=1)).max() < 1e-15
    for m in range(9):                                      # monotone in the logits
        assert np.array_equal(np.argsort(P[m], kind="stable"), np.argsort(Z[m], kind="stable"))


def test_softmax_closed_forms():
    N, K = 64, 8
    zeroX = f32(np.zeros((3, K))); W = rng_small((N, K), 3, "f32")
    P = oracle.gemm_rowreduce(zeroX, W, f32(np.full(N, 0.75)), "none", "softmax")
    assert np.array_equal(P, np.full((3, N), 1.0 / N))       # constant row -> exactly 1/N
    b = f32(np.log(np.arange(1, N + 1)))                      # P_j = (j+1) / (N(N+1)/2)
    P = oracle.gemm_rowreduce(zeroX, W, b, "none", "softmax")
    want = np.arange(1, N + 1) / (N * (N + 1) / 2)
    assert np.abs(P[1] / want - 1).max() < 3e-7               # fp32 rounding of ln(j+1)
    # shift invariance: adding a constant to every logit leaves the output unchanged
    b2 = f32(ki.widen(b) + 8.0)
    P2 = oracle.gemm_rowreduce(zeroX, W, b2, "none", "softmax")
    assert np.abs(P2 / P - 1).max() < 2e-6
    # one logit far above the rest -> one-hot, no overflow
    b3 = f32(np.zeros(N)); b3[17] = 3000.0
    P3 = oracle.gemm_rowreduce(zeroX, W, b3, "none", "softmax")
    assert P3[0, 17] == 1.0 and P3[0].sum() == 1.0 and not np.isnan(P3).any()


def test_rowsum_closed_forms():
    N, K, M = 48, 16, 5
    P = oracle.gemm_rowreduce(f32(np.zeros((M, K))), rng_small((N, K), 1, "f32"),
                              f32(np.zeros(N)), "sigmoid", "sum")
    assert np.array_equal(P, np.full(M, N / 2))
    # sigmoid(z) + sigmoid(-z) = 1: stacking W with -W and b with -b gives exactly N per row
    d = ki.gemm_inputs("c4", M=M, N=N, K=K)
    W2 = ki.store(np.concatenate([ki.widen(d["W"]), -ki.widen(d["W"])]), "bf16")
    b2 = ki.store(np.concatenate([ki.widen(d["b"]), -ki.widen(d["b"])]), "bf16")
    S = oracle.gemm_rowreduce(d["X"], W2, b2, "sigmoid", "sum")
    assert np.abs(S - N).max() < 1e-12
    S1 = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "sigmoid", "sum")
    assert ((S1 > 0) & (S1 < N)).all()
    Z = ki.widen(d["X"]) @ ki.widen(d["W"]).T + ki.widen(d["b"])
    assert np.abs(S1 - scipy.special.expit(Z).sum(axis=1)).max() < 1e-12
    # plain row sum of the GEMM output with no activation = X @ (sum of W rows) + sum b
    S0 = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", "sum")
    want = ki.widen(d["X"]) @ ki.widen(d["W"]).sum(axis=0) + ki.widen(d["b"]).sum()
    assert np.abs(S0 - want).max() < 1e-12


# ------------------------------------------------------------------ conv + GroupNorm
def test_conv_delta_kernels_pin_orientation_and_padding():
    Nb, C, H, W = 2, 3, 5, 4
    x = rng_small((Nb, C, H, W), 8, "bf16"); xw = ki.widen(x)
    wt = np.zeros((C, C, 3, 3)); wt[np.arange(C), np.arange(C), 1, 1] = 1.0
    assert np.array_equal(oracle.conv3x3_gn(x, bf(wt)), xw)                 # centre tap: copy
    wt = np.zeros((C, C, 3, 3)); wt[np.arange(C), np.arange(C), 0, 0] = 1.0
    y = oracle.conv3x3_gn(x, bf(wt))                                        # y[h,w] = x[h-1,w-1]
    want = np.zeros_like(xw); want[:, :, 1:, 1:] = xw[:, :, :-1, :-1]
    assert np.array_equal(y, want)
    wt = np.zeros((C, C, 3, 3)); wt[np.arange(C), np.arange(C), 2, 1] = 1.0
    y = oracle.conv3x3_gn(x, bf(wt))                                        # y[h,w] = x[h+1,w]
    want = np.zeros_like(xw); want[:, :, :-1, :] = xw[:, :, 1:, :]
    assert np.array_equal(y, want)


def test_conv_all_ones_counts_taps():
    Cin, H, W = 4, 6, 7
    y = oracle.conv3x3_gn(bf(np.ones((1, Cin, H, W))), bf(np.ones((2, Cin, 3, 3))))
    assert y[0, 0, 2, 3] == 9 * Cin and y[0, 1, 0, 3] == 6 * Cin and y[0, 0, H - 1, 0] == 4 * Cin
    assert y[0, 1, 3, W - 1] == 6 * Cin and y[0, 0, 0, 0] == 4 * Cin


def test_conv_matches_library_correlate_and_is_linear():
    Nb, Cin, H, W, Cout = 2, 3, 6, 5, 4
    d = ki.conv_inputs(Nb=Nb, Cin=Cin, H=H, W=W, Cout=Cout, groups=0, seed=5)
    y = oracle.conv3x3_gn(d["x"], d["w"], d["bias"])
    xw, ww, bw = ki.widen(d["x"]), ki.widen(d["w"]), ki.widen(d["bias"])
    for n in range(Nb):
        for o in range(Cout):
            ref = sum(scipy.signal.correlate2d(xw[n, c], ww[o, c], mode="same", boundary="fill")
                      for c in range(Cin)) + bw[o]
            assert np.abs(y[n, o] - ref).max() < 1e-13
    w2 = rng_small((Cout, Cin, 3, 3), 9, "bf16")
    wsum = bf(ww + ki.widen(w2))                      # sums of small dyadic values stay exact?
    if np.array_equal(ki.widen(wsum), ww + ki.widen(w2)):
        ya = oracle.conv3x3_gn(d["x"], d["w"]); yb = oracle.conv3x3_gn(d["x"], w2)
        assert np.abs(oracle.conv3x3_gn(d["x"], wsum) - (ya + yb)).max() < 1e-12


def test_conv_brute_force_exact_tiny():
    for (Nb, Cin, H, W, Cout) in [(1, 2, 1, 1, 4), (2, 3, 3, 3, 4), (1, 4, 5, 3, 8)]:
        d = ki.conv_inputs(Nb=Nb, Cin=Cin, H=H, W=W, Cout=Cout, groups=0, seed=2)
        y = oracle.conv3x3_gn(d["x"], d["w"], d["bias"], "relu")
        xw, ww, bw = ki.widen(d["x"]), ki.widen(d["w"]), ki.widen(d["bias"])
        for n in range(Nb):
            for o in range(Cout):
                for h in range(H):
                    for w in range(W):
                        acc = Fraction(float(bw[o]))
                        for s in range(3):
                            for r in range(3):
                                for c in range(Cin):
                                    hh, wc = h + r - 1, w + s - 1
                                    if 0 <= hh < H and 0 <= wc < W:
                                        acc += Fraction(float(xw[n, c, hh, wc])) * Fraction(float(ww[o, c, r, s]))
                        want = max(float(acc), 0.0)
                        assert abs(y[n, o, h, w] - want) < 1e-13


def test_groupnorm_moments_and_mapping():
    d = ki.conv_inputs(Nb=2, Cin=4, H=8, W=8, Cout=16, groups=4, seed=1)
    a = oracle.conv3x3_gn(d["x"], d["w"], d["bias"], "relu", groups=0)
    y = oracle.conv3x3_gn(d["x"], d["w"], d["bias"], "relu", groups=4, eps=1e-5)
    for n in range(2):
        for g in range(4):
            blk_a = a[n, 4 * g:4 * g + 4]; blk = y[n, 4 * g:4 * g + 4]    # contiguous channel groups
            var = blk_a.var()                                              # numpy: biased variance
            assert abs(blk.mean()) < 1e-12
            assert abs(blk.var() - var / (var + 1e-5)) < 1e-12
            assert np.abs(blk - (blk_a - blk_a.mean()) / np.sqrt(var + 1e-5)).max() < 1e-12
            # ReLU-clipped positions all share the group's minimum value -mu/sqrt(var+eps)
            if (blk_a == 0).any():
                assert np.abs(blk[blk_a == 0] + blk_a.mean() / np.sqrt(var + 1e-5)).max() < 1e-12


def test_groupnorm_biased_variance_four_element_group():
    # 1x1 image, 4 channels per group, x = 0 so a = bias: the group is {1,2,3,4}/4
    bias = bf(np.array([0.25, 0.5, 0.75, 1.0, 2.0, 2.0, 2.0, 2.0]))
    y = oracle.conv3x3_gn(bf(np.zeros((1, 2, 1, 1))), bf(np.zeros((8, 2, 3, 3))), bias, "relu",
                          groups=2, eps=0.0)
    v = np.array([0.25, 0.5, 0.75, 1.0]); mu = 0.625
    biased = math.sqrt(((v - mu) ** 2).sum() / 4)             # sqrt(5/64); unbiased would be /3
    assert np.abs(y[0, :4, 0, 0] - (v - mu) / biased).max() < 1e-14
    assert abs((y[0, :4, 0, 0] ** 2).sum() - 4.0) < 1e-13     # unit biased variance exactly
    # four equal constants: (a-mu) = 0; with eps > 0 the output is exactly 0, not 0/0
    y = oracle.conv3x3_gn(bf(np.zeros((1, 2, 1, 1))), bf(np.zeros((8, 2, 3, 3))), bias, "relu",
                          groups=2, eps=1e-5)
    assert np.array_equal(y[0, 4:, 0, 0], np.zeros(4))
    # eps sits inside the root: group {0.25..1} with eps = 5/64 doubles the variance term
    y = oracle.conv3x3_gn(bf(np.zeros((1, 2, 1, 1))), bf(np.zeros((8, 2, 3, 3))), bias, "relu",
                          groups=2, eps=5.0 / 64)
    assert np.abs(y[0, :4, 0, 0] - (v - mu) / math.sqrt(10.0 / 64)).max() < 1e-14


def test_groupnorm_affine_and_homogeneity():
    d = ki.conv_inputs(Nb=1, Cin=2, H=4, W=4, Cout=8, groups=2, seed=3)
    y0 = oracle.conv3x3_gn(d["x"], d["w"], d["bias"], "relu", groups=2)
    gamma = bf(np.array([1, 2, -1, 0.5, 1, 1, 4, -2.0])); beta = bf(np.arange(8) / 4.0)
    y1 = oracle.conv3x3_gn(d["x"], d["w"], d["bias"], "relu", groups=2, gamma=gamma, beta=beta)
    want = y0 * ki.widen(gamma)[None, :, None, None] + ki.widen(beta)[None, :, None, None]
    assert np.abs(y1 - want).max() < 1e-13
    # scaling w and bias by 2 (exact in bf16) changes the output only through eps
    w2 = bf(2 * ki.widen(d["w"])); b2 = bf(2 * ki.widen(d["bias"]))
    y2 = oracle.conv3x3_gn(d["x"], w2, b2, "relu", groups=2)
    assert np.abs(y2 - y0).max() < 1e-3 and np.abs(y2 - y0).max() > 0


# ------------------------------------------------------------------ input generator
def test_generator_is_deterministic_and_index_addressable():
    a = ki.normal(0, 1, (64, 32)); b = ki.normal(0, 1, (64, 32))
    assert np.array_equal(a, b)
    assert not np.array_equal(a, ki.normal(1, 1, (64, 32)))
    assert not np.array_equal(a, ki.normal(0, 2, (64, 32)))
    rows = [3, 17, 40]
    full = ki.gemm_inputs("c2", M=64, N=16, K=32)
    part = ki.gemm_inputs("c2", M=64, N=16, K=32, rows=rows)
    assert np.array_equal(part["X"], full["X"][rows]) and np.array_equal(part["R"], full["R"][rows])
    assert np.array_equal(part["W"], full["W"])


def test_generator_distributions():
    z = ki.normal(0, 1, (1 << 18,))
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01 and abs((z ** 3).mean()) < 0.03
    assert abs((z ** 4).mean() - 3.0) < 0.1
    u = ki.uniform(0, 2, (1 << 18,), -0.25, 0.25)
    assert u.min() >= -0.25 and u.max() < 0.25 and abs(u.mean()) < 1e-3
    assert abs(u.var() - 0.25 / 12) < 1e-4
    d = ki.gemm_inputs("c1")
    assert d["X"].dtype == np.float32 and d["X"].shape == (128, 512) and d["W"].shape == (256, 512)
    assert abs(float(np.abs(d["W"]).max()) - 1 / math.sqrt(512)) < 1e-3


def test_bf16_rounding_is_nearest_even():
    v = np.array([1 + 2 ** -8, 1 + 3 * 2 ** -8, 1 + 2 ** -7, -(1 + 2 ** -8), 1 + 2 ** -8 + 2 ** -20])
    got = ki.widen(ki.to_bf16_bits(v))
    assert np.array_equal(got, [1.0, 1 + 2 ** -6, 1 + 2 ** -7, -1.0, 1 + 2 ** -7])
    x = ki.normal(3, 1, (1000,))
    assert np.abs(ki.widen(ki.to_bf16_bits(x)) / x - 1).max() <= 2 ** -8


# ------------------------------------------------------------------ conv -> channel softmax -> pool
def test_channel_softmax_invariants_and_library_case():
    d = ki.conv_inputs(Nb=2, Cin=3, H=6, W=8, Cout=5, groups=0, seed=7)
    s = oracle.conv3x3_softmax_pool(d["x"], d["w"], d["bias"], pool=1)
    assert np.abs(s.sum(axis=1) - 1.0).max() < 1e-14 and (s > 0).all()      # over channels
    c = oracle.conv3x3_gn(d["x"], d["w"], d["bias"])                         # pinned above
    assert np.abs(s - scipy.special.softmax(c, axis=1)).max() < 1e-15
    # the reduction runs over channels, not over pixels: pixel sums are not 1
    assert np.abs(s.sum(axis=(2, 3)) - 1.0).min() > 0.5
    # shift invariance per pixel: adding a constant to every channel's bias changes nothing
    b2 = ki.store(ki.widen(d["bias"]) + 0.5, "bf16")
    if np.array_equal(ki.widen(b2), ki.widen(d["bias"]) + 0.5):
        s2 = oracle.conv3x3_softmax_pool(d["x"], d["w"], b2, pool=1)
        assert np.abs(s2 - s).max() < 1e-14
    # zero weights: every channel equal -> exactly 1/Cout
    z = oracle.conv3x3_softmax_pool(d["x"], bf(np.zeros((5, 3, 3, 3))), None, pool=1)
    assert np.array_equal(z, np.full_like(z, 0.2))


def test_channel_softmax_pooling():
    d = ki.conv_inputs(Nb=1, Cin=2, H=8, W=12, Cout=4, groups=0, seed=8)
    s = oracle.conv3x3_softmax_pool(d["x"], d["w"], d["bias"], pool=1)
    for k in (2, 4):
        p = oracle.conv3x3_softmax_pool(d["x"], d["w"], d["bias"], pool=k)
        want = s[:, :, :8 // k * k, :12 // k * k].reshape(1, 4, 8 // k, k, 12 // k, k).max(axis=(3, 5))
        assert p.shape == (1, 4, 8 // k, 12 // k) and np.array_equal(p, want)
    # two pools of 2 in a row (the paper's chain) equal one pool of 4
    p2 = oracle.conv3x3_softmax_pool(d["x"], d["w"], d["bias"], pool=2)
    twice = p2.reshape(1, 4, 2, 2, 3, 2).max(axis=(3, 5))
    assert np.array_equal(twice, oracle.conv3x3_softmax_pool(d["x"], d["w"], d["bias"], pool=4))
    # a ragged rim is dropped
    d3 = ki.conv_inputs(Nb=1, Cin=2, H=5, W=7, Cout=3, groups=0, seed=9)
    assert oracle.conv3x3_softmax_pool(d3["x"], d3["w"], None, pool=2).shape == (1, 3, 2, 3)


# ------------------------------------------------------------------ stored fixed points
def test_activation_fixed_points_from_golden_file():
    """Values of the activation definitions at fixed points, computed once with 40-digit
    arithmetic by tests/golden/make_activation_fixed_points.py (no oracle, no GPU)."""
    path = os.path.join(os.path.dirname(__file__), "golden", "activation_fixed_points.txt")
    n = 0
    for line in open(path):
        line = line.split("#")[0].split()
        if len(line) == 3:
            name, z, want = line[0], float(line[1]), float(line[2])
            assert abs(oracle.act(name, z) - want) <= 4e-16 * max(1.0, abs(want)), (name, z)
            n += 1
    assert n == 7


# ------------------------------------------------------------------ the worked chain's rewrites
def test_chain95_rewrites_agree():
    """Appendix C.2 prints four programs for the same post-matmul chain (iterations 15, 20, 25
    and 30); they differ only in how the same algebra is written.  Each variant is restated
    here from its description -- clamp by min/max or by two selects, exp(2s) evaluated twice or
    once, the erf argument inline or as a temporary -- and all of them must agree with each
    other and with the oracle's chain95 on a grid (values where exp(2s) is finite)."""
    c = golden()

    def swish(x):
        return x / (1.0 + math.exp(-x)) if x > -700 else 0.0

    def clamp_minmax(g):
        return min(max(g, c["hardtanh_lo"]), c["hardtanh_hi"])

    def clamp_select(g):
        return c["hardtanh_hi"] if g > c["hardtanh_hi"] else (c["hardtanh_lo"] if g < c["hardtanh_lo"] else g)

    def form_a(x):          # exponential written out twice, clamp by min/max
        s = swish(x)
        t = (math.exp(c["tanh_exp_factor"] * s) - 1.0) / (math.exp(c["tanh_exp_factor"] * s) + 1.0)
        return clamp_minmax(t * 0.5 * (1.0 + math.erf(t * c["erf_gelu_inner_scale"])))

    def form_b(x):          # same, clamp by two selects (two of the printed programs share this form)
        s = swish(x)
        t = (math.exp(2 * s) - 1) / (math.exp(2 * s) + 1)
        return clamp_select(t * 0.5 * (1.0 + math.erf(t * c["erf_gelu_inner_scale"])))

    def form_c(x):          # sigmoid reused, one exponential, erf argument as a temporary
        sg = 1.0 / (1.0 + math.exp(-x)) if x > -700 else 0.0
        s = sg * x
        e2 = math.exp(2.0 * s)
        t = (e2 - 1.0) / (e2 + 1.0)
        arg = t * c["erf_gelu_inner_scale"]
        return clamp_select(t * 0.5 * (1.0 + math.erf(arg)))

    zs = np.concatenate([np.linspace(-30.0, 30.0, 1201), [-300.0, -50.0, 50.0, 300.0, 1e-9, -1e-9]])
    for z in zs:
        z = float(z)
        a, b, cc = form_a(z), form_b(z), form_c(z)
        assert abs(a - b) < 1e-15 and abs(a - cc) < 1e-15, z
        assert abs(oracle.act("chain95", z) - a) < 1e-14, z
    # the chain's range: swish >= -0.2785, so tanh >= -0.2716 and gelu(erf) of it >= -0.107; the
    # upper clamp is reached only in the limit (gelu_erf(1) = 0.8413 < 1): hardtanh never acts
    vals = np.array([oracle.act("chain95", float(z)) for z in zs])
    assert vals.min() > -0.11 and vals.max() < 0.8414


# ------------------------------------------------------------------ full-size spot checks
# One sampled row (image) of every full-size benchmark configuration: the oracle's routine on
# that row against numpy / scipy fp64 on the same stored inputs.  Rows are independent, and the
# generator is index-addressed, so a row subset holds exactly the full tensor's values there.
def _rows_for(M):
    return np.array([0, M // 2 + 1, M - 1])


def test_full_size_c2_rows_against_numpy():
    rows = _rows_for(8192)
    d = ki.gemm_inputs("c2", seed=0, rows=rows)
    got = oracle.gemm_epilogue(d["X"], d["W"], d["b"], "gelu_tanh", 0.5, d["R"])
    z = ki.widen(d["X"]) @ ki.widen(d["W"]).T + ki.widen(d["b"])
    want = 0.5 * (0.5 * z * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))) + ki.widen(d["R"])
    assert got.shape == (3, 4096)
    assert np.abs(got - want).max() < 1e-12


def test_full_size_c3_rows_against_scipy():
    rows = _rows_for(4096)
    d = ki.gemm_inputs("c3", seed=0, rows=rows)
    got = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "none", "softmax")
    z = ki.widen(d["X"]) @ ki.widen(d["W"]).T + ki.widen(d["b"])
    want = scipy.special.softmax(z, axis=1)
    assert got.shape == (3, 8192)
    assert np.abs(got - want).max() < 1e-15 and np.abs(got / want - 1).max() < 1e-11


def test_full_size_c4_rows_against_scipy():
    rows = _rows_for(16384)
    d = ki.gemm_inputs("c4", seed=0, rows=rows)
    got = oracle.gemm_rowreduce(d["X"], d["W"], d["b"], "sigmoid", "sum").reshape(-1)
    z = ki.widen(d["X"]) @ ki.widen(d["W"]).T + ki.widen(d["b"])
    want = scipy.special.expit(z).sum(axis=1)
    assert np.abs(got - want).max() < 1e-10


def test_full_size_c5_image_against_numpy():
    d = ki.conv_inputs("c5", seed=0, images=[77])
    got = oracle.conv3x3_gn(d["x"], d["w"], d["bias"], "relu", d["groups"], d["eps"])
    x, w, b = ki.widen(d["x"])[0], ki.widen(d["w"]), ki.widen(d["bias"])
    xp = np.pad(x, ((0, 0), (1, 1), (1, 1)))
    win = np.lib.stride_tricks.sliding_window_view(xp, (3, 3), axis=(1, 2))      # [c, h, w, r, s]
    y = np.tensordot(w, win, axes=([1, 2, 3], [0, 3, 4])) + b[:, None, None]      # [o, h, w]
    a = np.maximum(y, 0.0).reshape(d["groups"], -1)
    want = ((a - a.mean(axis=1, keepdims=True)) / np.sqrt(a.var(axis=1, keepdims=True) + d["eps"])).reshape(y.shape)
    assert got.shape == (1, 128, 64, 64)
    assert np.abs(got[0] - want).max() < 1e-11


def test_generator_row_subsets_hold_the_full_tensor_values():
    a = ki.gemm_inputs("c2", seed=3, M=40, N=24, K=16)
    b = ki.gemm_inputs("c2", seed=3, M=40, N=24, K=16, rows=[3, 39, 0])
    assert (a["X"][[3, 39, 0]] == b["X"]).all() and (a["R"][[3, 39, 0]] == b["R"]).all()
    c = ki.conv_inputs(seed=2, Nb=5, Cin=3, H=4, W=6, Cout=2)
    e = ki.conv_inputs(seed=2, Nb=5, Cin=3, H=4, W=6, Cout=2, images=[4, 1])
    assert (c["x"][[4, 1]] == e["x"]).all()
