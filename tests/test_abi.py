"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, answers the pure-host queries, and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

import paper_2605_30359_b200 as kf

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(kf.LIB_PATH):
        from paper_2605_30359_b200.build import build
        build()
    return kf.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "kf.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(kf_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(kf.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_host_queries(lib):
    assert kf.kf_version() >= 100
    assert kf.status_string(kf.KF_OK) == "ok"
    assert "workspace" in kf.status_string(kf.KF_ERR_WORKSPACE)
    assert kf.kf_gemm_epilogue_workspace_bytes(8192, 4096, 4096, kf.KF_BF16) == 0
    # softmax first pass: (max, sum) per row and 256-column tile
    assert kf.kf_gemm_rowreduce_workspace_bytes(4096, 8192, 2048, kf.KF_BF16, 0) == 4096 * 64 * 8   # (max, sum) per half tile
    assert kf.kf_gemm_rowreduce_workspace_bytes(16384, 1024, 1024, kf.KF_BF16, 1) == 16384 * 4 * 4
    # fp32 chains stage the pre-reduction values
    assert kf.kf_gemm_rowreduce_workspace_bytes(128, 256, 512, kf.KF_F32, 0) == 128 * 256 * 4
    # conv: NHWC copy of x, repacked weights, per-tile channel statistics (16 tiles per image; the
    # all-SM GroupNorm kernel's per-tile group statistics share the region)
    assert kf.kf_conv3x3_workspace_bytes(128, 64, 64, 64, 128, kf.KF_BF16, 32) == \
        128 * 64 * 64 * 64 * 2 + 9 * 128 * 64 * 2 + 128 * 16 * 128 * 8
    assert kf.kf_conv3x3_workspace_bytes(1, 3, 5, 5, 4, kf.KF_F32, 0) == 0
    assert kf.kf_launch_count() >= 0


def test_bad_arguments_are_rejected_without_a_launch(lib):
    before = kf.kf_launch_count()
    p = 0x10000  # never dereferenced: validation fails first
    bad = kf.KF_ERR_INVALID_ARG
    ge = kf.kf_gemm_epilogue
    assert ge(0, 8, 8, 1, p, 8, p, 8, None, 0, 1.0, None, 0, p + 4096, 8, None, 0, None) == bad
    assert ge(8, 8, 8, 7, p, 8, p, 8, None, 0, 1.0, None, 0, p + 4096, 8, None, 0, None) == bad
    assert ge(8, 8, 8, 1, None, 8, p, 8, None, 0, 1.0, None, 0, p + 4096, 8, None, 0, None) == bad
    assert ge(8, 8, 8, 1, p, 4, p, 8, None, 0, 1.0, None, 0, p + 4096, 8, None, 0, None) == bad   # ldx < K
    assert ge(8, 8, 8, 1, p, 8, p, 8, None, 99, 1.0, None, 0, p + 4096, 8, None, 0, None) == bad  # act
    assert ge(8, 8, 8, 1, p, 8, p, 8, None, 0, 1.0, None, 0, p, 8, None, 0, None) == bad          # Y aliases X
    assert ge(8, 8, 8, 0, p + 2, 8, p, 8, None, 0, 1.0, None, 0, p + 4096, 8, None, 0, None) == bad  # fp32 misaligned
    assert ge(8, 8, 8, 1, p, 8, p, 8, None, 0, 1.0, p + 8192, 4, p + 4096, 8, None, 0, None) == bad  # ldr < N
    rr = kf.kf_gemm_rowreduce
    assert rr(8, 8, 8, 1, p, 8, p, 8, None, 0, 5, p + 4096, 8, 1, None, 0, None) == bad    # reduction
    assert rr(8, 8, 8, 1, p, 8, p, 8, None, 0, 1, p + 4096, 8, 1, None, 0, None) == bad    # sum wants fp32 out
    assert rr(8, 8, 8, 1, p, 8, p, 8, None, 0, 0, p + 4096, 4, 1, None, 0, None) == bad    # ldo < N
    cv = kf.kf_conv3x3_epilogue
    assert cv(1, 4, 4, 4, 6, 1, p, p, None, 0, 4, 1e-5, None, None, p + 4096, None, 0, None) == bad  # 4 !| 6
    assert cv(1, 4, 0, 4, 6, 1, p, p, None, 0, 0, 1e-5, None, None, p + 4096, None, 0, None) == bad
    assert cv(1, 4, 4, 4, 6, 1, p, p, None, 0, 0, 1e-5, None, None, p, None, 0, None) == bad         # y aliases x
    assert kf.kf_launch_count() == before


def test_binding_refuses_cpu_tensors(lib):
    import torch
    x = torch.zeros(4, 8)
    with pytest.raises(ValueError):
        kf.gemm_epilogue(x, x)


def test_oracle_and_cuda_path_share_no_code():
    """Neither side imports or includes the other; only kf_inputs serves both."""
    pkg = os.path.join(ROOT, "paper_2605_30359_b200")
    for dirpath, _, files in os.walk(pkg):
        if os.path.basename(dirpath) == "build":
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".cpp", ".h")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2605_30359_b200" not in text and "include/kf.h" not in text
            assert "libkf.so" not in text and "csrc" not in text
