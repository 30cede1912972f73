"""Host-side checks that need no GPU: the library loads, exports every declared symbol,
and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2506_04985_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def test_header_symbols_are_exported(B):
    text = open(os.path.join(ROOT, "include", "fpt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(fpt_[a-z0-9_]+)\s*\(", text))
    assert declared == set(B.EXPORTS)
    L = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name


def test_version_and_strerror(B):
    assert B.fpt_version() >= 100
    assert B.strerror(0) == "ok"
    for code in range(-6, 0):
        assert "unknown" not in B.strerror(code)
    assert "unknown" in B.strerror(-99)


def test_workspace_sizes(B):
    assert B.fpt_workspace_bytes(B.OP_GEMM, 128, 1024, 1024) >= 8192
    assert B.fpt_workspace_bytes(B.OP_GEMM, 64, 1024, 1024) > B.fpt_workspace_bytes(B.OP_GEMM, 128, 1024, 1024)
    lin = B.fpt_workspace_bytes(B.OP_LINEAR, 2048, 4096, 4096)
    assert lin >= 2048 * 4096 // 2 + 2048 * 4
    # the MLP block: the 16-bit buffer between the two matmuls is reserved only where a route uses it
    M, dff, d = 4096, 14336, 4096
    base = M * d // 2 + M * dff // 2                   # codes at the block input and at the down-projection input
    fused = B.fpt_workspace_bytes(B.OP_MLP, M, dff, d)
    assert base <= fused < base + (1 << 20), "fused route (more than 128 tokens): no gate||up buffer"
    had = B.fpt_workspace_bytes(B.OP_MLP_HADAMARD, M, dff, d)
    assert base + M * dff * 2 <= had < base + M * dff * 2 + (1 << 20), "with the transform: the bf16 products"
    for op in (B.OP_MLP, B.OP_MLP_HADAMARD):
        small = B.fpt_workspace_bytes(op, 64, dff, d)
        assert small >= 64 * d // 2 + 64 * dff // 2 + 64 * 2 * dff * 2, "unfused route: gate||up in bf16"
    assert B.fpt_workspace_bytes(99, 1, 1, 1) == 0
    assert B.fpt_workspace_bytes(B.OP_GEMM, 0, 8, 128) == 0


def test_argument_errors_are_reported_before_any_launch(B):
    L = B.lib()
    qp = B.QParams(4, True, 0.5, 0)
    fake = ctypes.c_void_p(0x1000)          # never dereferenced: all calls fail validation first
    odd = ctypes.c_void_p(0x1004)
    r = L.fpt_act_quant(None, None, 4, 128, 128, ctypes.byref(qp), B.RMSNORM, 1e-5, None, None, fake, None)
    assert r == B.ERR_BAD_ARG
    r = L.fpt_act_quant(None, fake, 4, 100, 100, ctypes.byref(qp), B.RMSNORM, 1e-5, None, None, fake, None)
    assert r == B.ERR_UNSUPPORTED                      # K not a multiple of 32
    r = L.fpt_act_quant(None, odd, 4, 128, 128, ctypes.byref(qp), B.RMSNORM, 1e-5, None, None, fake, None)
    assert r == B.ERR_ALIGNMENT
    r = L.fpt_act_quant(None, fake, 4, 128, 128, ctypes.byref(qp), B.SCALE_INPUT, 1e-5, None, None, fake, None)
    assert r == B.ERR_BAD_ARG                          # SCALE_INPUT without s_in
    q6 = B.QParams(6, True, 0.5, 0)
    r = L.fpt_act_quant(None, fake, 4, 128, 128, ctypes.byref(q6), B.RMSNORM, 1e-5, None, None, fake, None)
    assert r == B.ERR_UNSUPPORTED
    q8a = B.QParams(8, False, 0.5, 3)                  # 8-bit codes exist on the symmetric grid only
    r = L.fpt_act_quant(None, fake, 4, 128, 128, ctypes.byref(q8a), B.RMSNORM, 1e-5, None, None, fake, None)
    assert r == B.ERR_UNSUPPORTED
    r = L.fpt_act_quant_dynamic(None, fake, 4, 128, 128, 5, B.RMSNORM, 1e-5, None, fake, None, fake)
    assert r == B.ERR_UNSUPPORTED
    r = L.fpt_act_quant_dynamic(None, fake, 4, 128, 128, 4, B.RMSNORM, 1e-5, None, fake, None, None)
    assert r == B.ERR_BAD_ARG                          # the per-token scales must go somewhere
    a8 = lambda M, N, K, ws, wsb: (None, fake, fake, M, N, K, fake, B.DTYPE_F32, 0.5, None, None, None, fake, None, ws, wsb)
    assert L.fpt_w4a8_gemm(*a8(4, 64, 32768, fake, 1 << 30)) == B.ERR_UNSUPPORTED      # (float)acc would round
    assert L.fpt_w4a8_gemm(*a8(4, 64, 100, fake, 1 << 30)) == B.ERR_UNSUPPORTED
    assert L.fpt_w4a8_gemm(*a8(4, 64, 128, None, 0)) == B.ERR_WORKSPACE
    assert L.fpt_w4a8_gemm(*a8(4, 64, 128, fake, 16)) == B.ERR_WORKSPACE
    assert L.fpt_workspace_bytes(B.OP_GEMM_A8, 300, 512, 1024) == L.fpt_workspace_bytes(B.OP_GEMM, 300, 512, 1024)
    assert L.fpt_workspace_bytes(B.OP_GEMM_A8, 64, 128, 1024) > L.fpt_workspace_bytes(B.OP_GEMM, 64, 128, 1024)
    qbad = B.QParams(4, False, 0.5, 16)
    r = L.fpt_act_quant(None, fake, 4, 128, 128, ctypes.byref(qbad), B.RMSNORM, 1e-5, None, None, fake, None)
    assert r == B.ERR_BAD_ARG
    # matmul: K must be a multiple of 128, N of 8, workspace present and large enough
    args = lambda M, N, K, ws, wsb: (None, fake, fake, M, N, K, fake, B.DTYPE_F32, None, 0.5, 1, 0, None, None, None,
                                     fake, None, ws, wsb)
    assert L.fpt_w4a4_gemm(*args(16, 64, 96, fake, 1 << 30)) == B.ERR_UNSUPPORTED
    assert L.fpt_w4a4_gemm(*args(16, 60, 128, fake, 1 << 30)) == B.ERR_UNSUPPORTED
    assert L.fpt_w4a4_gemm(*args(16, 64, 128, None, 0)) == B.ERR_WORKSPACE
    assert L.fpt_w4a4_gemm(*args(16, 64, 128, fake, 8)) == B.ERR_WORKSPACE
    assert L.fpt_w4a4_gemm(*args(0, 64, 128, fake, 1 << 30)) == B.ERR_BAD_ARG
    # asymmetric activations need the weight row sums
    r = L.fpt_w4a4_gemm(None, fake, fake, 16, 64, 128, fake, B.DTYPE_F32, None, 0.5, 0, 8, None, None, None, fake,
                        None, fake, 1 << 30)
    assert r == B.ERR_BAD_ARG
    r = L.fpt_quantize_weights(None, fake, B.DTYPE_BF16, 8, 128, ctypes.byref(B.QParams(4, False, 1.0, 8)),
                               B.RANGE_MINMAX, 3.0, B.DTYPE_F32, fake, fake, None)
    assert r == B.ERR_UNSUPPORTED                      # weights use the symmetric grid
    r = L.fpt_decoder_mlp(None, fake, 8, 100, 256, fake, fake, fake, fake, B.DTYPE_F32, ctypes.byref(qp),
                          ctypes.byref(qp), 1e-5, None, None, 0, 0, fake, fake, 1 << 30)
    assert r == B.ERR_UNSUPPORTED
    assert L.fpt_check_status(None, None) == B.ERR_BAD_ARG


def test_oracle_and_library_share_no_code():
    """The checker must not import the product and the product must not import the checker."""
    for dirpath, _, files in os.walk(os.path.join(ROOT, "oracle")):
        for f in files:
            if f.endswith(".py"):
                src = open(os.path.join(dirpath, f)).read()
                assert "paper_2506_04985_b200" not in src and "ctypes" not in src
    for dirpath, _, files in os.walk(os.path.join(ROOT, "paper_2506_04985_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle", src, flags=re.M), f
