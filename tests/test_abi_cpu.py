"""CPU-only checks of the C ABI: the library loads, exports every symbol the header declares, and rejects
bad arguments on the host before anything is launched.  No compute calls."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2505_20932_b200 import build
    build.build_library()
    from paper_2505_20932_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "qwt2.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qwt_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(B):
    names = declared_functions()
    assert len(names) >= 18
    for n in names:
        assert hasattr(B.lib, n), f"libqwt2.so does not export {n}"
    assert set(names) == set(B.SIGNATURES), "binding and header disagree on the entry points"
    assert "sm_100a" in B.qwt_version()


def test_status_strings(B):
    seen = {B.qwt_status_string(s) for s in range(0, 10)}
    assert len(seen) == 10 and B.qwt_status_string(0) == "ok"


def test_workspace_sizes(B):
    assert B.qwt_cwac_workspace_bytes(0, 8) == 0
    w = B.qwt_cwac_workspace_bytes(403456, 3072)
    assert 0 < w < 64 << 20 and w % 1024 == 0
    assert B.qwt_qlinear_workspace_bytes(8192, 11008, 4096, B.QWT_W_INT8, B.QWT_OUT_INT8_PER_TOKEN) >= 4 * 8192
    assert B.qwt_qlinear_host_staging_bytes(788, 1536, 384, 0, 0) >= 788 * 384 + 788 * 1536
    assert B.qwt_cwac_host_staging_bytes(100, 64) > 0


def test_calibrate_argument_errors(B):
    buf = np.zeros(4096, np.float32)
    p = buf.ctypes.data
    assert p % 16 == 0
    ws = 1 << 20
    call = lambda *a: B.lib.qwt_cwac_calibrate(*a)
    assert call(None, p, 8, 8, 8, p, p, None, p, ws, None) == B.QWT_ERR_NULL
    assert call(p, p, 8, 8, 8, None, p, None, p, ws, None) == B.QWT_ERR_NULL
    assert call(p, p, 0, 8, 8, p, p, None, p, ws, None) == B.QWT_ERR_SHAPE
    assert call(p, p, 8, 8, 4, p, p, None, p, ws, None) == B.QWT_ERR_SHAPE          # ld < channels
    assert call(p, p, 8, 6, 6, p, p, None, p, ws, None) == B.QWT_ERR_ALIGN          # ld % 4
    assert call(p + 4, p, 8, 8, 8, p, p, None, p, ws, None) == B.QWT_ERR_ALIGN
    assert call(p, p, 8, 8, 8, p, p, None, p, 16, None) == B.QWT_ERR_WORKSPACE
    assert B.lib.qwt_cwac_solve(None, 8, p, p, None, None) == B.QWT_ERR_NULL
    assert B.lib.qwt_cwac_solve(p, 0, p, p, None, None) == B.QWT_ERR_SHAPE
    assert B.lib.qwt_cwac_fold(p, None, p, None, 8, p, p, None) == B.QWT_ERR_NULL   # a without b
    assert B.lib.qwt_cwac_fold(p, None, None, None, 0, p, p, None) == B.QWT_ERR_SHAPE


def test_forward_argument_errors(B):
    buf = np.zeros(1 << 16, np.int8)
    p = buf.ctypes.data
    assert p % 256 == 0 or True
    p = (p + 255) // 256 * 256
    big = 1 << 30
    f = lambda X, xs, W, wf, fs, fb, M, N, K, om, Y, ys, ws, wsb: B.lib.qwt_qlinear_cwac_forward(
        X, xs, W, wf, fs, fb, M, N, K, om, Y, ys, ws, wsb, None)
    I8, BF, F32, ACC = B.QWT_OUT_INT8_PER_TOKEN, B.QWT_OUT_BF16, B.QWT_OUT_FP32, B.QWT_OUT_INT32_ACC
    assert f(None, p, p, 0, p, p, 16, 16, 16, I8, p, p, p, big) == B.QWT_ERR_NULL
    assert f(p, None, p, 0, p, p, 16, 16, 16, I8, p, p, p, big) == B.QWT_ERR_NULL      # scales required
    assert f(p, p, p, 0, p, p, 16, 16, 16, I8, p, None, p, big) == B.QWT_ERR_NULL      # y_scale required for INT8
    assert f(p, p, p, 0, p, p, 0, 16, 16, I8, p, p, p, big) == B.QWT_ERR_SHAPE
    assert f(p, p, p, 0, p, p, 16, 16, 1 << 20, I8, p, p, p, big) == B.QWT_ERR_SHAPE   # accumulator could overflow
    assert f(p, p, p, 0, p, p, 16, 16, 24, I8, p, p, p, big) == B.QWT_ERR_UNSUPPORTED  # K % 16
    assert f(p, p, p, 1, p, p, 16, 16, 16, I8, p, p, p, big) == B.QWT_ERR_UNSUPPORTED  # packed int4 needs K % 32
    assert f(p, p, p, 0, p, p, 16, 24, 16, I8, p, p, p, big) == B.QWT_ERR_UNSUPPORTED  # N % 16 for INT8 out
    assert f(p, p, p, 0, p, p, 16, 12, 16, BF, p, None, p, big) == B.QWT_ERR_UNSUPPORTED
    assert f(p, p, p, 7, p, p, 16, 16, 16, I8, p, p, p, big) == B.QWT_ERR_UNSUPPORTED  # unknown weight format
    assert f(p, p, p, 0, p, p, 16, 16, 16, 9, p, p, p, big) == B.QWT_ERR_UNSUPPORTED   # unknown output mode
    assert f(p + 8, p, p, 0, p, p, 16, 16, 16, I8, p, p, p, big) == B.QWT_ERR_ALIGN
    assert f(p, p, p, 0, p, p, 16, 16, 16, I8, p, p, None, big) == B.QWT_ERR_NULL
    assert f(p, p, p, 0, p, p, 16, 16, 16, I8, p, p, p, 8) == B.QWT_ERR_WORKSPACE
    assert f(p, p, p, 0, p, p, 16, 16, 16, I8, p, p, p + 8, big) == B.QWT_ERR_WORKSPACE
    q = lambda *a: B.lib.qwt_quantize_rows_i8(*a)
    assert q(p, 4, 8, 8, 200, p, p, None) == B.QWT_ERR_UNSUPPORTED
    assert q(p, 4, 8, 4, 127, p, p, None) == B.QWT_ERR_SHAPE
    assert B.lib.qwt_pack_int4(p, 4, 7, p, None) == B.QWT_ERR_UNSUPPORTED


def test_valid_call_without_a_gpu_reports_a_cuda_error(B):
    torch = pytest.importorskip("torch")
    if torch.cuda.is_available():
        pytest.skip("a GPU is present: this checks the no-device error path only")
    buf = np.zeros(4096, np.float32)
    p = (buf.ctypes.data + 255) // 256 * 256
    s = B.lib.qwt_cwac_fold(p, None, None, None, 8, p, p, None)
    assert s in (B.QWT_ERR_CUDA, B.QWT_ERR_ARCH)     # never a silent CPU fallback
    e = C.c_int(0)
    assert B.lib.qwt_last_cuda_error(C.byref(e)) == B.QWT_OK


def test_product_path_does_not_import_the_oracle():
    import ast
    for rel in ["paper_2505_20932_b200/binding.py", "paper_2505_20932_b200/workload.py",
                "paper_2505_20932_b200/sharding.py", "paper_2505_20932_b200/build.py",
                "paper_2505_20932_b200/__init__.py"]:
        tree = ast.parse(open(os.path.join(ROOT, rel)).read())
        for node in ast.walk(tree):
            if isinstance(node, ast.Import):
                assert not any(a.name.split(".")[0] == "oracle" for a in node.names), rel
            if isinstance(node, ast.ImportFrom):
                assert (node.module or "").split(".")[0] != "oracle", rel
    for f in os.listdir(os.path.join(ROOT, "paper_2505_20932_b200", "csrc")):
        assert "oracle" not in open(os.path.join(ROOT, "paper_2505_20932_b200", "csrc", f)).read().lower(), f
    src = open(os.path.join(ROOT, "oracle", "qwt_oracle.py")).read()
    assert "paper_2505_20932_b200" not in src and "ctypes" not in src
