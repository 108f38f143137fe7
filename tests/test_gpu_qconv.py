"""GPU parity: k x k convolution as an implicit GEMM (activations read straight from the NHWC tensor by rank-4
tensor-map copies, no patch matrix) against the oracle's convolution by definition, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import qwt_oracle as O
from tolerances import assert_bf16_close, assert_codes_close, assert_fp32_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def B():
    from paper_2505_20932_b200 import binding
    return binding


def run_conv(B, X, xs, Wt, fs, fb, stride, pad, mode):
    Bn, Hh, Ww, C = X.shape
    N, kh, kw, _ = Wt.shape
    Ho, Wo = (Hh + 2 * pad - kh) // stride + 1, (Ww + 2 * pad - kw) // stride + 1
    dt = {B.QWT_OUT_INT8_PER_TOKEN: torch.int8, B.QWT_OUT_BF16: torch.bfloat16, B.QWT_OUT_FP32: torch.float32,
          B.QWT_OUT_INT32_ACC: torch.int32}[mode]
    guard = 64
    n_out = Bn * Ho * Wo * N
    Ybuf = torch.zeros(n_out + 2 * guard, dtype=dt, device=DEV)
    Yi = Ybuf.view(torch.int8 if dt == torch.int8 else (torch.int16 if dt == torch.bfloat16 else torch.int32))
    Yi.fill_(0x5A)
    Y = Ybuf[guard:guard + n_out]
    ysb = torch.full((Bn * Ho * Wo + 2 * guard,), -7.0, dtype=torch.float32, device=DEV)
    ys = ysb[guard:guard + Bn * Ho * Wo] if mode == B.QWT_OUT_INT8_PER_TOKEN else None
    wsb = B.qwt_qconv2d_workspace_bytes(Bn, Hh, Ww, C, N, kh, kw, stride, pad, mode)
    assert wsb > 0
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    ws.fill_(0xFF)
    d = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    B.qwt_qconv2d_cwac_forward(d(X), xs, d(Wt), d(fs), d(fb), Bn, Hh, Ww, C, N, kh, kw, stride, pad, mode, Y, ys, ws, wsb)
    B.qwt_qlinear_check_status(ws)
    gi = Yi.cpu().numpy()
    assert (gi[:guard] == 0x5A).all() and (gi[guard + n_out:] == 0x5A).all(), "output guard band overwritten"
    if ys is not None:
        g = ysb.cpu().numpy()
        assert (g[:guard] == -7.0).all() and (g[guard + Bn * Ho * Wo:] == -7.0).all(), "y_scale guard band overwritten"
    if dt == torch.bfloat16:
        out = Y.view(torch.int16).cpu().numpy().view(np.uint16)
    else:
        out = Y.cpu().numpy()
    return out.reshape(Bn * Ho * Wo, N), (None if ys is None else ys.cpu().numpy())


CASES = [
    # batch, H, W, C, Cout, k, stride, pad
    (2, 14, 14, 128, 64, 3, 1, 1),      # blocks of 16 x 8 positions cover a 14 x 14 image with waste on both sides
    (3, 7, 7, 256, 272, 3, 1, 1),       # several images per tile, two channel blocks per tap, N tail
    (1, 15, 13, 128, 48, 3, 2, 1),      # stride 2, odd sizes
    (2, 9, 20, 128, 528, 5, 1, 2),      # 5 x 5, three column tiles
    (1, 28, 28, 128, 128, 3, 1, 1),     # ResNet-50 stage 2 bottleneck convolution (one image)
    (5, 8, 8, 128, 32, 1, 1, 0),        # 1 x 1 through the same path
    (2, 12, 12, 128, 64, 7, 2, 3),      # 7 x 7 stride 2
]


@pytest.mark.parametrize("Bn,Hh,Ww,C,N,k,stride,pad", CASES)
def test_implicit_convolution_every_output_stage(B, Bn, Hh, Ww, C, N, k, stride, pad):
    rng = np.random.default_rng(Bn * 1000 + Hh * 10 + k + N)
    X = rng.integers(-127, 128, (Bn, Hh, Ww, C)).astype(np.int8)
    Wt = rng.integers(-127, 128, (N, k, k, C)).astype(np.int8)
    acc_ref = O.conv2d_int_nhwc(X, Wt, stride, pad).reshape(-1, N)
    M = acc_ref.shape[0]
    acc, _ = run_conv(B, X, 0.0, Wt, None, None, stride, pad, B.QWT_OUT_INT32_ACC)
    assert np.array_equal(acc.astype(np.int64), acc_ref)
    S_x = 0.02                                                                   # per-tensor activation scale
    fs = rng.uniform(1e-4, 3e-4, N).astype(np.float32)
    fb = (0.01 * rng.standard_normal(N)).astype(np.float32)
    z_ref = O.forward_folded(acc_ref, np.full(M, S_x, np.float32), fs, fb)
    z, _ = run_conv(B, X, S_x, Wt, fs, fb, stride, pad, B.QWT_OUT_FP32)
    assert_fp32_close(z, z_ref)
    bits, _ = run_conv(B, X, S_x, Wt, fs, fb, stride, pad, B.QWT_OUT_BF16)
    assert_bf16_close(bits, z_ref, O.to_bf16_bits, O.bf16_bits_to_f32)
    if N % 16 == 0:
        codes, ys = run_conv(B, X, S_x, Wt, fs, fb, stride, pad, B.QWT_OUT_INT8_PER_TOKEN)
        c_ref, ys_ref = O.requant_per_token(z_ref)
        assert np.allclose(ys, ys_ref, rtol=1e-5, atol=0)
        assert_codes_close(codes, c_ref)


def test_implicit_convolution_equals_the_patch_matrix_path(B):
    """Same integers as qwt_im2col_i8 followed by the forward call."""
    Bn, Hh, Ww, C, N, k, stride, pad = 2, 10, 11, 128, 80, 3, 1, 1
    rng = np.random.default_rng(4)
    X = rng.integers(-127, 128, (Bn, Hh, Ww, C)).astype(np.int8)
    Wt = rng.integers(-127, 128, (N, k, k, C)).astype(np.int8)
    acc, _ = run_conv(B, X, 0.0, Wt, None, None, stride, pad, B.QWT_OUT_INT32_ACC)
    Ho, Wo = Hh, Ww
    M, K = Bn * Ho * Wo, k * k * C
    P = torch.empty((M, K), dtype=torch.int8, device=DEV)
    dX = torch.from_numpy(X).to(DEV)
    B.qwt_im2col_i8(dX, Bn, Hh, Ww, C, k, k, stride, pad, P)
    Y = torch.empty((M, N), dtype=torch.int32, device=DEV)
    wsb = B.qwt_qlinear_workspace_bytes(M, N, K, B.QWT_W_INT8, B.QWT_OUT_INT32_ACC)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device=DEV)
    B.qwt_qlinear_cwac_forward(P, None, torch.from_numpy(Wt.reshape(N, K)).to(DEV), B.QWT_W_INT8, None, None, M, N, K,
                               B.QWT_OUT_INT32_ACC, Y, None, ws, wsb)
    torch.cuda.synchronize()
    assert np.array_equal(acc, Y.cpu().numpy())


def test_implicit_convolution_argument_errors(B):
    x = torch.zeros(1 << 16, dtype=torch.int8, device=DEV)
    f = torch.zeros(256, dtype=torch.float32, device=DEV)
    call = lambda *a, **k: B.qwt_qconv2d_cwac_forward(*a, check=False, **k)
    ok = (x, 0.02, x, f, f, 1, 8, 8, 128, 64, 3, 3, 1, 1, B.QWT_OUT_BF16, x, None, x, 1 << 16)
    assert call(*ok) == B.QWT_OK
    bad = list(ok); bad[8] = 64                        # C % 128
    assert call(*bad) == B.QWT_ERR_UNSUPPORTED
    bad = list(ok); bad[14] = B.QWT_OUT_INT8_STATIC
    assert call(*bad) == B.QWT_ERR_UNSUPPORTED
    bad = list(ok); bad[0] = None
    assert call(*bad) == B.QWT_ERR_NULL
    bad = list(ok); bad[18] = 16
    assert call(*bad) == B.QWT_ERR_WORKSPACE
    bad = list(ok); bad[14] = B.QWT_OUT_INT8_PER_TOKEN     # y_scale missing
    assert call(*bad) == B.QWT_ERR_NULL
    assert B.qwt_qconv2d_workspace_bytes(1, 8, 8, 100, 64, 3, 3, 1, 1, B.QWT_OUT_BF16) == 0
