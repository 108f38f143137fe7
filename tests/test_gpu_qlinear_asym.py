"""GPU parity of the layer with asymmetric (unsigned) codes and non-zero zero-points -- Eq. 1-2 and Eq. 6-7 as
printed -- against the CPU oracle, through the C ABI."""
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


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def gpu_quantize_u8(B, X):
    r, c = X.shape
    q = torch.empty((r, c), dtype=torch.uint8, device=DEV)
    s = torch.empty(r, dtype=torch.float32, device=DEV)
    z = torch.empty(r, dtype=torch.int32, device=DEV)
    rs = torch.empty(r, dtype=torch.int32, device=DEV)
    B.qwt_quantize_rows_u8(dev(X), r, c, c, q, s, z, rs)
    torch.cuda.synchronize()
    return q.cpu().numpy(), s.cpu().numpy(), z.cpu().numpy(), rs.cpu().numpy()


def gpu_forward_asym(B, Xq, xs, xz, Wq, wz, fs, fb, mode):
    M, K = Xq.shape
    N = Wq.shape[0]
    dt = {B.QWT_OUT_INT8_PER_TOKEN: torch.int8, B.QWT_OUT_BF16: torch.bfloat16, B.QWT_OUT_FP32: torch.float32,
          B.QWT_OUT_INT32_ACC: torch.int32}[mode]
    dW = dev(Wq)
    terms = torch.empty(2 * N, dtype=torch.int32, device=DEV)
    B.qwt_asym_weight_terms(dW, dev(wz.astype(np.int32)), N, K, terms)
    rs = dev(Xq.astype(np.int64).sum(axis=1).astype(np.int32))
    Y = torch.empty((M, N), dtype=dt, device=DEV)
    ys = torch.empty(M, dtype=torch.float32, device=DEV)
    wsb = B.qwt_qlinear_workspace_bytes(M, N, K, B.QWT_W_INT8, mode)
    ws = torch.full((max(wsb, 256),), 0xFF, dtype=torch.uint8, device=DEV)
    B.qwt_qlinear_cwac_forward_asym(dev(Xq), None if xs is None else dev(xs), dev(xz.astype(np.int32)), rs, dW, terms,
                                    None if fs is None else dev(fs), None if fb is None else dev(fb), M, N, K, mode, Y,
                                    ys if mode == B.QWT_OUT_INT8_PER_TOKEN else None, ws, wsb)
    B.qwt_qlinear_check_status(ws)
    t = terms.cpu().numpy()
    assert np.array_equal(t[:N], -wz) and np.array_equal(t[N:], K * wz - Wq.astype(np.int64).sum(axis=1))
    return Y, ys


def test_rowwise_asymmetric_quantizer_matches_the_oracle(B):
    rng = np.random.default_rng(41)
    X = (rng.standard_normal((300, 400)) * rng.lognormal(0, 1, (300, 1)) + rng.normal(0, 1, (300, 1))).astype(np.float32)
    X[7] = 2.5                                            # constant row
    q, s, z, rs = gpu_quantize_u8(B, X)
    q_ref, s_ref, z_ref = O.quantize_rows_asym(X)
    assert np.array_equal(s, s_ref) and np.array_equal(z, z_ref) and np.array_equal(q, q_ref)
    assert np.array_equal(rs, q_ref.astype(np.int64).sum(axis=1))


SHAPES = [(128, 256, 256), (1, 16, 16), (130, 272, 400), (788, 1536, 384), (257, 4096, 512), (2000, 384, 1536)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_eq7_accumulators_bit_exact(B, M, N, K):
    rng = np.random.default_rng(M + N + K)
    Xq = rng.integers(0, 256, (M, K)).astype(np.uint8)
    Wq = rng.integers(0, 256, (N, K)).astype(np.uint8)
    xz = rng.integers(0, 256, M)
    wz = rng.integers(0, 256, N)
    Y, _ = gpu_forward_asym(B, Xq, None, xz, Wq, wz, None, None, B.QWT_OUT_INT32_ACC)
    assert np.array_equal(Y.cpu().numpy().astype(np.int64), O.int_matmul_asym(Xq, xz, Wq, wz))


def test_eq7_extreme_codes(B):
    M, N, K = 130, 144, 4096
    Xq = np.full((M, K), 255, np.uint8)
    Wq = np.full((N, K), 255, np.uint8)
    Y, _ = gpu_forward_asym(B, Xq, None, np.zeros(M, int), Wq, np.zeros(N, int), None, None, B.QWT_OUT_INT32_ACC)
    assert int(Y[0, 0]) == 255 * 255 * K
    Y, _ = gpu_forward_asym(B, Xq, None, np.full(M, 255), Wq, np.full(N, 128), None, None, B.QWT_OUT_INT32_ACC)
    assert not Y.cpu().numpy().any()                      # (x_q - Z_x) = 0 everywhere


@pytest.mark.parametrize("M,N,K", [(130, 272, 400), (788, 1536, 384), (2000, 384, 1536)])
def test_asymmetric_layer_end_to_end(B, M, N, K):
    """Quantize activations per token and weights per channel with Eq. 1-2, run the layer with folded CWAC in the
    FP32, BF16 and per-token INT8 output stages, compare with the oracle evaluated from Eq. 6's definition."""
    rng = np.random.default_rng(M + N)
    X = (rng.standard_normal((M, K)) * rng.lognormal(0, 0.5, (1, K)) + 0.3).astype(np.float32)
    W = (0.02 * rng.standard_normal((N, K))).astype(np.float32)
    xq, xs, xz = O.quantize_rows_asym(X)
    wq, ws, wz = O.quantize_rows_asym(W)
    bias = (0.01 * rng.standard_normal(N)).astype(np.float32)
    a = (1 + 0.05 * rng.standard_normal(N)).astype(np.float32)
    b = (0.02 * rng.standard_normal(N)).astype(np.float32)
    fs64, fb64 = O.cwac_fold(ws, bias, a, b)
    fs, fb = fs64.astype(np.float32), fb64.astype(np.float32)
    acc = O.int_matmul_asym(xq, xz, wq, wz)
    z_ref = O.forward_folded(acc, xs, fs, fb)
    # the quantized layer approximates the full-precision one (Eq. 6)
    y_fp = O.cwac_apply(O.linear_fp(X, W, bias), a, b)
    assert np.abs(z_ref - y_fp).max() < 0.05 * np.abs(y_fp).max()
    Y, _ = gpu_forward_asym(B, xq, xs, xz, wq, wz, fs, fb, B.QWT_OUT_FP32)
    assert_fp32_close(Y.cpu().numpy(), z_ref)
    Y, _ = gpu_forward_asym(B, xq, xs, xz, wq, wz, fs, fb, B.QWT_OUT_BF16)
    assert_bf16_close(Y.view(torch.int16).cpu().numpy().view(np.uint16), z_ref, O.to_bf16_bits, O.bf16_bits_to_f32)
    Y, ys = gpu_forward_asym(B, xq, xs, xz, wq, wz, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
    c_ref, ys_ref = O.requant_per_token(z_ref)
    assert np.allclose(ys.cpu().numpy(), ys_ref, rtol=1e-5)
    assert_codes_close(Y.cpu().numpy(), c_ref)
