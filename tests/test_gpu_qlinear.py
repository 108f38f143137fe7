"""GPU parity: the CWAC-fused quantized linear layer against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest

from oracle import qwt_oracle as O
from paper_2505_20932_b200 import workload as WL
from tolerances import assert_bf16_close, assert_codes_close, assert_fp32_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    import gpu_harness
    return gpu_harness


@pytest.fixture(scope="module")
def B():
    from paper_2505_20932_b200 import binding
    return binding


def random_layer(M, N, K, seed, planted=True):
    rng = np.random.default_rng(seed)
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    Wq = rng.integers(-127, 128, (N, K)).astype(np.int8)
    xs = rng.uniform(0.01, 0.05, M).astype(np.float32)
    ws = rng.uniform(1e-4, 3e-4, N).astype(np.float32)
    bias = (0.01 * rng.standard_normal(N)).astype(np.float32)
    a = (1 + 0.05 * rng.standard_normal(N)).astype(np.float32)
    b = (0.02 * rng.standard_normal(N)).astype(np.float32)
    fs64, fb64 = O.cwac_fold(ws, bias, a, b)
    return Xq, Wq, xs, fs64.astype(np.float32), fb64.astype(np.float32)


SHAPES = [
    (128, 128, 128),     # exactly one tile, one k-block
    (128, 256, 256),
    (1, 16, 16),         # smallest legal problem
    (130, 272, 400),     # ragged in M, N and K (K tail of 16 bytes)
    (788, 1536, 384),    # config 1
    (300, 528, 1040),    # several k-blocks with a tail, N tail of 16
    (257, 4096, 512),    # many column tiles per strip
    (2000, 384, 1536),   # more tiles than SMs: second round of the persistent loop
]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_int32_accumulators_bit_exact(H, B, M, N, K):
    Xq, Wq, *_ = random_layer(M, N, K, seed=M + N + K)
    acc, _ = H.gpu_forward(Xq, None, Wq, None, None, B.QWT_OUT_INT32_ACC)
    assert np.array_equal(acc.astype(np.int64), O.int_matmul(Xq, Wq))


def test_int32_extreme_codes(H, B):
    M, N, K = 130, 144, 4096
    Xq = np.full((M, K), 127, np.int8)
    Xq[::2] = -127
    Wq = np.full((N, K), -127, np.int8)
    Wq[::3] = 127
    acc, _ = H.gpu_forward(Xq, None, Wq, None, None, B.QWT_OUT_INT32_ACC)
    assert np.array_equal(acc.astype(np.int64), O.int_matmul(Xq, Wq))
    assert abs(int(acc[0, 0])) == 127 * 127 * K


def test_longest_reduction_stays_inside_int32(H, B):
    """K = 131072, the longest the interface accepts: 127 * 127 * K = 2 114 060 288 < 2^31, with both signs; one more
    k-block of 16 is refused."""
    M, N, K = 130, 144, 131072
    Xq = np.full((M, K), 127, np.int8)
    Xq[1::2] = -127
    Wq = np.full((N, K), 127, np.int8)
    Wq[2::3] = -127
    acc, _ = H.gpu_forward(Xq, None, Wq, None, None, B.QWT_OUT_INT32_ACC)
    assert int(acc[0, 0]) == 127 * 127 * K and int(acc[1, 0]) == -127 * 127 * K and int(acc[1, 2]) == 127 * 127 * K
    assert np.array_equal(acc.astype(np.int64), O.int_matmul(Xq, Wq))
    import torch
    d = H.dev(np.zeros((1, K + 16), np.int8))
    y = torch.zeros(16, dtype=torch.int32, device=H.DEV)
    w = H.dev(np.zeros((16, K + 16), np.int8))
    ws = H.empty_bytes(4096)
    assert B.qwt_qlinear_cwac_forward(d, None, w, B.QWT_W_INT8, None, None, 1, 16, K + 16, B.QWT_OUT_INT32_ACC, y, None,
                                      ws, 4096, check=False) == B.QWT_ERR_SHAPE


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_fp32_output_within_tolerance(H, B, M, N, K):
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=M + N + K + 1)
    z, _ = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_FP32)
    z_ref = O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb)
    assert_fp32_close(z, z_ref)


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_int8_per_token_output(H, B, M, N, K):
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=M + N + K + 2)
    codes, ys = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
    z_ref = O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb)
    c_ref, ys_ref = O.requant_per_token(z_ref)
    assert np.allclose(ys, ys_ref, rtol=1e-5, atol=0)
    assert_codes_close(codes, c_ref)
    # the codes reproduce z to half a step of the row's own scale
    err = np.abs(z_ref - ys[:, None].astype(np.float64) * codes)
    assert np.all(err <= 0.5 * ys[:, None] * (1 + 1e-4) + 1e-6)
    assert codes.min() >= -127


@pytest.mark.parametrize("M,N,K", [(130, 272, 400), (788, 1536, 384), (257, 4096, 512)])
def test_bf16_output(H, B, M, N, K):
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=M + N + K + 3)
    bits, _ = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_BF16)
    z_ref = O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb)
    assert_bf16_close(bits, z_ref, O.to_bf16_bits, O.bf16_bits_to_f32)     # <= 1 bf16 ulp on <= 0.01 % of the elements


def test_zero_rows_and_zero_scale(H, B):
    M, N, K = 140, 160, 128
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=77)
    Xq[5] = 0
    xs[9] = 0.0
    fb[:] = 0.0
    codes, ys = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
    assert ys[5] == 0 and ys[9] == 0 and not codes[5].any() and not codes[9].any()
    c_ref, ys_ref = O.requant_per_token(O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb))
    assert_codes_close(codes, c_ref)


@pytest.mark.parametrize("M,N,K", [(94757, 208, 64), (25088, 256, 128), (19000, 144, 48)])
def test_whole_row_inside_one_tile(H, B, M, N, K):
    """128 < N <= 256 with many rows: a row strip is one 256-wide tile, its two units exchange their row maxima
    inside the CTA (several tiles per CTA, so the exchange buffers and barrier phases alternate)."""
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=M + N)
    codes, ys = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
    c_ref, ys_ref = O.requant_per_token(O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb))
    assert np.allclose(ys, ys_ref, rtol=1e-5)
    assert_codes_close(codes, c_ref)


@pytest.mark.parametrize("M,N,K,own", [(10000, 400, 272, "1"), (10000, 400, 272, "0"), (40000, 512, 64, "1"), (9500, 272, 1040, "1")])
def test_rows_spanning_two_tiles(H, B, M, N, K, own, monkeypatch):
    """256 < N <= 512 with at least half a grid of strips: a CTA takes whole strips and settles the row maxima inside
    itself (several strips per CTA: both exchange buffers and barrier phases); switched off, the same layer goes
    through the exchange between CTAs.  Same results either way."""
    monkeypatch.setenv("QWT_OWN_STRIPS", own)
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=M + N + K)
    codes, ys = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
    c_ref, ys_ref = O.requant_per_token(O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb))
    assert np.allclose(ys, ys_ref, rtol=1e-5)
    assert_codes_close(codes, c_ref)


def test_config1_layer_end_to_end(H, B):
    """Config 1: quantize -> calibrate CWAC on 32 images -> fold -> fused forward, every stage against the oracle."""
    spec = WL.config_layers(1)[0]
    d = WL.host_layer_inputs(spec, seed=0)
    Xq, xs = O.quantize_rows_sym(d["X"], 127)
    Wq, ws = O.quantize_rows_sym(d["W"], 127)
    gXq, gxs = H.gpu_quantize_rows(d["X"], 127)
    gWq, gws = H.gpu_quantize_rows(d["W"], 127)
    assert np.array_equal(gXq, Xq) and np.array_equal(gxs, xs) and np.array_equal(gWq, Wq) and np.array_equal(gws, ws)

    # calibration pair on the 6304 calibration tokens (Section 3.3): Y_full and Y_quant of the same X_in
    Xcq, xcs = O.quantize_rows_sym(d["Xc"], 127)
    q_out = O.dequant(O.int_matmul(Xcq, Wq), xcs, ws, d["bias"])
    fp_out = O.linear_fp(d["Xc"], d["W"], d["bias"])
    gq, _ = H.gpu_forward(Xcq, xcs, Wq, ws, d["bias"], B.QWT_OUT_FP32)     # no CWAC yet: fscale = S_W, fbias = bias
    assert_fp32_close(gq, q_out, "q_out")
    fp32, q32 = fp_out.astype(np.float32), q_out.astype(np.float32)
    a_ref, b_ref, _ = O.cwac_fit(fp32, q32)
    ga, gb, nd = H.gpu_calibrate(fp32, q32)
    from tolerances import assert_ab_close
    assert nd == 0
    assert_ab_close(ga, gb, a_ref, b_ref, np.maximum(np.abs(fp_out.mean(0)), fp_out.std(0)))
    assert 0.99 < a_ref.mean() < 1.01                     # W8A8: the compensation is close to identity

    a32, b32 = a_ref.astype(np.float32), b_ref.astype(np.float32)
    fs_ref, fb_ref = O.cwac_fold(ws, d["bias"], a32, b32)
    gfs, gfb = H.gpu_fold(ws, d["bias"], a32, b32)
    assert np.allclose(gfs, fs_ref, rtol=1e-6) and np.allclose(gfb, fb_ref, rtol=1e-6, atol=1e-9)

    # forward with the folded parameters == unfolded reference (dequant, then CWAC)
    z_unfolded = O.qlinear_cwac_reference(Xq, xs, Wq, ws, d["bias"], a32, b32)
    fs32, fb32 = fs_ref.astype(np.float32), fb_ref.astype(np.float32)
    gz, _ = H.gpu_forward(Xq, xs, Wq, fs32, fb32, B.QWT_OUT_FP32)
    assert_fp32_close(gz, z_unfolded, "z (folded GPU vs unfolded oracle)")
    codes, ys = H.gpu_forward(Xq, xs, Wq, fs32, fb32, B.QWT_OUT_INT8_PER_TOKEN)
    c_ref, ys_ref = O.requant_per_token(O.forward_folded(O.int_matmul(Xq, Wq), xs, fs32, fb32))
    assert np.allclose(ys, ys_ref, rtol=1e-5)
    assert_codes_close(codes, c_ref)
    # CWAC lowers the error against the full-precision layer (what Eq. 3 minimises on the calibration set)
    y_fp = O.linear_fp(d["X"], d["W"], d["bias"])
    y_q = O.dequant(O.int_matmul(Xq, Wq), xs, ws, d["bias"])
    assert np.sum((gz - y_fp) ** 2) <= np.sum((y_q - y_fp) ** 2) * 1.001


def test_forward_from_host_memory(H, B):
    import torch
    M, N, K = 300, 528, 1040
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=5)
    dW, dfs, dfb = H.dev(Wq), H.dev(fs), H.dev(fb)
    Y = np.zeros((M, N), np.int8)
    ys = np.zeros(M, np.float32)
    sb = B.qwt_qlinear_host_staging_bytes(M, N, K, B.QWT_W_INT8, B.QWT_OUT_INT8_PER_TOKEN)
    st = H.empty_bytes(sb)
    B.qwt_qlinear_cwac_forward_host(Xq, xs, dW, B.QWT_W_INT8, dfs, dfb, M, N, K, B.QWT_OUT_INT8_PER_TOKEN, Y, ys, st, sb)
    c_ref, ys_ref = O.requant_per_token(O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb))
    assert np.allclose(ys, ys_ref, rtol=1e-5)
    assert_codes_close(Y, c_ref)


@pytest.mark.parametrize("mode", ["int8", "bf16"])
def test_forward_from_host_memory_in_row_chunks(H, B, mode):
    """More than 4096 rows: the host-buffer call pipelines row chunks over two streams; same bits as one device call."""
    import torch
    M, N, K = 9001, 272, 144
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=8)
    out_mode = B.QWT_OUT_INT8_PER_TOKEN if mode == "int8" else B.QWT_OUT_BF16
    dW, dfs, dfb = H.dev(Wq), H.dev(fs), H.dev(fb)
    hx = torch.from_numpy(Xq).pin_memory()
    hxs = torch.from_numpy(xs).pin_memory()
    hy = torch.zeros((M, N), dtype=torch.int8 if mode == "int8" else torch.bfloat16).pin_memory()
    hys = torch.zeros(M, dtype=torch.float32).pin_memory()
    sb = B.qwt_qlinear_host_staging_bytes(M, N, K, B.QWT_W_INT8, out_mode)
    st = H.empty_bytes(sb)
    st.fill_(0xFF)
    for _ in range(2):          # the second call reuses the helper streams
        B.qwt_qlinear_cwac_forward_host(hx.data_ptr(), hxs.data_ptr(), dW, B.QWT_W_INT8, dfs, dfb, M, N, K, out_mode,
                                        hy.data_ptr(), hys.data_ptr() if mode == "int8" else None, st, sb)
    ref, ys_ref = H.gpu_forward(Xq, xs, Wq, fs, fb, out_mode)
    if mode == "int8":
        assert np.array_equal(hy.numpy(), ref) and np.array_equal(hys.numpy(), ys_ref)
        c_ref, _ = O.requant_per_token(O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb))
        assert_codes_close(hy.numpy(), c_ref)
    else:
        assert np.array_equal(hy.view(torch.int16).numpy().view(np.uint16), ref)


# ------------------------------------------------------------------ packed 4-bit weights (W4A8)

def random_w4_layer(M, N, K, seed):
    rng = np.random.default_rng(seed)
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    Wq = rng.integers(-7, 8, (N, K)).astype(np.int8)
    xs = rng.uniform(0.01, 0.05, M).astype(np.float32)
    ws = rng.uniform(2e-3, 6e-3, N).astype(np.float32)
    bias = (0.01 * rng.standard_normal(N)).astype(np.float32)
    a = (1 + 0.05 * rng.standard_normal(N)).astype(np.float32)
    b = (0.02 * rng.standard_normal(N)).astype(np.float32)
    fs64, fb64 = O.cwac_fold(ws, bias, a, b)
    return Xq, Wq, O.pack_int4(Wq), xs, fs64.astype(np.float32), fb64.astype(np.float32)


W4_SHAPES = [(128, 128, 128), (1, 16, 32), (130, 272, 416), (300, 2304, 768), (500, 768, 3072), (2000, 384, 1536)]


@pytest.mark.parametrize("M,N,K", W4_SHAPES)
def test_w4_int32_accumulators_bit_exact(H, B, M, N, K):
    Xq, Wq, Wp, *_ = random_w4_layer(M, N, K, seed=M + N + K)
    acc, _ = H.gpu_forward(Xq, None, Wp, None, None, B.QWT_OUT_INT32_ACC, wfmt=B.QWT_W_INT4_PACKED, K=K)
    assert np.array_equal(acc.astype(np.int64), O.int_matmul(Xq, Wq))


def test_w4_extreme_codes(H, B):
    M, N, K = 130, 144, 3072
    Xq = np.full((M, K), 127, np.int8)
    Xq[1::2] = -127
    Wq = np.full((N, K), -7, np.int8)
    Wq[::3] = 7
    Wq[:, 1::2] *= -1                                     # even and odd nibbles differ
    acc, _ = H.gpu_forward(Xq, None, O.pack_int4(Wq), None, None, B.QWT_OUT_INT32_ACC, wfmt=B.QWT_W_INT4_PACKED, K=K)
    assert np.array_equal(acc.astype(np.int64), O.int_matmul(Xq, Wq))


@pytest.mark.parametrize("M,N,K", W4_SHAPES)
def test_w4_bf16_fp32_and_int8_outputs(H, B, M, N, K):
    Xq, Wq, Wp, xs, fs, fb = random_w4_layer(M, N, K, seed=M + N + K + 7)
    z_ref = O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb)
    z, _ = H.gpu_forward(Xq, xs, Wp, fs, fb, B.QWT_OUT_FP32, wfmt=B.QWT_W_INT4_PACKED, K=K)
    assert_fp32_close(z, z_ref)
    if N % 8 == 0:
        bits, _ = H.gpu_forward(Xq, xs, Wp, fs, fb, B.QWT_OUT_BF16, wfmt=B.QWT_W_INT4_PACKED, K=K)
        assert_bf16_close(bits, z_ref, O.to_bf16_bits, O.bf16_bits_to_f32)
    codes, ys = H.gpu_forward(Xq, xs, Wp, fs, fb, B.QWT_OUT_INT8_PER_TOKEN, wfmt=B.QWT_W_INT4_PACKED, K=K)
    c_ref, ys_ref = O.requant_per_token(z_ref)
    assert np.allclose(ys, ys_ref, rtol=1e-5)
    assert_codes_close(codes, c_ref)


def test_w4_quantize_pack_forward_chain(H, B):
    """Config 3 shaped layer (one ViT-B fc1 at a reduced token count): W4 per-channel quantizer -> packing -> BF16 forward."""
    spec = WL.LayerSpec("vit_b.fc1", 600, 768, 3072, 4, "bf16", "lognormal_channel", 600)
    d = WL.host_layer_inputs(spec, seed=3)
    Xq, xs = O.quantize_rows_sym(d["X"], 127)
    Wq, ws = O.quantize_rows_sym(d["W"], 7)
    gWq, gws = H.gpu_quantize_rows(d["W"], 7)
    assert np.array_equal(gWq, Wq) and np.array_equal(gws, ws)
    assert np.array_equal(H.gpu_pack_int4(gWq), O.pack_int4(Wq))
    fs, fb = O.cwac_fold(ws, d["bias"], None, None)
    fs, fb = fs.astype(np.float32), fb.astype(np.float32)
    bits, _ = H.gpu_forward(Xq, xs, O.pack_int4(Wq), fs, fb, B.QWT_OUT_BF16, wfmt=B.QWT_W_INT4_PACKED, K=spec.K)
    z_ref = O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb)
    assert_bf16_close(bits, z_ref, O.to_bf16_bits, O.bf16_bits_to_f32)


# ------------------------------------------------------------------ CNN-shaped layers (1x1 convolutions)

def test_resnet50_pointwise_convolutions(H, B):
    """A 1x1 convolution in NHWC layout is the same quantized linear layer (M = B*H*W, K = C_in, N = C_out):
    ResNet-50 bottleneck shapes at a small batch, quantize -> forward in both INT8 modes, against the oracle."""
    for spec in WL.resnet50_pointwise_layers(batch=1, calib_images=1):
        if spec.M > 1600:
            spec = WL.LayerSpec(spec.name, 1600, spec.K, spec.N, 8, "int8", spec.act, 64)
        d = WL.host_layer_inputs(spec, seed=11, calib_rows=8)
        Xq, xs = O.quantize_rows_sym(d["X"], 127)
        Wq, ws = O.quantize_rows_sym(d["W"], 127)
        fs, fb = O.cwac_fold(ws, d["bias"], None, None)
        fs, fb = fs.astype(np.float32), fb.astype(np.float32)
        acc = O.int_matmul(Xq, Wq)
        codes, ys = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
        c_ref, ys_ref = O.requant_per_token(O.forward_folded(acc, xs, fs, fb))
        assert np.allclose(ys, ys_ref, rtol=1e-5), spec.name
        assert_codes_close(codes, c_ref, spec.name)
        raw, _ = H.gpu_forward(Xq, None, Wq, None, None, B.QWT_OUT_INT32_ACC)
        assert np.array_equal(raw.astype(np.int64), acc), spec.name


@pytest.mark.parametrize("Bn,Hh,Ww,C,N,k,stride,pad", [(2, 14, 14, 64, 64, 3, 1, 1), (1, 15, 13, 32, 48, 3, 2, 1),
                                                        (2, 8, 8, 16, 32, 5, 1, 2), (1, 7, 7, 128, 16, 7, 2, 3)])
def test_convolution_through_the_patch_matrix(H, B, Bn, Hh, Ww, C, N, k, stride, pad):
    """k x k convolution = qwt_im2col_i8 + the same forward call with K = k*k*C: raw accumulators against the
    oracle's convolution by definition (bit-exact), then the folded FP32 output with a per-tensor input scale."""
    import torch
    rng = np.random.default_rng(Bn * 1000 + Hh * 10 + k)
    X = rng.integers(-127, 128, (Bn, Hh, Ww, C)).astype(np.int8)
    Wq = rng.integers(-127, 128, (N, k, k, C)).astype(np.int8)
    Ho, Wo = (Hh + 2 * pad - k) // stride + 1, (Ww + 2 * pad - k) // stride + 1
    M, K = Bn * Ho * Wo, k * k * C
    P = torch.full((M, K), 0x5A, dtype=torch.int8, device=H.DEV)
    B.qwt_im2col_i8(H.dev(X), Bn, Hh, Ww, C, k, k, stride, pad, P)
    torch.cuda.synchronize()
    Ph = P.cpu().numpy()
    acc_ref = O.conv2d_int_nhwc(X, Wq, stride, pad).reshape(M, N)
    assert np.array_equal(O.int_matmul(Ph, Wq.reshape(N, K)), acc_ref)          # the patch matrix itself
    acc, _ = H.gpu_forward(Ph, None, Wq.reshape(N, K), None, None, B.QWT_OUT_INT32_ACC)
    assert np.array_equal(acc.astype(np.int64), acc_ref)
    xs = np.full(M, 0.02, np.float32)                                            # per-tensor activation scale
    fs = rng.uniform(1e-4, 3e-4, N).astype(np.float32)
    fb = (0.01 * rng.standard_normal(N)).astype(np.float32)
    z, _ = H.gpu_forward(Ph, xs, Wq.reshape(N, K), fs, fb, B.QWT_OUT_FP32)
    assert_fp32_close(z, O.forward_folded(acc_ref, xs, fs, fb))


@pytest.mark.parametrize("M,N,K,expand", [(300, 2304, 768, "1"), (2000, 384, 1536, "0"), (130, 272, 416, "1")])
def test_w4_both_weight_paths(H, B, M, N, K, expand, monkeypatch):
    """Packed weights are either converted on chip per tile or expanded once into the workspace (the default above
    1024 rows); both paths give the same integers."""
    monkeypatch.setenv("QWT_W4_EXPAND", expand)
    Xq, Wq, Wp, xs, fs, fb = random_w4_layer(M, N, K, seed=M + N + K + 11)
    acc, _ = H.gpu_forward(Xq, None, Wp, None, None, B.QWT_OUT_INT32_ACC, wfmt=B.QWT_W_INT4_PACKED, K=K)
    assert np.array_equal(acc.astype(np.int64), O.int_matmul(Xq, Wq))
    codes, ys = H.gpu_forward(Xq, xs, Wp, fs, fb, B.QWT_OUT_INT8_PER_TOKEN, wfmt=B.QWT_W_INT4_PACKED, K=K)
    c_ref, ys_ref = O.requant_per_token(O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb))
    assert np.allclose(ys, ys_ref, rtol=1e-5)
    assert_codes_close(codes, c_ref)


@pytest.mark.parametrize("M,N,K", [(300, 528, 1040), (256, 256, 128), (128 * 5 + 7, 1024, 400), (3000, 2304, 512)])
def test_cta_pairs_every_output_stage(H, B, M, N, K, monkeypatch):
    """Clusters of two CTAs with MMAs of M = 256 (tcgen05 cta_group::2), forced on for small ragged layers: an odd
    number of row strips (the odd CTA of the last pair then has no rows), N and K tails, several tiles per pair."""
    monkeypatch.setenv("QWT_PAIR", "1")
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=M + N + K + 5)
    acc_ref = O.int_matmul(Xq, Wq)
    z_ref = O.forward_folded(acc_ref, xs, fs, fb)
    acc, _ = H.gpu_forward(Xq, None, Wq, None, None, B.QWT_OUT_INT32_ACC)
    assert np.array_equal(acc.astype(np.int64), acc_ref)
    z, _ = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_FP32)
    assert_fp32_close(z, z_ref)
    bits, _ = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_BF16)
    assert_bf16_close(bits, z_ref, O.to_bf16_bits, O.bf16_bits_to_f32)
    codes, ys = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
    c_ref, ys_ref = O.requant_per_token(z_ref)
    assert np.allclose(ys, ys_ref, rtol=1e-5, atol=0)
    assert_codes_close(codes, c_ref)


@pytest.mark.parametrize("M,N,K,force", [(6221, 1536, 400, "1"), (5117, 1552, 1024, "1"), (6221, 1536, 400, None)])
def test_cta_pairs_with_resident_w_halves(H, B, M, N, K, force, monkeypatch):
    """Short K, many rows, at least six column tiles: every CTA of a pair keeps its half of the pair's W tile in shared
    memory for the whole call and streams X only (a number of pairs that is a multiple of the column tiles, so that a
    pair never changes its column tile).  Ragged M, N and K; K = 1024 takes the instantiation with the narrow staging
    boxes.  Forced on, the per-token INT8 exchange runs over the pairs as well; left to the plan (force None), the
    other output modes take the path by themselves."""
    if force is not None:
        monkeypatch.setenv("QWT_PAIR_RESIDENT", force)
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=M + N + K + 9)
    acc_ref = O.int_matmul(Xq, Wq)
    z_ref = O.forward_folded(acc_ref, xs, fs, fb)
    acc, _ = H.gpu_forward(Xq, None, Wq, None, None, B.QWT_OUT_INT32_ACC)
    assert np.array_equal(acc.astype(np.int64), acc_ref)
    z, _ = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_FP32)
    assert_fp32_close(z, z_ref)
    bits, _ = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_BF16)
    assert_bf16_close(bits, z_ref, O.to_bf16_bits, O.bf16_bits_to_f32)
    codes, ys = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
    c_ref, ys_ref = O.requant_per_token(z_ref)
    assert np.allclose(ys, ys_ref, rtol=1e-5, atol=0)
    assert_codes_close(codes, c_ref)


@pytest.mark.parametrize("M,N,K", [(6221, 1536, 416), (5117, 1552, 1024)])
def test_w4_resident_halves_expanded_on_chip(H, B, M, N, K):
    """Packed weights, many rows, at least six column tiles, short K: the plan runs the int8 pair kernel on W halves that
    every CTA expands once, on chip, from the packed tile (no workspace copy of W).  Ragged M, N and K (a last k-block
    of 32 elements); extreme nibbles in the first rows; every output stage against the oracle."""
    Xq, Wq, Wp, xs, fs, fb = random_w4_layer(M, N, K, seed=M + N + K + 13)
    Wq[:3, :] = np.array([[-7], [7], [0]], np.int8)
    Wq[1, 1::2] = -7                                       # even and odd nibbles differ
    Wp = O.pack_int4(Wq)
    acc_ref = O.int_matmul(Xq, Wq)
    z_ref = O.forward_folded(acc_ref, xs, fs, fb)
    acc, _ = H.gpu_forward(Xq, None, Wp, None, None, B.QWT_OUT_INT32_ACC, wfmt=B.QWT_W_INT4_PACKED, K=K)
    assert np.array_equal(acc.astype(np.int64), acc_ref)
    z, _ = H.gpu_forward(Xq, xs, Wp, fs, fb, B.QWT_OUT_FP32, wfmt=B.QWT_W_INT4_PACKED, K=K)
    assert_fp32_close(z, z_ref)
    bits, _ = H.gpu_forward(Xq, xs, Wp, fs, fb, B.QWT_OUT_BF16, wfmt=B.QWT_W_INT4_PACKED, K=K)
    assert_bf16_close(bits, z_ref, O.to_bf16_bits, O.bf16_bits_to_f32)
    codes, ys = H.gpu_forward(Xq, xs, Wp, fs, fb, B.QWT_OUT_INT8_PER_TOKEN, wfmt=B.QWT_W_INT4_PACKED, K=K)
    c_ref, ys_ref = O.requant_per_token(z_ref)
    assert np.allclose(ys, ys_ref, rtol=1e-5, atol=0)
    assert_codes_close(codes, c_ref)


@pytest.mark.parametrize("M,N,K", [(2600, 4112, 128), (10916, 4112, 800)])
def test_counter_exchange_with_half_empty_last_column_tile(H, B, M, N, K):
    """Per-token INT8 over more than 32 units per row strip (the counter-and-flag exchange) with a last column tile whose
    second unit lies right of the matrix: a group that was handed such a unit takes no part in that exchange, and the
    phases of its exchange barriers must not count it (they once did: the group's next exchange then waited on the
    wrong phase and ran into the wait limit)."""
    Xq, Wq, xs, fs, fb = random_layer(M, N, K, seed=M + N + K + 21)
    z_ref = O.forward_folded(O.int_matmul(Xq, Wq), xs, fs, fb)
    codes, ys = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
    c_ref, ys_ref = O.requant_per_token(z_ref)
    assert np.allclose(ys, ys_ref, rtol=1e-5, atol=0)
    assert_codes_close(codes, c_ref)
