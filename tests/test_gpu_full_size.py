"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times
(device-resident inputs, the library's own plan for these shapes).  Where the oracle cannot evaluate a whole
output in seconds it evaluates sampled rows (whole rows: the per-token scale depends on the complete row) or
sampled channels (calibration is independent per channel)."""
import numpy as np
import pytest
import torch

from oracle import qwt_oracle as O
from paper_2505_20932_b200 import workload as WL
from tolerances import assert_ab_close, assert_bf16_close, assert_codes_close, assert_fp32_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def B():
    from paper_2505_20932_b200 import binding
    return binding


def quant_rows(B, X, qmax):
    r, c = X.shape
    q = torch.empty((r, c), dtype=torch.int8, device=DEV)
    s = torch.empty(r, dtype=torch.float32, device=DEV)
    B.qwt_quantize_rows_i8(X, r, c, c, qmax, q, s)
    return q, s


def recipe_layer(B, spec, seed):
    """Device inputs of one layer of a benchmark configuration, drawn and prepared the way bench.py prepares them:
    the configuration's activation recipe and weights (workload.py), quantized by the library's row quantizer, packed
    for 4-bit weights, with a seeded compensation (a ~ N(1, 0.05), b ~ N(0, 0.02)) folded in by qwt_cwac_fold.
    Returns device tensors (Xq, xs, W as passed to the library, Wq codes, fs, fb)."""
    X = WL.device_activations(spec.act, spec.M, spec.K, seed, spec.name + "|infer", DEV)
    Xq, xs = quant_rows(B, X, 127)
    del X
    Wf = WL.device_weights(spec.N, spec.K, seed, spec.name, device=DEV)
    Wq, w_scale = quant_rows(B, Wf, 127 if spec.w_bits == 8 else 7)
    del Wf
    W = Wq
    if spec.w_bits == 4:
        W = torch.empty((spec.N, spec.K // 2), dtype=torch.uint8, device=DEV)
        B.qwt_pack_int4(Wq, spec.N, spec.K, W)
    a, b = WL.host_planted_cwac(spec.N, seed, spec.name)
    bias = torch.from_numpy(WL.host_bias(spec.N, seed, spec.name)).to(DEV)
    fs = torch.empty(spec.N, dtype=torch.float32, device=DEV)
    fb = torch.empty(spec.N, dtype=torch.float32, device=DEV)
    B.qwt_cwac_fold(w_scale, bias, torch.from_numpy(a).to(DEV), torch.from_numpy(b).to(DEV), spec.N, fs, fb)
    torch.cuda.synchronize()
    return Xq, xs, W, Wq, fs, fb


def run_forward(B, Xq, xs, W, fs, fb, mode, wfmt, K):
    M, N = Xq.shape[0], W.shape[0]
    dt = {B.QWT_OUT_INT8_PER_TOKEN: torch.int8, B.QWT_OUT_BF16: torch.bfloat16}[mode]
    Y = torch.empty((M, N), dtype=dt, device=DEV)
    ys = torch.empty(M, dtype=torch.float32, device=DEV)
    wsb = B.qwt_qlinear_workspace_bytes(M, N, K, wfmt, mode)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device=DEV)
    for _ in range(2):      # twice on the same workspace, as the benchmark does
        B.qwt_qlinear_cwac_forward(Xq, xs, W, wfmt, fs, fb, M, N, K, mode, Y, ys if mode == B.QWT_OUT_INT8_PER_TOKEN else None,
                                   ws, wsb)
    B.qwt_qlinear_check_status(ws)
    return Y, ys


def sample_rows(M, seed, n=64):
    return np.unique(np.concatenate([np.random.default_rng(seed).integers(0, M, n), [0, 127, 128, M - 1]]))


def oracle_rows(Xq, xs, Wq, fs, fb, rows=None):
    """The oracle's compensated output z (float64) for whole rows of the layer (all rows when rows is None)."""
    if rows is not None:
        rt = torch.from_numpy(rows).to(DEV)
        Xq, xs = Xq[rt], xs[rt]
    return O.forward_folded(O.int_matmul(Xq.cpu().numpy(), Wq.cpu().numpy()), xs.cpu().numpy(), fs.cpu().numpy(),
                            fb.cpu().numpy())


@pytest.mark.parametrize("layer", [0, 1, 2, 3])
def test_config2_layers_whole_output(B, layer):
    """DeiT-S block (qkv, proj, fc1, fc2) at 64 x 197 tokens, LogNormal channel scales: every code and every scale."""
    spec = WL.config_layers(2)[layer]
    Xq, xs, W, Wq, fs, fb = recipe_layer(B, spec, seed=layer)
    Y, ys = run_forward(B, Xq, xs, W, fs, fb, B.QWT_OUT_INT8_PER_TOKEN, B.QWT_W_INT8, spec.K)
    c_ref, ys_ref = O.requant_per_token(oracle_rows(Xq, xs, Wq, fs, fb))
    assert np.allclose(ys.cpu().numpy(), ys_ref, rtol=1e-5)
    assert_codes_close(Y.cpu().numpy(), c_ref)


@pytest.mark.parametrize("layer", [0, 4, 6, 7, 11, 13])
def test_config4_layers_sampled_rows(B, layer):
    """LLaMA-7B shaped layers (q, gate, down at 2048 and 8192 tokens), 0.1 % of the input channels x 50."""
    spec = WL.config_layers(4)[layer]
    Xq, xs, W, Wq, fs, fb = recipe_layer(B, spec, seed=40 + layer)
    Y, ys = run_forward(B, Xq, xs, W, fs, fb, B.QWT_OUT_INT8_PER_TOKEN, B.QWT_W_INT8, spec.K)
    rows = sample_rows(spec.M, 5)
    rt = torch.from_numpy(rows).to(DEV)
    c_ref, ys_ref = O.requant_per_token(oracle_rows(Xq, xs, Wq, fs, fb, rows))
    assert np.allclose(ys[rt].cpu().numpy(), ys_ref, rtol=1e-5)
    assert_codes_close(Y[rt].cpu().numpy(), c_ref)
    # properties that hold for every row: the scale is positive and every row reaches an end code
    assert bool((ys > 0).all()) and bool((Y.abs().amax(dim=1) == 127).all())


@pytest.mark.parametrize("w4_path", ["default", "pairs", "single_cta"])
@pytest.mark.parametrize("layer", [0, 1, 2, 3])
def test_config3_layers_sampled_rows_w4_bf16(B, layer, w4_path, monkeypatch):
    """ViT-B block at 128 x 197 tokens, packed 4-bit weights, BF16 output, through the three weight paths: the plan's
    own choice for this many rows (the weights expanded once per call into the workspace), nibbles expanded in shared
    memory by the converter warps of CTA pairs, each CTA its half of the W tile (QWT_W4_EXPAND=0), and the same
    expansion by single CTAs (QWT_W4_EXPAND=0, QWT_PAIR=0)."""
    monkeypatch.delenv("QWT_W4_EXPAND", raising=False)
    monkeypatch.delenv("QWT_PAIR", raising=False)
    if w4_path != "default":
        monkeypatch.setenv("QWT_W4_EXPAND", "0")
    if w4_path == "single_cta":
        monkeypatch.setenv("QWT_PAIR", "0")
    spec = WL.config_layers(3)[layer]
    Xq, xs, W, Wq, fs, fb = recipe_layer(B, spec, seed=30 + layer)
    Y, _ = run_forward(B, Xq, xs, W, fs, fb, B.QWT_OUT_BF16, B.QWT_W_INT4_PACKED, spec.K)
    rows = sample_rows(spec.M, 6)
    rt = torch.from_numpy(rows).to(DEV)
    z = oracle_rows(Xq, xs, Wq, fs, fb, rows)
    bits = Y[rt].view(torch.int16).cpu().numpy().view(np.uint16)
    assert_bf16_close(bits, z, O.to_bf16_bits, O.bf16_bits_to_f32)


@pytest.mark.parametrize("R,layer,noise", [(128 * 2048, 0, 0.0), (128 * 2048, 0, 0.01), (32768, 4, 0.0)])
def test_config4_calibration_planted_and_refit(B, R, layer, noise):
    """Config 4's calibration leg: q_out is the layer's own FP32 output on the calibration tokens (spot-checked against
    the oracle), fp_out = a* q_out + b* (+ noise of 1 % of the channel's spread).  Without noise the refit must return
    the planted pair; with or without, sampled channels must match the oracle's fit of the same two matrices.
    q (4096 wide) at the config's 262 144 rows; gate (11 008 wide) at 32 768 rows."""
    spec = WL.config_layers(4)[layer]
    N, K = spec.N, spec.K
    seed = 400 + layer
    Xc = WL.device_activations(spec.act, R, K, seed, spec.name + "|calib", DEV)
    Xq, xs = quant_rows(B, Xc, 127)
    del Xc
    Wf = WL.device_weights(N, K, seed, spec.name, device=DEV)
    Wq, w_scale = quant_rows(B, Wf, 127)
    del Wf
    bias = torch.from_numpy(WL.host_bias(N, seed, spec.name)).to(DEV)
    q_out = torch.empty((R, N), dtype=torch.float32, device=DEV)
    wsb = B.qwt_qlinear_workspace_bytes(R, N, K, B.QWT_W_INT8, B.QWT_OUT_FP32)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device=DEV)
    B.qwt_qlinear_cwac_forward(Xq, xs, Wq, B.QWT_W_INT8, w_scale, bias, R, N, K, B.QWT_OUT_FP32, q_out, None, ws, wsb)
    B.qwt_qlinear_check_status(ws)
    rows = sample_rows(R, 8, 12)
    rt = torch.from_numpy(rows).to(DEV)
    q_ref = O.dequant(O.int_matmul(Xq[rt].cpu().numpy(), Wq.cpu().numpy()), xs[rt].cpu().numpy(), w_scale.cpu().numpy(),
                      bias.cpu().numpy())
    assert_fp32_close(q_out[rt].cpu().numpy(), q_ref, "q_out")
    del Xq, xs
    a_star, b_star = WL.host_planted_cwac(N, seed, spec.name)
    fp = q_out * torch.from_numpy(a_star).to(DEV)[None, :]
    fp += torch.from_numpy(b_star).to(DEV)[None, :]
    if noise > 0:
        g = torch.Generator(device=DEV)
        g.manual_seed(seed)
        sd = q_out[:8192].std(dim=0)
        for r0 in range(0, R, 32768):
            r1 = min(R, r0 + 32768)
            fp[r0:r1] += torch.randn((r1 - r0, N), generator=g, device=DEV) * (noise * sd)[None, :]
    a = torch.empty(N, dtype=torch.float32, device=DEV)
    b = torch.empty(N, dtype=torch.float32, device=DEV)
    nd = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    cwsb = B.qwt_cwac_workspace_bytes(R, N)
    cws = torch.empty(max(cwsb, 256), dtype=torch.uint8, device=DEV)
    B.qwt_cwac_calibrate(fp, q_out, R, N, N, a, b, nd, cws, cwsb)
    torch.cuda.synchronize()
    assert int(nd.item()) == 0
    ah, bh = a.cpu().numpy(), b.cpu().numpy()
    ch = np.unique(np.concatenate([np.random.default_rng(9).integers(0, N, 40), [0, 127, 128, N - 1]]))
    ct = torch.from_numpy(ch).to(DEV)
    fph, qh = fp[:, ct].cpu().numpy(), q_out[:, ct].cpu().numpy()
    scale = np.maximum(np.abs(fph.astype(np.float64).mean(0)), fph.astype(np.float64).std(0))
    a_ref, b_ref, _ = O.cwac_fit(fph, qh)
    assert_ab_close(ah[ch], bh[ch], a_ref, b_ref, scale)
    if noise == 0:
        # every channel against the planted pair (fp_out carries one FP32 rounding per element of a* q + b*)
        sd_all = (q_out[:32768].double().std(dim=0) * torch.from_numpy(np.abs(a_star)).to(DEV)).cpu().numpy()
        assert_ab_close(ah, bh, a_star, b_star, np.maximum(sd_all, np.abs(b_star)))
    else:
        assert np.abs(ah - a_star).max() < 5e-3 and np.abs(a_ref - a_star[ch]).max() < 5e-3


def test_very_wide_layer_takes_the_two_kernel_path(B):
    """More column tiles than the persistent grid has CTAs (N > 148 x 256): the layer's FP32 output goes through
    scratch in the workspace and the row quantizer writes codes and scales."""
    M, N, K = 100, 148 * 256 + 48, 64
    g = torch.Generator(device=DEV)
    g.manual_seed(77)
    Xq = torch.randint(-127, 128, (M, K), generator=g, device=DEV, dtype=torch.int8)
    Wq = torch.randint(-127, 128, (N, K), generator=g, device=DEV, dtype=torch.int8)
    xs = torch.rand(M, generator=g, device=DEV) * 0.04 + 0.01
    fs = torch.rand(N, generator=g, device=DEV) * 2e-4 + 1e-4
    fb = torch.randn(N, generator=g, device=DEV) * 0.01
    assert B.qwt_qlinear_workspace_bytes(M, N, K, B.QWT_W_INT8, B.QWT_OUT_INT8_PER_TOKEN) >= 4 * M * N   # the FP32 scratch
    B.qwt_launch_count_reset()
    Y, ys = run_forward(B, Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN, B.QWT_W_INT8, K)
    assert B.qwt_launch_count() == 4                # two calls x (layer kernel + row quantizer)
    c_ref, ys_ref = O.requant_per_token(oracle_rows(Xq, xs, Wq, fs, fb))
    assert np.allclose(ys.cpu().numpy(), ys_ref, rtol=1e-5)
    assert_codes_close(Y.cpu().numpy(), c_ref)


@pytest.mark.parametrize("C,bits", [(768, 4), (3072, 8)])
def test_config5_calibration_sampled_channels(B, C, bits):
    R = WL.CALIB_SWEEP_ROWS                       # 403,456 rows
    fp, q, sig = WL.device_calib_pair(R, C, bits, seed=0, device=DEV)
    a = torch.empty(C, dtype=torch.float32, device=DEV)
    b = torch.empty(C, dtype=torch.float32, device=DEV)
    wsb = B.qwt_cwac_workspace_bytes(R, C)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device=DEV)
    B.qwt_cwac_calibrate(fp, q, R, C, C, a, b, None, ws, wsb)
    torch.cuda.synchronize()
    ch = np.unique(np.concatenate([np.random.default_rng(7).integers(0, C, 40), [0, 127, 128, C - 1]]))
    ct = torch.from_numpy(ch).to(DEV)
    fph, qh = fp[:, ct].cpu().numpy(), q[:, ct].cpu().numpy()
    a_ref, b_ref, nd = O.cwac_fit(fph, qh)
    assert nd == 0
    assert_ab_close(a[ct].cpu().numpy(), b[ct].cpu().numpy(), a_ref, b_ref, np.maximum(np.abs(fph.mean(0)), fph.std(0)))
    # every channel: the closed form for independent uniform noise, a = s^2 / (s^2 + D^2 / 12) with D = 8 s / (2^b - 1)
    expect = 1.0 / (1.0 + (8.0 / (2 ** bits - 1)) ** 2 / 12.0)
    assert np.abs(a.cpu().numpy() - expect).max() < 6.0 / np.sqrt(R) * (1.2 if bits == 4 else 0.1) + 1e-4
    assert np.abs(b.cpu().numpy() / sig).max() < 6.0 / np.sqrt(R)


def test_config2_fused_calibration_sampled_channels(B):
    """Calibration inside the layer at config 2's calibration size (512 images x 197 tokens, the qkv projection):
    the oracle recomputes the quantized layer for sampled channels and fits them against the same fp_out."""
    M, N, K = 512 * 197, 1152, 384
    g = torch.Generator(device=DEV)
    g.manual_seed(11)
    Xq = torch.randint(-127, 128, (M, K), generator=g, device=DEV, dtype=torch.int8)
    Wq = torch.randint(-127, 128, (N, K), generator=g, device=DEV, dtype=torch.int8)
    xs = torch.rand(M, generator=g, device=DEV) * 0.04 + 0.01
    ws = torch.rand(N, generator=g, device=DEV) * 2e-4 + 1e-4
    bias = torch.randn(N, generator=g, device=DEV) * 0.5 + 1.0
    # a synthetic "full-precision" output: a per-channel affine image of the integer product plus noise
    # (built from float arithmetic of the inputs only, never from the library's own q)
    gain = 1.0 + 0.05 * torch.randn(N, generator=g, device=DEV)
    fp = torch.empty((M, N), dtype=torch.float32, device=DEV)
    for r0 in range(0, M, 16384):
        r1 = min(M, r0 + 16384)
        acc = Xq[r0:r1].float() @ Wq.float().t()                       # exact: |acc| < 2^24
        fp[r0:r1] = (acc * xs[r0:r1, None] * ws[None, :] + bias[None, :]) * gain[None, :]
        fp[r0:r1] += 0.02 * torch.randn((r1 - r0, N), generator=g, device=DEV)
    a = torch.empty(N, dtype=torch.float32, device=DEV)
    b = torch.empty(N, dtype=torch.float32, device=DEV)
    nd = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    wsb = B.qwt_qlinear_cwac_calibrate_workspace_bytes(M, N, K, B.QWT_W_INT8)
    wsp = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    B.qwt_qlinear_cwac_calibrate(Xq, xs, Wq, B.QWT_W_INT8, ws, bias, fp, N, M, N, K, None, a, b, nd, wsp, wsb)
    B.qwt_qlinear_check_status(wsp)
    assert int(nd.item()) == 0
    ch = np.unique(np.concatenate([np.random.default_rng(5).integers(0, N, 24), [0, 127, 128, 255, 256, N - 1]]))
    ct = torch.from_numpy(ch).to(DEV)
    q = O.dequant(O.int_matmul(Xq.cpu().numpy(), Wq[ct].cpu().numpy()), xs.cpu().numpy(), ws[ct].cpu().numpy(),
                  bias[ct].cpu().numpy())
    fph = fp[:, ct].cpu().numpy()
    a_ref, b_ref, _ = O.cwac_fit(fph, q)
    assert_ab_close(a[ct].cpu().numpy(), b[ct].cpu().numpy(), a_ref, b_ref, np.maximum(np.abs(fph.mean(0)), fph.std(0)))
    assert np.abs(a_ref - gain[ct].cpu().numpy()).max() < 0.01       # the planted per-channel gain is what the fit finds
