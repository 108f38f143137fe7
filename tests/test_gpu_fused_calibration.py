"""GPU parity: CWAC calibration accumulated in the epilogue of the quantized layer (Section 3.3 on Eq. 6-8),
against the oracle's layer followed by the oracle's least-squares fit (through the C ABI)."""
import numpy as np
import pytest

from oracle import qwt_oracle as O
from tolerances import assert_ab_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    import gpu_harness
    return gpu_harness


@pytest.fixture(scope="module")
def B():
    from paper_2505_20932_b200 import binding
    return binding


def layer(M, N, K, seed, qmax_w=127, bias_mean=0.0, ld=None):
    """A float layer, its quantized twin and both outputs on the same M rows."""
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((M, K)).astype(np.float32) * rng.uniform(0.5, 2.0, (M, 1)).astype(np.float32)
    W = (rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32)
    bias = (bias_mean + 0.1 * rng.standard_normal(N)).astype(np.float32)
    Xq, xs = O.quantize_rows_sym(X, 127)
    Wq, ws = O.quantize_rows_sym(W, qmax_w)
    f = O.linear_fp(X, W, bias).astype(np.float32)
    q = O.dequant(O.int_matmul(Xq, Wq), xs, ws, bias)            # float64
    ld = N if ld is None else ld
    fp = np.zeros((M, ld), np.float32)
    fp[:, :N] = f
    fp[:, N:] = 1e30                                             # padding columns must never be read into a sum
    return Xq, xs, Wq, ws, bias, fp, f, q


def nat_scale(f):
    f = f.astype(np.float64)
    return np.maximum(np.abs(f.mean(0)), f.std(0))


SHAPES = [
    (128, 128, 128, 0.0),      # one strip, one unit
    (130, 272, 400, 0.0),      # ragged in M, N and K
    (6304, 384, 384, 0.0),     # config 1's calibration rows on a DeiT-S projection
    (2000, 1536, 384, 5.0),    # channel means far from zero: the shift carries the precision
    (300, 528, 1040, -3.0),
    (257, 4096, 512, 0.0),     # many column tiles per strip
    (20000, 256, 128, 2.0),    # more tiles than CTAs
]


@pytest.mark.parametrize("M,N,K,bm", SHAPES)
def test_fused_calibration_matches_oracle(H, B, M, N, K, bm):
    Xq, xs, Wq, ws, bias, fp, f, q = layer(M, N, K, seed=M + N + K, bias_mean=bm)
    a, b, nd, stats = H.gpu_calibrate_fused(Xq, xs, Wq, ws, bias, fp, stats=np.zeros((5, N)))
    a_ref, b_ref, nd_ref = O.cwac_fit(f, q)
    assert nd == nd_ref == 0
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(f))
    s_ref = O.cwac_stats(f, q)
    assert np.array_equal(stats[0], s_ref[0])
    scale = np.stack([np.abs(q).sum(0), np.abs(f.astype(np.float64)).sum(0), np.abs(q * f).sum(0), (q * q).sum(0)])
    assert np.all(np.abs(stats[1:] - s_ref[1:]) <= 2e-6 * scale + 1e-9)


def test_fused_equals_forward_then_calibrate(H, B):
    """The same q values feed both paths; only the summation order differs."""
    M, N, K = 3000, 768, 384
    Xq, xs, Wq, ws, bias, fp, f, q = layer(M, N, K, seed=3, bias_mean=1.0)
    a1, b1, nd1, _ = H.gpu_calibrate_fused(Xq, xs, Wq, ws, bias, fp)
    gq, _ = H.gpu_forward(Xq, xs, Wq, ws, bias, B.QWT_OUT_FP32)
    a2, b2, nd2 = H.gpu_calibrate(fp, gq)
    assert nd1 == nd2 == 0
    assert np.allclose(a1, a2, rtol=2e-6, atol=0) and np.allclose(b1, b2, rtol=2e-6, atol=1e-6)


def test_fused_packed_int4_weights(H, B):
    M, N, K = 1000, 640, 512
    Xq, xs, Wq, ws, bias, fp, f, q = layer(M, N, K, seed=4, qmax_w=7)
    a, b, nd, _ = H.gpu_calibrate_fused(Xq, xs, H.gpu_pack_int4(Wq), ws, bias, fp, wfmt=B.QWT_W_INT4_PACKED, K=K)
    a_ref, b_ref, _ = O.cwac_fit(f, q)
    assert nd == 0
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(f))
    assert np.abs(a_ref - 1).max() > 1e-3                    # W4: the compensation is not the identity


def test_fused_streaming_and_padding(H, B):
    """Two batches through the running statistics == one call; fp_out with a leading dimension > N; no bias."""
    M, N, K = 1500, 400, 256
    Xq, xs, Wq, ws, bias, fp, f, q = layer(M, N, K, seed=5, ld=416)
    q = q - bias[None, :].astype(np.float64)                 # the layer without its bias
    cut = 700
    _, _, _, st = H.gpu_calibrate_fused(Xq[:cut], xs[:cut], Wq, ws, None, fp[:cut], stats=np.zeros((5, N)), solve=False)
    a, b, nd, st = H.gpu_calibrate_fused(Xq[cut:], xs[cut:], Wq, ws, None, fp[cut:], stats=st)
    a_ref, b_ref, _ = O.cwac_fit(f, q)
    assert nd == 0 and np.all(st[0] == M)
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(f))
    a1, b1, _, _ = H.gpu_calibrate_fused(Xq, xs, Wq, ws, None, fp)
    assert np.allclose(a, a1, rtol=1e-6) and np.allclose(b, b1, rtol=1e-6, atol=1e-7)


def test_fused_reproducible_and_degenerate(H, B):
    M, N, K = 5000, 1152, 384
    Xq, xs, Wq, ws, bias, fp, f, q = layer(M, N, K, seed=6)
    r1 = H.gpu_calibrate_fused(Xq, xs, Wq, ws, bias, fp, stats=np.zeros((5, N)))
    r2 = H.gpu_calibrate_fused(Xq, xs, Wq, ws, bias, fp, stats=np.zeros((5, N)))
    assert np.array_equal(r1[0], r2[0]) and np.array_equal(r1[1], r2[1]) and np.array_equal(r1[3], r2[3])
    # a single row: every channel is degenerate, a = 1 and b = f - q
    a, b, nd, _ = H.gpu_calibrate_fused(Xq[:1], xs[:1], Wq, ws, bias, fp[:1])
    assert nd == N and np.all(a == 1.0)
    assert np.allclose(b, f[0].astype(np.float64) - q[0], rtol=1e-5, atol=1e-6)


def test_fused_argument_errors(H, B):
    import torch
    M, N, K = 128, 128, 128
    Xq, xs, Wq, ws, bias, fp, f, q = layer(M, N, K, seed=7)
    d = H.dev
    args = [d(Xq), d(xs), d(Wq), B.QWT_W_INT8, d(ws), d(bias), d(fp), N, M, N, K, None]
    a = torch.empty(N, device=H.DEV)
    wsb = B.qwt_qlinear_cwac_calibrate_workspace_bytes(M, N, K, B.QWT_W_INT8)
    w = H.empty_bytes(wsb)
    assert B.qwt_qlinear_cwac_calibrate(*args, None, None, None, w, wsb, check=False) == B.QWT_ERR_NULL
    assert B.qwt_qlinear_cwac_calibrate(*args, a, None, None, w, wsb, check=False) == B.QWT_ERR_NULL
    assert B.qwt_qlinear_cwac_calibrate(*args, a, a.clone(), None, w, wsb - 1, check=False) == B.QWT_ERR_WORKSPACE
    bad = list(args)
    bad[7] = N - 4                                            # ld < N
    assert B.qwt_qlinear_cwac_calibrate(*bad, a, a.clone(), None, w, wsb, check=False) == B.QWT_ERR_SHAPE


def test_fused_resident_weights_many_tiles_per_cta(H, B):
    """One column tile, W resident in shared memory, six row strips per CTA: a group's warps reuse their staging slots
    unit after unit without the parameter slice ever being reloaded.  Every channel against the oracle's sums, and two
    runs on the same input bit for bit."""
    M, N, K = 128 * 148 * 6 - 40, 256, 128
    Xq, xs, Wq, ws, bias, fp, f, q = layer(M, N, K, seed=8, bias_mean=0.5)
    r1 = H.gpu_calibrate_fused(Xq, xs, Wq, ws, bias, fp, stats=np.zeros((5, N)))
    r2 = H.gpu_calibrate_fused(Xq, xs, Wq, ws, bias, fp, stats=np.zeros((5, N)))
    assert np.array_equal(r1[0], r2[0]) and np.array_equal(r1[1], r2[1]) and np.array_equal(r1[3], r2[3])
    a_ref, b_ref, nd_ref = O.cwac_fit(f, q)
    assert r1[2] == nd_ref == 0
    assert_ab_close(r1[0], r1[1], a_ref, b_ref, nat_scale(f))
    s_ref = O.cwac_stats(f, q)
    scale = np.stack([np.abs(q).sum(0), np.abs(f.astype(np.float64)).sum(0), np.abs(q * f).sum(0), (q * q).sum(0)])
    assert np.array_equal(r1[3][0], s_ref[0])
    assert np.all(np.abs(r1[3][1:] - s_ref[1:]) <= 2e-6 * scale + 1e-9)


def test_fused_channel_means_far_above_their_spread(H, B):
    """|mean| / std of the layer's output around 1e4 (a large bias on a unit-spread product): the variance is then a
    difference of sums that agree to eight digits, which the shifted sums never form.  (At this ratio the fit is
    already sensitive to the FP32 rounding of q itself -- steps of 1e-3 at 1e4 -- so the oracle fits the FP32 values
    of its own q, as the layer's FP32 output stage would deliver them; a ratio of 3e4 moves b by its whole tolerance
    when sixteen of a million q values round the other way.)"""
    M, N, K = 4000, 256, 256
    Xq, xs, Wq, ws, bias, fp, f, q = layer(M, N, K, seed=9, bias_mean=1.0e4)
    a, b, nd, _ = H.gpu_calibrate_fused(Xq, xs, Wq, ws, bias, fp)
    a_ref, b_ref, nd_ref = O.cwac_fit(f, q.astype(np.float32))
    assert nd == nd_ref == 0
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(f))
