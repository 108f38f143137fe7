"""GPU parity on seeded random layer shapes and calibration problems: the forward plan has many branches (tile width, resident W tile, own strips,
CTA pairs, resident W halves, packed weights on chip or through the workspace, the three row-maximum exchanges, the
two-kernel fallback), chosen from M, N, K, the weight format and the output mode; shapes drawn at random, ragged in every
dimension, walk through them without anybody having picked the edges by hand.  Every case is checked against the oracle."""
import numpy as np
import pytest

from oracle import qwt_oracle as O
from tolerances import assert_ab_close, assert_bf16_close, assert_codes_close, assert_fp32_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    import gpu_harness
    return gpu_harness


@pytest.fixture(scope="module")
def B():
    from paper_2505_20932_b200 import binding
    return binding


def draw_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        big = i % 3 == 0                                   # a third of the cases fill the GPU several times over
        M = int(rng.integers(3000, 9000)) if big else int(rng.integers(1, 1500))
        N = 16 * int(rng.integers(1, 200 if big else 130))   # output rows are 16-byte multiples in every mode
        w4 = bool(rng.integers(0, 2))
        K = (32 if w4 else 16) * int(rng.integers(1, 40 if w4 else 80))
        mode = ("int8", "bf16", "fp32", "acc")[int(rng.integers(0, 4))]
        cases.append((M, N, K, w4, mode))
    return cases


CASES = draw_cases(60, seed=20250520)


@pytest.mark.parametrize("M,N,K,w4,mode", CASES)
def test_random_shape_against_the_oracle(H, B, M, N, K, w4, mode):
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    qmax = 7 if w4 else 127
    Wq = rng.integers(-qmax, qmax + 1, (N, K)).astype(np.int8)
    xs = rng.uniform(0.01, 0.05, M).astype(np.float32)
    ws = rng.uniform(1e-4, 3e-4, N).astype(np.float32) * (127.0 / qmax)
    bias = (0.01 * rng.standard_normal(N)).astype(np.float32)
    a = (1 + 0.05 * rng.standard_normal(N)).astype(np.float32)
    b = (0.02 * rng.standard_normal(N)).astype(np.float32)
    fs64, fb64 = O.cwac_fold(ws, bias, a, b)
    fs, fb = fs64.astype(np.float32), fb64.astype(np.float32)
    W = O.pack_int4(Wq) if w4 else Wq
    kw = dict(wfmt=B.QWT_W_INT4_PACKED, K=K) if w4 else {}
    acc_ref = O.int_matmul(Xq, Wq)
    if mode == "acc":
        acc, _ = H.gpu_forward(Xq, None, W, None, None, B.QWT_OUT_INT32_ACC, **kw)
        assert np.array_equal(acc.astype(np.int64), acc_ref)
        return
    z_ref = O.forward_folded(acc_ref, xs, fs, fb)
    if mode == "fp32":
        z, _ = H.gpu_forward(Xq, xs, W, fs, fb, B.QWT_OUT_FP32, **kw)
        assert_fp32_close(z, z_ref)
    elif mode == "bf16":
        bits, _ = H.gpu_forward(Xq, xs, W, fs, fb, B.QWT_OUT_BF16, **kw)
        assert_bf16_close(bits, z_ref, O.to_bf16_bits, O.bf16_bits_to_f32)
    else:
        codes, ys = H.gpu_forward(Xq, xs, W, fs, fb, B.QWT_OUT_INT8_PER_TOKEN, **kw)
        c_ref, ys_ref = O.requant_per_token(z_ref)
        assert np.allclose(ys, ys_ref, rtol=1e-5, atol=0)
        assert_codes_close(codes, c_ref)


def draw_calibrations(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        rows = int(rng.integers(1, 300)) if i % 4 == 0 else int(rng.integers(300, 60_000))
        C = int(rng.integers(1, 700))
        ld = 4 * ((C + 3) // 4) + 4 * int(rng.integers(0, 3))        # rows of 16-byte multiples, sometimes padded
        out.append((rows, C, ld, int(rng.integers(0, 1 << 30))))
    return out


@pytest.mark.parametrize("rows,C,ld,seed", draw_calibrations(24, seed=5))
def test_random_calibration_against_the_oracle(H, rows, C, ld, seed):
    """Random lengths, channel counts (ragged against the 128-channel slabs) and leading dimensions; per channel a random
    mean (up to a thousand spreads away), spread, slope and noise level, and a few constant channels (Eq. 4's degenerate
    case).  (a, b) and the degenerate count against the oracle's centred two-pass fit."""
    rng = np.random.default_rng(seed)
    mean = rng.standard_normal(C) * 10.0 ** rng.uniform(-2, 3, C)
    spread = 10.0 ** rng.uniform(-2, 1, C)
    q = np.full((rows, ld), 7e29, np.float32)                        # the padding columns must not matter
    f = np.full((rows, ld), -3e29, np.float32)
    q[:, :C] = (mean[None, :] + spread[None, :] * rng.standard_normal((rows, C))).astype(np.float32)
    slope = 1 + 0.1 * rng.standard_normal(C)
    noise = spread * 10.0 ** rng.uniform(-3, -1, C)
    f[:, :C] = (slope[None, :] * q[:, :C].astype(np.float64) + rng.standard_normal(C)[None, :] * spread[None, :] +
                noise[None, :] * rng.standard_normal((rows, C))).astype(np.float32)
    dead = rng.random(C) < 0.03
    q[:, :C][:, dead] = q[0, :C][dead][None, :]
    a, b, nd = H.gpu_calibrate(f, q, channels=C)
    a_ref, b_ref, nd_ref = O.cwac_fit(f[:, :C], q[:, :C])
    assert nd == nd_ref
    f64 = f[:, :C].astype(np.float64)
    assert_ab_close(a, b, a_ref, b_ref, np.maximum(np.abs(f64.mean(0)), f64.std(0)))


def draw_shape(rng):
    kind = rng.integers(0, 4)
    M = int(rng.integers(1, 400)) if kind == 0 else (int(rng.integers(9000, 30000)) if kind == 1 else int(rng.integers(400, 9000)))
    N = 16 * int(rng.integers(1, 130)) if rng.random() < 0.7 else 16 * int(rng.integers(1, 33))
    K = 16 * int(rng.integers(1, 48))
    return M, N, K


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes(H, B, seed):
    """Few to 30 000 rows (one tile, own strips, several tiles per CTA), N from 16 to 2064 (every exchange protocol of the
    per-token INT8 output), K from 16 to 752: per-token INT8 and one other output stage per shape."""
    rng = np.random.default_rng(seed)
    for it in range(10):
        M, N, K = draw_shape(rng)
        Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
        Wq = rng.integers(-127, 128, (N, K)).astype(np.int8)
        xs = rng.uniform(0.01, 0.05, M).astype(np.float32)
        fs = rng.uniform(1e-4, 3e-4, N).astype(np.float32)
        fb = (0.01 * rng.standard_normal(N)).astype(np.float32)
        acc = O.int_matmul(Xq, Wq)
        z = O.forward_folded(acc, xs, fs, fb)
        c_ref, ys_ref = O.requant_per_token(z)
        codes, ys = H.gpu_forward(Xq, xs, Wq, fs, fb, B.QWT_OUT_INT8_PER_TOKEN)
        assert np.allclose(ys, ys_ref, rtol=1e-5), (M, N, K)
        assert_codes_close(codes, c_ref, f"codes {M} x {N} x {K}")
        mode = (B.QWT_OUT_FP32, B.QWT_OUT_BF16, B.QWT_OUT_INT32_ACC)[it % 3]
        y, _ = H.gpu_forward(Xq, xs, Wq, fs, fb, mode)
        if mode == B.QWT_OUT_FP32:
            assert_fp32_close(y, z, f"z {M} x {N} x {K}")
        elif mode == B.QWT_OUT_INT32_ACC:
            assert np.array_equal(y.astype(np.int64), acc), (M, N, K)
        else:
            assert_bf16_close(y, z, O.to_bf16_bits, O.bf16_bits_to_f32, f"bf16 {M} x {N} x {K}")
