"""GPU parity of the static-scale form of the folded layer (Section 3.4, Eq. 10-11 as printed): integer accumulator
offset + per-channel multiplier, against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

from oracle import qwt_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    import gpu_harness
    return gpu_harness


@pytest.fixture(scope="module")
def B():
    from paper_2505_20932_b200 import binding
    return binding


def layer(M, N, K, seed, w_bits=8):
    rng = np.random.default_rng(seed)
    qmax = 127 if w_bits == 8 else 7
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    Wq = rng.integers(-qmax, qmax + 1, (N, K)).astype(np.int8)
    ws = rng.uniform(1e-4, 3e-4, N).astype(np.float32) * (127 // qmax)
    bias = (0.01 * rng.standard_normal(N)).astype(np.float32)
    a = (1 + 0.05 * rng.standard_normal(N)).astype(np.float32)
    b = (0.02 * rng.standard_normal(N)).astype(np.float32)
    S_x = np.float32(0.03)
    # output scale: the compensated output's spread / 127 over the whole tensor, so a few elements clip
    acc = O.int_matmul(Xq[: min(M, 64)], Wq)
    real = a.astype(np.float64) * (acc * float(S_x) * ws.astype(np.float64) + bias) + b
    S_r = np.float32(np.abs(real).max() / 127.0 * 0.9)
    return Xq, Wq, ws, bias, a, b, S_x, S_r


def oracle_fold(ws, bias, a, b, S_x, S_r):
    beta = a.astype(np.float64) * bias.astype(np.float64) + b.astype(np.float64)
    return O.fold_integer_offset(a, beta, float(S_x), ws, float(S_r))


SHAPES = [(128, 256, 256), (1, 16, 16), (130, 272, 400), (788, 1536, 384), (257, 4096, 512), (2000, 384, 1536)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_fold_static_and_forward_match_the_oracle(H, B, M, N, K):
    Xq, Wq, ws, bias, a, b, S_x, S_r = layer(M, N, K, seed=M + N + K)
    Mp_ref, off_ref = oracle_fold(ws, bias, a, b, S_x, S_r)
    mult, off = H.gpu_fold_static(ws, bias, a, b, S_x, S_r)
    assert np.allclose(mult, Mp_ref, rtol=2e-7, atol=0)
    # the offset is a rounded float64 quotient: equal, except where the quotient sits on a rounding tie
    beta = a.astype(np.float64) * bias.astype(np.float64) + b.astype(np.float64)
    quo = beta / (a.astype(np.float64) * float(S_x) * ws.astype(np.float64))
    tie = np.abs(quo - np.floor(quo) - 0.5) < 1e-9
    assert np.array_equal(off[~tie], off_ref[~tie]) and np.abs(off - off_ref).max() <= 1
    assert np.abs(off).mean() > 20                      # the offsets are large, as Section 3.4 remarks
    # forward with the GPU's own fold: bit-exact codes (integer sum, one FP32 product, round, clip)
    codes, _ = H.gpu_forward(Xq, None, Wq, mult, off, B.QWT_OUT_INT8_STATIC)
    ref = O.requant_static(O.int_matmul(Xq, Wq), mult, off)
    assert np.array_equal(codes, ref)
    assert (np.abs(ref) == 127).any() and codes.min() >= -127      # the case does clip somewhere


def test_static_codes_track_the_compensated_output(H, B):
    """S_r * codes stays within half an output step plus half an accumulator step of the unfolded Eq. 9 value."""
    M, N, K = 300, 528, 1040
    Xq, Wq, ws, bias, a, b, S_x, S_r = layer(M, N, K, seed=9)
    mult, off = H.gpu_fold_static(ws, bias, a, b, S_x, S_r)
    codes, _ = H.gpu_forward(Xq, None, Wq, mult, off, B.QWT_OUT_INT8_STATIC)
    xs = np.full(M, S_x, np.float32)
    real = O.qlinear_cwac_reference(Xq, xs, Wq, ws, bias, a, b)
    inside = np.abs(real / float(S_r)) < 126
    err = np.abs(float(S_r) * codes.astype(np.float64) - real)
    bound = float(S_r) / 2 + np.abs(a.astype(np.float64) * float(S_x) * ws) / 2
    assert np.all(err[inside] <= (bound[None, :].repeat(M, 0))[inside] * (1 + 1e-5) + 1e-7)


def test_static_with_packed_int4_weights(H, B):
    M, N, K = 300, 768, 768
    Xq, Wq, ws, bias, a, b, S_x, S_r = layer(M, N, K, seed=4, w_bits=4)
    mult, off = H.gpu_fold_static(ws, bias, a, b, S_x, S_r)
    codes, _ = H.gpu_forward(Xq, None, O.pack_int4(Wq), mult, off, B.QWT_OUT_INT8_STATIC, wfmt=B.QWT_W_INT4_PACKED, K=K)
    assert np.array_equal(codes, O.requant_static(O.int_matmul(Xq, Wq), mult, off))


def test_static_with_packed_int4_weights_resident_halves(H, B):
    """The same through the pair kernel whose W halves are expanded on chip once per CTA (many rows, six column tiles):
    the integer offsets are then sixteenfold like the operands."""
    M, N, K = 6200, 1536, 416
    Xq, Wq, ws, bias, a, b, S_x, S_r = layer(M, N, K, seed=6, w_bits=4)
    mult, off = H.gpu_fold_static(ws, bias, a, b, S_x, S_r)
    codes, _ = H.gpu_forward(Xq, None, O.pack_int4(Wq), mult, off, B.QWT_OUT_INT8_STATIC, wfmt=B.QWT_W_INT4_PACKED, K=K)
    assert np.array_equal(codes, O.requant_static(O.int_matmul(Xq, Wq), mult, off))
