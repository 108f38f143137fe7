"""GPU parity on seeded random layer shapes: few to 30 000 rows (one tile, own strips, several tiles per CTA), N from 16
to 2064 (every exchange protocol of the per-token INT8 output), K from 16 to 752, all against the oracle."""
import numpy as np
import pytest

from oracle import qwt_oracle as O
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


def draw_shape(rng):
    kind = rng.integers(0, 4)
    M = int(rng.integers(1, 400)) if kind == 0 else (int(rng.integers(9000, 30000)) if kind == 1 else int(rng.integers(400, 9000)))
    N = 16 * int(rng.integers(1, 130)) if rng.random() < 0.7 else 16 * int(rng.integers(1, 33))
    K = 16 * int(rng.integers(1, 48))
    return M, N, K


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes(H, B, seed):
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
