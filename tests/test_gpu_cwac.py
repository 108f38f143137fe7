"""GPU parity: CWAC calibration, fold and the row quantizer against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest

from oracle import qwt_oracle as O
from paper_2505_20932_b200 import workload as WL
from tolerances import assert_ab_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    import gpu_harness
    return gpu_harness


def nat_scale(fp):
    fp = fp.astype(np.float64)
    return np.maximum(np.abs(fp.mean(0)), fp.std(0))


@pytest.mark.parametrize("rows,C,bits", [(6304, 1536, 8), (1000, 768, 4), (129, 132, 4), (1, 4, 8), (7, 8, 8),
                                         (50_000, 384, 4)])
def test_calibrate_matches_oracle(H, rows, C, bits):
    fp, q, _ = WL.host_calib_pair(rows, C, bits, seed=rows + C)
    a, b, nd = H.gpu_calibrate(fp, q)
    a_ref, b_ref, nd_ref = O.cwac_fit(fp, q)
    assert nd == nd_ref
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(fp))


def test_calibrate_channel_means_far_above_their_spread(H):
    """|mean| / std between 1e4 and 1e5: var(q) = E[q^2] - E[q]^2 loses nine to ten digits to cancellation."""
    rng = np.random.default_rng(17)
    rows, C = 20_000, 256
    ratio = np.geomspace(1e4, 1e5, C)
    q = (rng.standard_normal((rows, C)) + ratio[None, :]).astype(np.float32)
    f = (1.03 * q.astype(np.float64) + 0.25 + 0.05 * rng.standard_normal((rows, C))).astype(np.float32)
    a, b, nd = H.gpu_calibrate(f, q)
    a_ref, b_ref, nd_ref = O.cwac_fit(f, q)
    assert nd == nd_ref == 0
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(f))


def test_calibrate_leading_dimension_and_ragged_channels(H):
    # 130 channels inside rows of 136 floats: the padding columns hold garbage that must not matter
    rows, C, ld = 777, 130, 136
    fp, q, _ = WL.host_calib_pair(rows, C, 4, seed=5, ld=ld)
    fp[:, C:] = 1e30
    q[:, C:] = -1e30
    a, b, nd = H.gpu_calibrate(fp, q, channels=C)
    a_ref, b_ref, _ = O.cwac_fit(fp[:, :C], q[:, :C])
    assert a.shape == (C,) and nd == 0
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(fp[:, :C]))


def test_calibrate_planted_identity_and_offset_channels(H):
    rng = np.random.default_rng(3)
    rows, C = 4096, 256
    q = (rng.standard_normal((rows, C)) * rng.lognormal(0, 1, C)).astype(np.float32)
    q[:, :64] += np.float32(25.0)            # channels whose mean dwarfs their spread
    q[:, 64:96] *= np.float32(1e-3)
    a_star = (1 + 0.05 * rng.standard_normal(C)).astype(np.float32)
    b_star = (0.02 * rng.standard_normal(C)).astype(np.float32)
    f = (q.astype(np.float64) * a_star + b_star).astype(np.float32)
    a, b, nd = H.gpu_calibrate(f, q)
    a_ref, b_ref, _ = O.cwac_fit(f, q)
    assert nd == 0
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(f))
    assert np.allclose(a, a_star, rtol=2e-5, atol=1e-6)     # f32 rounding of f perturbs the planted line slightly
    a, b, nd = H.gpu_calibrate(q, q)                         # quantized output == full-precision output
    assert np.allclose(a, 1.0, rtol=0, atol=1e-6) and np.all(np.abs(b) <= 1e-5 * nat_scale(q) + 1e-7)


def test_calibrate_degenerate_channels(H):
    rng = np.random.default_rng(4)
    rows, C = 300, 12
    q = rng.standard_normal((rows, C)).astype(np.float32)
    f = (0.9 * q + 0.1).astype(np.float32)
    q[:, 3] = 2.5
    q[:, 7] = 0.0
    a, b, nd = H.gpu_calibrate(f, q)
    a_ref, b_ref, nd_ref = O.cwac_fit(f, q)
    assert nd == nd_ref == 2
    assert a[3] == 1.0 and a[7] == 1.0
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(f))


def test_streamed_statistics_equal_one_shot(H):
    rows, C = 5000, 200
    fp, q, _ = WL.host_calib_pair(rows, C, 4, seed=9)
    a1, b1, _ = H.gpu_calibrate(fp, q)
    a2, b2, nd, stats = H.gpu_calibrate_streamed(fp, q, batches=7)
    ref = O.cwac_stats(fp, q)
    assert np.allclose(stats, ref, rtol=2e-6, atol=1e-4)      # short FP32 runs inside the kernel
    assert stats[0, 0] == rows
    a_ref, b_ref, _ = O.cwac_fit(fp, q)
    assert_ab_close(a2, b2, a_ref, b_ref, nat_scale(fp))
    assert np.allclose(a1, a2, rtol=1e-6) and nd == 0


def test_calibrate_is_reproducible(H):
    fp, q, _ = WL.host_calib_pair(20_000, 768, 4, seed=1)
    a1, b1, _ = H.gpu_calibrate(fp, q)
    a2, b2, _ = H.gpu_calibrate(fp, q)
    assert np.array_equal(a1, a2) and np.array_equal(b1, b2)


def test_calibrate_from_host_memory(H):
    import torch
    from paper_2505_20932_b200 import binding as B
    rows, C = 40_000, 512     # several staging chunks? (64 MiB per slot -> one chunk here; 2nd case below)
    fp, q, _ = WL.host_calib_pair(rows, C, 4, seed=2)
    a = np.empty(C, np.float32)
    b = np.empty(C, np.float32)
    nd = np.full(1, -1, np.int32)
    sb = B.qwt_cwac_host_staging_bytes(rows, C)
    st = H.empty_bytes(sb)
    B.qwt_cwac_calibrate_host(fp, q, rows, C, C, a, b, nd, st, sb)
    a_ref, b_ref, _ = O.cwac_fit(fp, q)
    assert nd[0] == 0
    assert_ab_close(a, b, a_ref, b_ref, nat_scale(fp))


def test_fold_matches_oracle(H):
    rng = np.random.default_rng(6)
    n = 1000
    ws = rng.uniform(1e-4, 3e-4, n).astype(np.float32)
    bias = (0.01 * rng.standard_normal(n)).astype(np.float32)
    a = (1 + 0.05 * rng.standard_normal(n)).astype(np.float32)
    b = (0.02 * rng.standard_normal(n)).astype(np.float32)
    for (bb, aa, b2) in [(bias, a, b), (None, a, b), (bias, None, None), (None, None, None)]:
        fs, fb = H.gpu_fold(ws, bb, aa, b2)
        fs_ref, fb_ref = O.cwac_fold(ws, bb, aa, b2)
        assert np.allclose(fs, fs_ref, rtol=1e-6, atol=0)
        assert np.allclose(fb, fb_ref, rtol=1e-6, atol=1e-9)


@pytest.mark.parametrize("rows,cols,qmax", [(788, 384, 127), (1536, 384, 127), (64, 768, 7), (3, 16, 127), (33, 1000, 7),
                                            (5, 18, 127), (33, 1001, 7)])      # the last two: no 16-byte row pieces
def test_row_quantizer_bit_exact(H, rows, cols, qmax):
    X = WL.host_activations("sparse_outlier", rows, cols, seed=rows, tag="q")
    if rows > 2:
        X[2] = 0
    codes, scale = H.gpu_quantize_rows(X, qmax)
    c_ref, s_ref = O.quantize_rows_sym(X, qmax)
    assert np.array_equal(scale, s_ref)
    assert np.array_equal(codes, c_ref)


def test_pack_int4_bit_exact(H):
    rng = np.random.default_rng(8)
    c = rng.integers(-7, 8, (37, 64)).astype(np.int8)
    assert np.array_equal(H.gpu_pack_int4(c), O.pack_int4(c))


def test_batched_calibration_is_the_single_calls_bit_for_bit(H):
    """Several layers in one call: same partition, same order, hence the same bits as one call per layer, with the
    fold of Eq. 11 done on the way when asked for; more problems than one launch takes go in groups."""
    import torch
    from paper_2505_20932_b200 import binding as B
    rng = np.random.default_rng(3)
    shapes = [(6304, 384, 384), (1000, 768, 768), (129, 132, 136), (1, 4, 4), (3000, 1152, 1152)] * 9   # 45 problems
    items, keep, single = [], [], []
    for i, (rows, C, ld) in enumerate(shapes):
        fp, q, _ = WL.host_calib_pair(rows, ld, 4 if i % 2 else 8, seed=100 + i)
        dfp, dq = H.dev(fp), H.dev(q)
        a, b = (torch.full((C,), 7.0, device=H.DEV) for _ in range(2))
        fold = i % 3 != 0
        ws_, bias = (H.dev(rng.uniform(1e-3, 2e-3, C).astype(np.float32)), H.dev(rng.standard_normal(C).astype(np.float32))) if fold else (None, None)
        fs, fb = (torch.zeros(C, device=H.DEV), torch.zeros(C, device=H.DEV)) if fold else (None, None)
        items.append((dfp, dq, rows, C, ld, a, b, ws_, bias if i % 2 else None, fs, fb))
        keep.append((fp, q, C, a, b, ws_, bias if i % 2 else None, fs, fb))
    probs = B.calib_problems(items)
    wsb = B.qwt_cwac_calibrate_batch_workspace_bytes(probs)
    ws = H.empty_bytes(wsb)
    ws.fill_(0xFF)
    nd = torch.full((1,), -1, dtype=torch.int32, device=H.DEV)
    B.qwt_cwac_calibrate_batch(probs, nd, ws, wsb)
    torch.cuda.synchronize()
    nd_total = 0
    for fp, q, C, a, b, ws_, bias, fs, fb in keep:
        a1, b1, nd1 = H.gpu_calibrate(fp, q, channels=C)
        nd_total += nd1
        assert np.array_equal(a.cpu().numpy(), a1) and np.array_equal(b.cpu().numpy(), b1)
        if ws_ is not None:
            gfs, gfb = H.gpu_fold(ws_.cpu().numpy(), None if bias is None else bias.cpu().numpy(), a1, b1)
            assert np.array_equal(fs.cpu().numpy(), gfs) and np.array_equal(fb.cpu().numpy(), gfb)
    assert int(nd.item()) == nd_total
    # and against the oracle, one of them
    fp, q, C, a, b = keep[4][:5]
    a_ref, b_ref, _ = O.cwac_fit(fp[:, :C], q[:, :C])
    assert_ab_close(a.cpu().numpy(), b.cpu().numpy(), a_ref, b_ref, nat_scale(fp[:, :C]))
