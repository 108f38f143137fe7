"""Pins for the CPU oracle: every oracle function is checked against something other
than itself -- hand-evaluated fixtures of the paper's equations, brute force, closed
forms, invariants, or an independent library routine.  CPU only."""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import qwt_oracle as O
from paper_2505_20932_b200 import workload as WL

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


# ------------------------------------------------------------------ Eq. 1-2 quantizers

def test_uniform_quantize_hand_cases():
    for c in gold("eq1_eq2_hand.json")["cases"]:
        codes, s, z = O.uniform_quantize(np.array(c["x"]), c["bits"])
        assert s == pytest.approx(c["s"], rel=1e-15)
        assert z == c["z"]
        assert codes.tolist() == c["codes"]


def test_uniform_quantize_error_bound_and_range():
    rng = np.random.default_rng(1)
    for bits in (2, 4, 6, 8):
        x = rng.standard_normal(4000) * 3 + 0.7
        codes, s, z = O.uniform_quantize(x, bits)
        qmax = 2 ** bits - 1
        assert codes.min() >= 0 and codes.max() <= qmax
        assert codes[np.argmin(x)] == 0 and codes[np.argmax(x)] == qmax
        xh = s * (codes - z)
        unclipped = (np.rint(x / s) + z >= 0) & (np.rint(x / s) + z <= qmax)
        assert np.all(np.abs(x - xh)[unclipped] <= s / 2 * (1 + 1e-12))
        assert np.all(np.abs(x - xh) <= s * (1 + 1e-12))       # a clipped end point loses at most one step


def test_symmetric_quantizer_is_eq1_with_zero_point_zero():
    # Eq. 1 with s = absmax/qmax, z = 0, clip range moved to the signed interval.
    rng = np.random.default_rng(2)
    X = rng.standard_normal((17, 96)).astype(np.float32)
    for qmax in (127, 7):
        codes, scale = O.quantize_rows_sym(X, qmax)
        for r in range(X.shape[0]):
            s = np.float32(np.abs(X[r]).max()) / np.float32(qmax)
            want = [int(np.clip(np.rint(np.float32(v) / s), -qmax, qmax)) for v in X[r]]
            assert codes[r].tolist() == want
            assert scale[r] == s


def test_symmetric_quantizer_properties():
    rng = np.random.default_rng(3)
    X = (rng.standard_normal((64, 200)) * rng.lognormal(0, 1, (64, 1))).astype(np.float32)
    X[5] = 0.0
    for qmax in (127, 7):
        codes, scale = O.quantize_rows_sym(X, qmax)
        assert codes.dtype == np.int8 and scale.dtype == np.float32
        assert codes.min() >= -qmax and codes.max() <= qmax           # -128 / -8 never produced
        assert scale[5] == 0 and not codes[5].any()                    # all-zero row rule
        err = np.abs(X.astype(np.float64) - scale[:, None].astype(np.float64) * codes)
        assert np.all(err <= scale[:, None].astype(np.float64) / 2 * (1 + 1e-6))   # never clips: |x - s q| <= s/2
        am = np.argmax(np.abs(X), axis=1)
        got = np.abs(codes[np.arange(64), am].astype(int))
        assert np.all(got[scale > 0] == qmax)                          # the absmax element takes the end code
        # idempotence: s*code quantizes to code (same row scale because the end code is present)
        again, scale2 = O.quantize_rows_sym((scale[:, None] * codes).astype(np.float32), qmax)
        assert np.array_equal(again, codes)
        assert np.allclose(scale2, scale, rtol=1e-6)


def test_pack_int4_layout():
    # low nibble = even element, high nibble = odd element, two's complement
    assert O.pack_int4(np.array([[-1, 7]])).tolist() == [[0x7F]]
    assert O.pack_int4(np.array([[3, -2]])).tolist() == [[0xE3]]
    assert O.pack_int4(np.array([[0, -7, 5, 0]])).tolist() == [[0x90, 0x05]]
    rng = np.random.default_rng(4)
    c = rng.integers(-7, 8, size=(9, 64)).astype(np.int8)
    p = O.pack_int4(c)
    assert p.shape == (9, 32) and p.dtype == np.uint8
    assert np.array_equal(O.unpack_int4(p), c)


# ------------------------------------------------------------------ Eq. 6-7 integer product

def brute_matmul(Xq, Wq):
    M, K = Xq.shape
    N = Wq.shape[0]
    out = [[0] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            s = 0
            for k in range(K):
                s += int(Xq[m, k]) * int(Wq[n, k])
            out[m][n] = s
    return np.array(out, dtype=np.int64)


@pytest.mark.parametrize("M,N,K", [(3, 5, 16), (8, 8, 32), (5, 7, 48), (1, 1, 1)])
def test_int_matmul_brute_force(M, N, K):
    rng = np.random.default_rng(M * 100 + N * 10 + K)
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    Wq = rng.integers(-127, 128, (N, K)).astype(np.int8)
    assert np.array_equal(O.int_matmul(Xq, Wq), brute_matmul(Xq, Wq))


def test_int_matmul_extremes_and_selection():
    K = 11008
    Xq = np.full((2, K), 127, np.int8)
    Xq[1] = -127
    Wq = np.full((3, K), 127, np.int8)
    Wq[2] = -127
    acc = O.int_matmul(Xq, Wq)
    e = 127 * 127 * K
    assert acc.tolist() == [[e, e, -e], [-e, -e, e]]
    # a weight matrix of unit rows picks out columns of X (wrong operand transposition fails this)
    rng = np.random.default_rng(5)
    Xq = rng.integers(-127, 128, (6, 10)).astype(np.int8)
    Wsel = np.zeros((4, 10), np.int8)
    for n, k in enumerate([7, 0, 3, 9]):
        Wsel[n, k] = 1
    assert np.array_equal(O.int_matmul(Xq, Wsel), Xq[:, [7, 0, 3, 9]].astype(np.int64))


def test_int_matmul_matches_integer_arithmetic_medium():
    rng = np.random.default_rng(6)
    Xq = rng.integers(-127, 128, (70, 384)).astype(np.int8)
    Wq = rng.integers(-127, 128, (90, 384)).astype(np.int8)
    want = Xq.astype(np.int64) @ Wq.astype(np.int64).T       # numpy's integer loops, no floating point
    assert np.array_equal(O.int_matmul(Xq, Wq), want)


def test_eq7_hand_cases_and_expansion():
    for c in gold("eq7_hand.json")["cases"]:
        got = O.qlinear_eq7(np.array(c["Wq"]), np.array(c["xq"]), np.array(c["Zw"]), c["Zx"])
        assert got.tolist() == c["bracket"]
    rng = np.random.default_rng(7)
    Wq = rng.integers(0, 256, (6, 40))
    xq = rng.integers(0, 256, 40)
    Zw = rng.integers(0, 256, 6)
    Zx = 131
    direct = [sum((int(Wq[n, k]) - int(Zw[n])) * (int(xq[k]) - Zx) for k in range(40)) for n in range(6)]
    assert O.qlinear_eq7(Wq, xq, Zw, Zx).tolist() == direct
    # zero-points 0 -> the three correction terms vanish and Eq. 7 is the plain product
    X8 = rng.integers(-127, 128, (1, 40)).astype(np.int8)
    W8 = rng.integers(-127, 128, (6, 40)).astype(np.int8)
    assert np.array_equal(O.qlinear_eq7(W8, X8[0], np.zeros(6, int), 0), O.int_matmul(X8, W8)[0])


def test_dequant_is_eq6_with_zero_zero_points():
    # S_r (r_q - Z_r) = S_W (W_q - Z_W) S_x (x_q - Z_x): with Z = 0 the right side is S_W S_x W_q x_q
    acc = np.array([[10, -4], [3, 0]])
    y = O.dequant(acc, np.array([0.5, 2.0]), np.array([0.1, 0.25]), np.array([1.0, -1.0]))
    assert np.allclose(y, [[10 * 0.5 * 0.1 + 1, -4 * 0.5 * 0.25 - 1], [3 * 2 * 0.1 + 1, -1.0]], rtol=1e-15)
    y0 = O.dequant(acc, np.array([0.5, 2.0]), np.array([0.1, 0.25]), None)
    assert np.allclose(y0, [[0.5, -0.5], [0.6, 0.0]], rtol=1e-15)


def test_quantized_layer_approximates_fp_layer():
    # End-to-end sanity of o1-o4: the dequantized product approaches X W^T + bias as codes get finer.
    spec = WL.LayerSpec("t", 32, 64, 48, 8, "int8", "normal", 32)
    d = WL.host_layer_inputs(spec, seed=11)
    Xq, xs = O.quantize_rows_sym(d["X"], 127)
    Wq, ws = O.quantize_rows_sym(d["W"], 127)
    y = O.dequant(O.int_matmul(Xq, Wq), xs, ws, d["bias"])
    ref = O.linear_fp(d["X"], d["W"], d["bias"])
    rel = np.linalg.norm(y - ref) / np.linalg.norm(ref)
    assert rel < 0.02
    Wq4, ws4 = O.quantize_rows_sym(d["W"], 7)
    y4 = O.dequant(O.int_matmul(Xq, Wq4), xs, ws4, d["bias"])
    rel4 = np.linalg.norm(y4 - ref) / np.linalg.norm(ref)
    assert rel < rel4 < 0.3


# ------------------------------------------------------------------ Eq. 3-5 fit

def test_fit_hand_cases():
    for c in gold("eq4_eq5_hand.json")["cases"]:
        a, b, nd = O.cwac_fit(np.array(c["f"])[:, None], np.array(c["q"])[:, None])
        assert a[0] == pytest.approx(c["alpha"], abs=1e-14)
        assert b[0] == pytest.approx(c["beta"], abs=1e-14)
        assert nd == 0


def test_apply_hand_case_and_fit_residual():
    """alpha (.) y + beta per channel: a worked case, and the least-squares property that ties it to the fit
    (after compensation the residual has zero mean and is uncorrelated with q in every channel)."""
    y = np.array([[1.0, 2.0], [3.0, 4.0]])
    assert np.array_equal(O.cwac_apply(y, np.array([2.0, 0.5]), np.array([1.0, -1.0])), np.array([[3.0, 0.0], [7.0, 1.0]]))
    rng = np.random.default_rng(12)
    q = rng.standard_normal((500, 7)) + rng.uniform(-2, 2, 7)
    f = q * rng.uniform(0.5, 1.5, 7) + 0.3 * rng.standard_normal((500, 7)) + rng.uniform(-1, 1, 7)
    a, b, _ = O.cwac_fit(f, q)
    res = f - O.cwac_apply(q, a, b)
    assert np.abs(res.mean(0)).max() < 1e-12 and np.abs((res * q).mean(0)).max() < 1e-12


def test_fit_planted_recovery_and_identity():
    rng = np.random.default_rng(8)
    q = rng.standard_normal((50, 7)) * 3 + 1
    a_star = rng.standard_normal(7)
    b_star = rng.standard_normal(7)
    a, b, _ = O.cwac_fit(q * a_star + b_star, q)
    assert np.allclose(a, a_star, rtol=0, atol=1e-12) and np.allclose(b, b_star, rtol=0, atol=1e-12)
    a, b, _ = O.cwac_fit(q, q)                      # quantized output == full-precision output
    assert np.allclose(a, 1.0, atol=1e-14) and np.allclose(b, 0.0, atol=1e-14)


def test_fit_normal_equations_and_optimality():
    rng = np.random.default_rng(9)
    q = rng.standard_normal((400, 5)) + 0.3
    f = 0.9 * q + 0.1 * rng.standard_normal((400, 5)) - 0.2
    a, b, _ = O.cwac_fit(f, q)
    r = f - (a * q + b)
    assert np.all(np.abs(r.sum(0)) < 1e-10)           # residual orthogonal to the constant
    assert np.all(np.abs((r * q).sum(0)) < 1e-10)     # and to the regressor
    sse = (r ** 2).sum(0)
    for da, db in itertools.product((-1e-3, 0, 1e-3), repeat=2):
        r2 = f - ((a + da) * q + (b + db))
        assert np.all((r2 ** 2).sum(0) >= sse - 1e-12)


def test_fit_equals_textbook_normal_equation_solve():
    rng = np.random.default_rng(10)
    q = rng.standard_normal((300, 4)) * 2 + 5
    f = rng.standard_normal((300, 4))
    a, b, _ = O.cwac_fit(f, q)
    L = np.longdouble
    for c in range(4):
        x = q[:, c].astype(L)
        y = f[:, c].astype(L)
        n = L(len(x))
        # [sum x^2  sum x][a]   [sum x y]
        # [sum x    n    ][b] = [sum y  ]
        sxx, sx, sxy, sy = (x * x).sum(), x.sum(), (x * y).sum(), y.sum()
        det = sxx * n - sx * sx
        a_t = (sxy * n - sx * sy) / det
        b_t = (sxx * sy - sx * sxy) / det
        assert float(a_t) == pytest.approx(a[c], rel=1e-11)
        assert float(b_t) == pytest.approx(b[c], rel=1e-10, abs=1e-12)
        pa, pb = np.polyfit(q[:, c], f[:, c], 1)        # independent library routine (QR least squares)
        assert pa == pytest.approx(a[c], rel=1e-10) and pb == pytest.approx(b[c], rel=1e-9, abs=1e-12)


def test_fit_equivariances_and_permutation():
    rng = np.random.default_rng(11)
    q = rng.standard_normal((128, 3))
    f = 1.1 * q + 0.05 * rng.standard_normal((128, 3)) + 0.3
    a, b, _ = O.cwac_fit(f, q)
    a2, b2, _ = O.cwac_fit(f, 4.0 * q)
    assert np.allclose(a2, a / 4, rtol=1e-12) and np.allclose(b2, b, rtol=1e-11, atol=1e-13)
    a3, b3, _ = O.cwac_fit(f, q + 2.5)
    assert np.allclose(a3, a, rtol=1e-12) and np.allclose(b3, b - 2.5 * a, rtol=1e-11)
    a4, b4, _ = O.cwac_fit(f + 7.0, q)
    assert np.allclose(a4, a, rtol=1e-12) and np.allclose(b4, b + 7.0, rtol=1e-12)
    a5, b5, _ = O.cwac_fit(-3.0 * f, q)
    assert np.allclose(a5, -3 * a, rtol=1e-12) and np.allclose(b5, -3 * b, rtol=1e-12)
    p = rng.permutation(128)
    a6, b6, _ = O.cwac_fit(f[p], q[p])
    assert np.allclose(a6, a, rtol=1e-12) and np.allclose(b6, b, rtol=1e-11, atol=1e-14)


def test_fit_degenerate_variance_rule():
    q = np.array([[2.0, 1.0, 0.0], [2.0, 3.0, 0.0], [2.0, 5.0, 0.0]])
    f = np.array([[1.0, 1.0, 4.0], [2.0, 3.0, 5.0], [6.0, 5.0, 6.0]])
    a, b, nd = O.cwac_fit(f, q)
    assert nd == 2
    assert a.tolist() == [1.0, 1.0, 1.0]
    assert b[0] == pytest.approx(3.0 - 2.0) and b[1] == pytest.approx(0.0) and b[2] == pytest.approx(5.0)
    a, b, nd = O.cwac_fit(np.array([[3.0]]), np.array([[1.0]]))        # a single row
    assert nd == 1 and a[0] == 1.0 and b[0] == 2.0


def test_fit_uniform_noise_closed_form():
    # q = f + U(-D/2, D/2) independent of f: alpha -> sigma^2 / (sigma^2 + D^2/12), beta -> 0
    R, C = 200_000, 6
    for bits, want in ((4, 1.0 / (1.0 + (8.0 / 15) ** 2 / 12)), (8, 1.0 / (1.0 + (8.0 / 255) ** 2 / 12))):
        fp, q, sig = WL.host_calib_pair(R, C, bits, seed=3)
        a, b, nd = O.cwac_fit(fp, q)
        assert nd == 0
        assert np.all(np.abs(a - want) < 6.0 / np.sqrt(R) * (8.0 / (2 ** bits - 1)))
        assert np.all(np.abs(b) < 6.0 * sig * (8.0 / (2 ** bits - 1)) / np.sqrt(12 * R) + 1e-6)
    assert abs(1.0 / (1.0 + (8.0 / 15) ** 2 / 12) - 0.97685) < 1e-5


def test_stats_determine_the_fit():
    # Eq. 4-5 are functions of (n, sum q, sum f, sum qf, sum q^2) only
    rng = np.random.default_rng(12)
    q = rng.standard_normal((500, 4)) + 1
    f = 0.8 * q + 0.1 * rng.standard_normal((500, 4))
    n, sq, sf, sqf, sqq = O.cwac_stats(f, q)
    var = sqq / n - (sq / n) ** 2
    cov = sqf / n - (sq / n) * (sf / n)
    a, b, _ = O.cwac_fit(f, q)
    assert np.allclose(cov / var, a, rtol=1e-10)
    assert np.allclose(sf / n - cov / var * sq / n, b, rtol=1e-9, atol=1e-12)


# ------------------------------------------------------------------ Eq. 9-11 fold

def test_folded_path_equals_unfolded_path():
    rng = np.random.default_rng(13)
    M, N, K = 24, 40, 64
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    Wq = rng.integers(-127, 128, (N, K)).astype(np.int8)
    xs = rng.uniform(0.01, 0.05, M).astype(np.float32)
    ws = rng.uniform(1e-4, 3e-4, N).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32) * 0.01
    a = (1 + 0.05 * rng.standard_normal(N)).astype(np.float32)
    b = (0.02 * rng.standard_normal(N)).astype(np.float32)
    acc = O.int_matmul(Xq, Wq)
    z = O.qlinear_cwac_reference(Xq, xs, Wq, ws, bias, a, b)
    fs, fb = O.cwac_fold(ws, bias, a, b)
    z2 = O.forward_folded(acc, xs, fs, fb)
    assert np.max(np.abs(z - z2)) <= 1e-12 * np.max(np.abs(z))
    # missing pieces: no bias, no CWAC -> plain dequant
    fs0, fb0 = O.cwac_fold(ws, None, None, None)
    assert np.array_equal(fs0, ws.astype(np.float64)) and not fb0.any()
    assert np.allclose(O.forward_folded(acc, xs, fs0, fb0), O.dequant(acc, xs, ws, None), rtol=1e-15)
    # negative / zero alpha are legal in the folded form (no division)
    a[0], a[1] = -0.5, 0.0
    fs, fb = O.cwac_fold(ws, bias, a, b)
    z3 = O.forward_folded(acc, xs, fs, fb)
    assert np.allclose(z3, O.qlinear_cwac_reference(Xq, xs, Wq, ws, bias, a, b), rtol=1e-12, atol=1e-15)
    assert np.allclose(z3[:, 1], b[1], rtol=1e-7)


def test_integer_offset_fold_hand_cases_and_rounding_bound():
    for c in gold("eq10_eq11_hand.json")["cases"]:
        Mp, off = O.fold_integer_offset([c["alpha"]], [c["beta"]], c["S_x"], [c["S_W"]], c["S_r"])
        assert Mp[0] == pytest.approx(c["Mp"], rel=1e-14) and off[0] == c["offset"]
    # Eq. 10 vs Eq. 9: alpha folds without loss, beta loses at most half an accumulator step
    rng = np.random.default_rng(14)
    N = 32
    alpha = 1 + 0.05 * rng.standard_normal(N)
    beta = 0.02 * rng.standard_normal(N)
    S_x, S_r = 0.03, 0.02
    S_W = rng.uniform(1e-4, 3e-4, N)
    acc = rng.integers(-50000, 50000, (10, N))
    Mp, off = O.fold_integer_offset(alpha, beta, S_x, S_W, S_r)
    lhs = S_r * Mp * (acc + off)                     # S_r (r_q - Z_r) from Eq. 10 before rounding r_q
    rhs = alpha * S_W * S_x * acc + beta             # Eq. 9 right-hand side (zero-points 0)
    assert np.all(np.abs(lhs - rhs) <= np.abs(alpha * S_x * S_W) / 2 * (1 + 1e-9))
    assert np.abs(beta / (alpha * S_x * S_W)).mean() > 100        # offsets are large, as the paper remarks


# ------------------------------------------------------------------ output stage

def test_requant_per_token_properties():
    rng = np.random.default_rng(15)
    z = rng.standard_normal((40, 300)) * rng.lognormal(0, 1, (40, 1))
    z[7] = 0
    codes, ys = O.requant_per_token(z)
    z32 = z.astype(np.float32)
    assert np.array_equal(ys, (np.abs(z32).max(1) / np.float32(127)).astype(np.float32))
    assert ys[7] == 0 and not codes[7].any()
    assert codes.min() >= -127 and codes.max() <= 127
    err = np.abs(z32.astype(np.float64) - ys[:, None].astype(np.float64) * codes)
    assert np.all(err <= 0.5 * ys[:, None] * (1 + 1e-4))
    am = np.argmax(np.abs(z32), axis=1)
    assert np.all(np.abs(codes[np.arange(40), am].astype(int))[ys > 0] == 127)


def test_bf16_rounding_hand_cases_and_library():
    # 1 + 2^-8 lies halfway between 1 and 1 + 2^-7: ties to even -> 1.0;  1 + 3*2^-8 -> 1 + 2^-6
    cases = {1.0: 0x3F80, 1.0 + 2 ** -8: 0x3F80, 1.0 + 3 * 2 ** -8: 0x3F82, -2.0: 0xC000,
             1.0 + 2 ** -8 + 2 ** -20: 0x3F81, 0.0: 0x0000, 3.3895313892515355e38: 0x7F7F}
    for v, bits in cases.items():
        assert int(O.to_bf16_bits(np.array([v]))[0]) == bits, v
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(16)
    z = (rng.standard_normal(200_000) * np.exp(rng.uniform(-20, 20, 200_000))).astype(np.float32)
    want = torch.from_numpy(z).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.to_bf16_bits(z), want)
    assert np.array_equal(O.bf16_bits_to_f32(want), torch.from_numpy(z).to(torch.bfloat16).float().numpy())


# ------------------------------------------------------------------ parameter budget (Tables 1, 9)

def test_cwac_parameter_budget_matches_printed_delta():
    g = gold("table1_delta_mb.json")
    per = g["bytes_per_value"] * g["values_per_channel"]
    vit_b = sum(s.N for s in WL.config_layers(3)) * per / 1e6
    deit_s = sum(s.N for s in WL.config_layers(2)) * per / 1e6
    assert round(vit_b, 1) == g["vit_b_delta_mb"]
    assert round(deit_s, 1) == g["deit_s_delta_mb"]


# ------------------------------------------------------------------ Eq. 10 with static scales (integer-offset form)

def test_static_requant_hand_fixture():
    g = gold("eq10_static_requant_hand.json")
    got = O.requant_static(np.array(g["acc"]), np.array(g["Mp"]), np.array(g["off"]))
    # 0.001 is not a binary fraction: the hand values at exact .5 ties (1.5, 127.5, 3.5) must not depend on it
    assert np.array_equal(got[:, [0, 1, 3]], np.array(g["expected"])[:, [0, 1, 3]])
    assert np.all(np.abs(got[:, 2].astype(int) - np.array(g["expected"])[:, 2]) <= 1)
    assert got[2, 2] == 127 and got[1, 3] == -127 and got[3, 3] == -127       # clipping


def test_static_requant_equals_quantizing_the_compensated_output():
    """Eq. 9 -> Eq. 10: dividing the compensated real output by S_r and rounding gives the same codes as the
    integer-offset form whenever beta / (alpha S_x S_W) is an integer (then Eq. 10 loses nothing), and differs
    by at most one step otherwise (beta is off by at most half an accumulator step, Section 3.4)."""
    rng = np.random.default_rng(21)
    M, N = 64, 48
    alpha = 1 + 0.05 * rng.standard_normal(N)
    S_W = rng.uniform(1e-4, 3e-4, N)
    S_x, S_r = 0.03, 0.02
    acc = rng.integers(-60000, 60000, (M, N))
    k = rng.integers(-500, 500, N)
    beta_exact = k * alpha * S_x * S_W                      # beta / (alpha S_x S_W) = k exactly
    Mp, off = O.fold_integer_offset(alpha, beta_exact, S_x, S_W, S_r)
    assert np.array_equal(off, k)
    real = (alpha * S_W * S_x)[None, :] * acc + beta_exact[None, :]          # Eq. 9 right-hand side
    direct = np.clip(np.rint(real / S_r), -127, 127)
    got = O.requant_static(acc, Mp, off).astype(np.int64)
    # float32 product against the float64 quotient: equal except within 1e-4 of a rounding tie
    near_tie = np.abs((real / S_r) - np.floor(real / S_r) - 0.5) < 1e-4
    assert np.array_equal(got[~near_tie], direct[~near_tie]) and np.abs(got - direct).max() <= 1
    # arbitrary beta: at most one output step away, and the real-valued error obeys the Section 3.4 bound
    beta = 0.02 * rng.standard_normal(N)
    Mp, off = O.fold_integer_offset(alpha, beta, S_x, S_W, S_r)
    real = (alpha * S_W * S_x)[None, :] * acc + beta[None, :]
    direct = np.clip(np.rint(real / S_r), -127, 127)
    got = O.requant_static(acc, Mp, off).astype(np.int64)
    assert np.abs(got - direct).max() <= 1
    unclipped = np.abs(real / S_r) < 126
    err = np.abs(S_r * got - real)[unclipped]
    assert np.all(err <= S_r / 2 + (np.abs(alpha * S_x * S_W) / 2)[None, :].repeat(M, 0)[unclipped] + 1e-9)


def test_static_requant_zero_point_and_symmetry():
    acc = np.array([[10, -10, 0]])
    Mp = np.array([1.0, 1.0, 1.0])
    off = np.array([0, 0, 0])
    assert O.requant_static(acc, Mp, off, Z_r=5).tolist() == [[15, -5, 5]]
    a = np.arange(-300, 300).reshape(1, -1)
    r = O.requant_static(a, np.full(600, 0.7), np.zeros(600, dtype=int))
    assert np.array_equal(r, -O.requant_static(-a, np.full(600, 0.7), np.zeros(600, dtype=int)))   # odd function


# ------------------------------------------------------------------ asymmetric codes (Eq. 1-2 and Eq. 6-7 in full)

def test_rowwise_asymmetric_quantizer_is_eq1_eq2_per_row():
    rng = np.random.default_rng(31)
    X = (rng.standard_normal((6, 50)) * rng.lognormal(0, 1, (6, 1)) + rng.normal(0, 2, (6, 1))).astype(np.float32)
    q, s, z = O.quantize_rows_asym(X, 8)
    for r in range(X.shape[0]):
        qr, sr, zr = O.uniform_quantize(X[r], 8)           # the per-tensor form pinned by the hand fixture
        assert z[r] == zr and s[r] == pytest.approx(sr, rel=1e-6)
        assert np.abs(q[r].astype(int) - qr).max() <= 1    # float32 vs float64 quotient: at most a tie apart
        assert np.count_nonzero(q[r].astype(int) - qr) <= 1
    assert q.min() == 0 and q.max() == 255                 # the extremes of a row take the end codes
    back = s[:, None] * (q.astype(np.float64) - z[:, None])
    # rows whose range contains 0: half a step from rounding x, half from rounding the zero-point, one more where
    # the shifted end code clips.  Rows that lie on one side of 0 have their zero-point clipped by Eq. 2 and are
    # represented badly -- that is the quantizer as printed, kept as is.
    spans0 = (X.min(axis=1) <= 0) & (X.max(axis=1) >= 0)
    assert spans0.sum() >= 3 and (~spans0).sum() >= 1
    err = np.abs(back - X) / s[:, None]
    assert np.all(err[spans0] <= 2.0 * (1 + 1e-3)) and np.mean(err[spans0] <= 1 + 1e-3) > 0.97
    assert np.all(np.isin(z[~spans0], (0, 255)))
    qc, sc, zc = O.quantize_rows_asym(np.full((1, 8), 3.0, np.float32))
    assert sc[0] == 1.0 and np.all(qc == qc[0, 0])


def test_asymmetric_product_equals_eq7_expansion_and_brute_force():
    rng = np.random.default_rng(32)
    M, N, K = 5, 7, 48
    Xq = rng.integers(0, 256, (M, K)).astype(np.uint8)
    Wq = rng.integers(0, 256, (N, K)).astype(np.uint8)
    Zx = rng.integers(0, 256, M)
    Zw = rng.integers(0, 256, N)
    acc = O.int_matmul_asym(Xq, Zx, Wq, Zw)
    brute = np.zeros((M, N), dtype=np.int64)
    for m in range(M):
        for n in range(N):
            for k in range(K):
                brute[m, n] += (int(Wq[n, k]) - int(Zw[n])) * (int(Xq[m, k]) - int(Zx[m]))
    assert np.array_equal(acc, brute)
    for m in range(M):                                     # Eq. 7's four terms, pinned separately by eq7_hand.json
        assert np.array_equal(acc[m], O.qlinear_eq7(Wq, Xq[m], Zw, int(Zx[m])))
    # zero zero-points: the symmetric product
    assert np.array_equal(O.int_matmul_asym(Xq, 0, Wq, np.zeros(N)), O.int_matmul(Xq.astype(np.int64), Wq.astype(np.int64)))
    # the real-valued product is recovered: S_W (W_q - Z_W) S_x (x_q - Z_x) ~ W x  (Eq. 6)
    X = rng.standard_normal((20, 64)).astype(np.float32) + 1.0
    W = (0.02 * rng.standard_normal((12, 64))).astype(np.float32)
    xq, xs, xz = O.quantize_rows_asym(X)
    wq, ws, wz = O.quantize_rows_asym(W)
    y = O.int_matmul_asym(xq, xz, wq, wz) * xs[:, None].astype(np.float64) * ws[None, :]
    ref = X.astype(np.float64) @ W.astype(np.float64).T
    assert np.abs(y - ref).max() < 0.02 * np.abs(ref).max() + 1e-3


# ------------------------------------------------------------------ convolution (CWAC after quantized convolutions)

def test_integer_convolution_definition():
    rng = np.random.default_rng(51)
    Bn, H, W, C, N = 2, 5, 6, 3, 4
    X = rng.integers(-127, 128, (Bn, H, W, C))
    # 1x1: the linear layer over B*H*W tokens
    W1 = rng.integers(-127, 128, (N, 1, 1, C))
    assert np.array_equal(O.conv2d_int_nhwc(X, W1).reshape(-1, N), O.int_matmul(X.reshape(-1, C), W1.reshape(N, C)))
    # 3x3, stride 2, padding 1: brute force over every index
    W3 = rng.integers(-127, 128, (N, 3, 3, C))
    got = O.conv2d_int_nhwc(X, W3, stride=2, pad=1)
    Ho, Wo = (H + 2 - 3) // 2 + 1, (W + 2 - 3) // 2 + 1
    assert got.shape == (Bn, Ho, Wo, N)
    for b in range(Bn):
        for ho in range(Ho):
            for wo in range(Wo):
                for n in range(N):
                    t = 0
                    for i in range(3):
                        for j in range(3):
                            y, x = ho * 2 + i - 1, wo * 2 + j - 1
                            if 0 <= y < H and 0 <= x < W:
                                t += int(np.dot(X[b, y, x], W3[n, i, j]))
                    assert got[b, ho, wo, n] == t
    # a kernel that is 1 at its centre tap of channel c copies that channel (catches a flipped or shifted window)
    Wd = np.zeros((C, 3, 3, C), dtype=np.int64)
    for c in range(C):
        Wd[c, 1, 1, c] = 1
    assert np.array_equal(O.conv2d_int_nhwc(X, Wd, stride=1, pad=1), X)
