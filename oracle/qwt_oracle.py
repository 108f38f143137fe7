"""CPU oracle for the CWAC-fused quantized linear layer and the CWAC fit (QwT-v2).

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow definition of what the
CUDA library computes.  It is imported by the tests, by the smoke check and by
the benchmark's CPU-baseline leg, never by the product path, and it shares no
code with the CUDA sources.

Conventions
-----------
* Floating-point results are float64 unless stated.  Where floating point decides
  an *integer* (a quantized code) the decision is taken in float32 -- the precision
  the kernels work in -- so that both sides round the same quotient.
* The rounding function of Eq. 1 is round-half-to-even (``np.rint``).
* Symmetric quantizers (zero-point 0, signed codes in [-qmax, qmax]) are the
  Z = 0 special case of Eq. 1-2 / Eq. 6-11; the general asymmetric forms are also
  given (``uniform_quantize``, ``qlinear_eq7``) and tested to reduce to them.

Every function names the passage of the paper it follows.

Parity status: every function below is pinned by tests/test_oracle_*.py against
closed forms, brute force or identities the paper states.  The paper's accuracy
tables (ImageNet, COCO, CLIP, DiT, LLaMA) are NOT reproduced: parity unpinned for
end-to-end model accuracy (needs datasets and trained weights).
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np

F32 = np.float32
F64 = np.float64


# =========================================================================== quantizers (Section 3.2)

def uniform_quantize(x: np.ndarray, bits: int) -> Tuple[np.ndarray, float, int]:
    """Eq. 1-2, per tensor: asymmetric uniform quantizer.

    s = (max - min) / (2^b - 1);  z = clip(round(-min / s), 0, 2^b - 1);
    x_q = clip(round(x / s) + z, 0, 2^b - 1).
    Returns (codes int64, s, z).  A constant tensor (max == min) has s = 0 in Eq. 2;
    it is given s = 1 so that every code equals z.
    """
    x = np.asarray(x, dtype=F64)
    qmax = 2 ** bits - 1
    lo, hi = float(x.min()), float(x.max())
    s = (hi - lo) / qmax
    if s == 0.0:
        s = 1.0
    z = int(np.clip(np.rint(-lo / s), 0, qmax))
    xq = np.clip(np.rint(x / s) + z, 0, qmax).astype(np.int64)
    return xq, s, z


def quantize_rows_sym(X: np.ndarray, qmax: int = 127) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 1-2 with z = 0 and signed codes, one scale per row (per token for
    activations, per output channel for weights [N, K]).

    scale[r] = absmax_r / qmax (float32);  code = clip(round(x / scale[r]), -qmax, qmax).
    The quotient is formed in float32 (the code is an integer decision).
    A row of zeros gets scale 0 and codes 0.
    Returns (codes int8 [R, C], scale float32 [R]).
    """
    X = np.ascontiguousarray(X, dtype=F32)
    ax = np.max(np.abs(X), axis=1).astype(F32)
    scale = (ax / F32(qmax)).astype(F32)
    safe = np.where(scale > 0, scale, F32(1.0)).astype(F32)
    qf = np.rint((X / safe[:, None]).astype(F32))
    codes = np.clip(qf, -qmax, qmax).astype(np.int8)
    codes[scale == 0] = 0
    return codes, scale


def pack_int4(codes: np.ndarray) -> np.ndarray:
    """Two signed 4-bit codes per byte: element 2j in the low nibble, 2j+1 in the
    high nibble, two's complement.  [N, K] int8 in [-8, 7] -> [N, K/2] uint8."""
    c = np.asarray(codes).astype(np.int16)
    assert c.shape[-1] % 2 == 0 and c.min() >= -8 and c.max() <= 7
    lo = (c[..., 0::2] & 0xF).astype(np.uint8)
    hi = (c[..., 1::2] & 0xF).astype(np.uint8)
    return (lo | (hi << 4)).astype(np.uint8)


def unpack_int4(packed: np.ndarray) -> np.ndarray:
    """Inverse of :func:`pack_int4`: [N, K/2] uint8 -> [N, K] int8."""
    p = np.asarray(packed, dtype=np.uint8)
    lo = (p & 0xF).astype(np.int16)
    hi = (p >> 4).astype(np.int16)
    lo = np.where(lo >= 8, lo - 16, lo)
    hi = np.where(hi >= 8, hi - 16, hi)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.int8)
    out[..., 0::2] = lo
    out[..., 1::2] = hi
    return out


# =========================================================================== integer product (Section 3.4)

def int_matmul(Xq: np.ndarray, Wq: np.ndarray) -> np.ndarray:
    """The W_q x_q term of Eq. 7: acc[m, n] = sum_k Xq[m, k] * Wq[n, k], exact.

    Evaluated with a float64 matrix product: every product and every partial sum is
    an integer of magnitude <= 128^2 * K < 2^53, so float64 arithmetic is exact in
    any summation order.  Returned as int64.
    """
    Xq = np.asarray(Xq)
    Wq = np.asarray(Wq)
    K = Xq.shape[1]
    assert Wq.shape[1] == K and 128 * 128 * K < 2 ** 53
    acc = Xq.astype(F64) @ Wq.astype(F64).T
    return acc.astype(np.int64)


def conv2d_int_nhwc(Xq: np.ndarray, Wq: np.ndarray, stride: int = 1, pad: int = 0) -> np.ndarray:
    """Integer convolution by its definition (the paper places CWAC after every quantized convolution as well,
    Section 3.3): acc[b, ho, wo, n] = sum_{i, j, c} Xq[b, ho*stride + i - pad, wo*stride + j - pad, c] * Wq[n, i, j, c],
    positions outside the image contribute 0 (symmetric codes: zero-point 0).  Xq [B, H, W, C], Wq [N, kh, kw, C].
    Returns int64 [B, Ho, Wo, N]."""
    Xq = np.asarray(Xq, dtype=np.int64)
    Wq = np.asarray(Wq, dtype=np.int64)
    Bn, H, W, C = Xq.shape
    N, kh, kw, C2 = Wq.shape
    assert C == C2
    Ho = (H + 2 * pad - kh) // stride + 1
    Wo = (W + 2 * pad - kw) // stride + 1
    Xp = np.zeros((Bn, H + 2 * pad, W + 2 * pad, C), dtype=np.int64)
    Xp[:, pad:pad + H, pad:pad + W, :] = Xq
    acc = np.zeros((Bn, Ho, Wo, N), dtype=np.int64)
    for i in range(kh):
        for j in range(kw):
            patch = Xp[:, i:i + stride * (Ho - 1) + 1:stride, j:j + stride * (Wo - 1) + 1:stride, :]   # [B, Ho, Wo, C]
            acc += patch @ Wq[:, i, j, :].T
    return acc


def qlinear_eq7(Wq: np.ndarray, xq: np.ndarray, Zw: np.ndarray, Zx: int) -> np.ndarray:
    """Bracket of Eq. 7 for one input vector, with the sums the paper's notation leaves
    implicit:  sum_k (Wq[n,k] - Zw[n]) (xq[k] - Zx)
             = Wq xq - Zw[n] sum_k xq[k] - Zx sum_k Wq[n,k] + K Zx Zw[n].   (int64)"""
    Wq = np.asarray(Wq, dtype=np.int64)
    xq = np.asarray(xq, dtype=np.int64)
    Zw = np.asarray(Zw, dtype=np.int64)
    K = xq.shape[0]
    return Wq @ xq - Zw * xq.sum() - Zx * Wq.sum(axis=1) + K * Zx * Zw


def quantize_rows_asym(X: np.ndarray, bits: int = 8) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Eq. 1-2 applied to every row on its own (per token for activations, per output channel for weights):
    unsigned codes in [0, 2^b - 1], scale s_r = (max_r - min_r) / (2^b - 1), zero-point
    z_r = clip(round(-min_r / s_r), 0, 2^b - 1).  The quotients are formed in float32 (integer decisions).
    A constant row gets scale 1 (Eq. 2 would give 0).  Returns (codes uint8, scale float32, zero int32)."""
    X = np.ascontiguousarray(X, dtype=F32)
    qmax = F32(2 ** bits - 1)
    lo = X.min(axis=1).astype(F32)
    hi = X.max(axis=1).astype(F32)
    s = ((hi - lo) / qmax).astype(F32)
    s = np.where(s > 0, s, F32(1.0)).astype(F32)
    z = np.clip(np.rint((-lo / s).astype(F32)), 0, qmax).astype(np.int32)
    q = np.clip(np.rint((X / s[:, None]).astype(F32)) + z[:, None].astype(F32), 0, qmax)
    return q.astype(np.uint8), s, z


def int_matmul_asym(Xq: np.ndarray, Zx: np.ndarray, Wq: np.ndarray, Zw: np.ndarray) -> np.ndarray:
    """The bracket of Eq. 6 by its definition: acc[m, n] = sum_k (Wq[n, k] - Zw[n]) (Xq[m, k] - Zx[m]),
    exact (float64 product of small integers, every partial sum below 2^53).  Zx per row (a scalar broadcasts:
    the paper's per-tensor activation zero-point), Zw per output channel."""
    Xc = np.asarray(Xq, dtype=F64) - np.broadcast_to(np.asarray(Zx, dtype=F64), (np.shape(Xq)[0],))[:, None]
    Wc = np.asarray(Wq, dtype=F64) - np.asarray(Zw, dtype=F64)[:, None]
    assert 256 * 256 * Xc.shape[1] < 2 ** 53
    return (Xc @ Wc.T).astype(np.int64)


def dequant(acc: np.ndarray, x_scale: np.ndarray, w_scale: np.ndarray,
            bias: Optional[np.ndarray]) -> np.ndarray:
    """Eq. 6 with all zero-points 0: real-valued layer output
    y[m, n] = S_x[m] * S_W[n] * acc[m, n] (+ bias[n], which the engine adds separately)."""
    y = np.asarray(acc, dtype=F64) * np.asarray(x_scale, dtype=F64)[:, None] * np.asarray(w_scale, dtype=F64)[None, :]
    if bias is not None:
        y = y + np.asarray(bias, dtype=F64)[None, :]
    return y


# =========================================================================== CWAC (Section 3.3)

def cwac_apply(y: np.ndarray, a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Compensated output alpha (.) Y_quant + beta (Section 3.3, after Eq. 5)."""
    return np.asarray(a, dtype=F64)[None, :] * np.asarray(y, dtype=F64) + np.asarray(b, dtype=F64)[None, :]


def cwac_fit(fp_out: np.ndarray, q_out: np.ndarray, var_rel_eps: float = 1e-12
             ) -> Tuple[np.ndarray, np.ndarray, int]:
    """Eq. 3-5: per output channel c, the least-squares line through (q, f):

        alpha_c = Cov(f_c, q_c) / Var(q_c),   beta_c = E[f_c] - alpha_c E[q_c].

    Two-pass, mean-centred, float64.  (Normalising by R or R-1 cancels in alpha.)
    Degenerate channel (Var(q_c) <= var_rel_eps * E[q_c^2], i.e. a constant column, or
    a single row): every (alpha, beta = E[f] - alpha E[q]) minimises Eq. 3; alpha = 1 is
    chosen, so beta = E[f] - E[q].
    Returns (a float64 [C], b float64 [C], number of degenerate channels).
    """
    f = np.asarray(fp_out, dtype=F64)
    q = np.asarray(q_out, dtype=F64)
    assert f.shape == q.shape and f.ndim == 2
    R = f.shape[0]
    mq = q.sum(axis=0) / R
    mf = f.sum(axis=0) / R
    dq = q - mq[None, :]
    df = f - mf[None, :]
    var = (dq * dq).sum(axis=0) / R
    cov = (dq * df).sum(axis=0) / R
    msq = (q * q).sum(axis=0) / R
    degenerate = var <= var_rel_eps * msq
    a = np.where(degenerate, 1.0, cov / np.where(degenerate, 1.0, var))
    b = mf - a * mq
    return a, b, int(degenerate.sum())


def cwac_stats(fp_out: np.ndarray, q_out: np.ndarray) -> np.ndarray:
    """The five per-channel sums Eq. 4-5 are functions of: [n, sum q, sum f, sum q f, sum q^2]
    as float64 [5, C] (the streaming state of the calibration kernels)."""
    f = np.asarray(fp_out, dtype=F64)
    q = np.asarray(q_out, dtype=F64)
    n = np.full(f.shape[1], float(f.shape[0]))
    return np.stack([n, q.sum(0), f.sum(0), (q * f).sum(0), (q * q).sum(0)])


# =========================================================================== fold (Section 3.4, Eq. 9-11)

def cwac_fold(w_scale: np.ndarray, bias: Optional[np.ndarray], a: Optional[np.ndarray],
              b: Optional[np.ndarray]) -> Tuple[np.ndarray, np.ndarray]:
    """Absorb CWAC into the layer's requantization parameters.

    Eq. 9 puts alpha on the product and beta beside it; Eq. 11 moves alpha into the
    multiplier M' = alpha S_x S_W / S_r.  With a per-token S_x and a per-token S_r that
    are only known at run time, the static part of M' is  fs[n] = alpha[n] S_W[n]  and
    the additive part is  fb[n] = alpha[n] bias[n] + beta[n]  (CWAC acts on the module
    output, which includes the bias).  Missing bias = 0, missing (a, b) = (1, 0).
    """
    w_scale = np.asarray(w_scale, dtype=F64)
    n = w_scale.shape[0]
    a64 = np.ones(n) if a is None else np.asarray(a, dtype=F64)
    b64 = np.zeros(n) if b is None else np.asarray(b, dtype=F64)
    bias64 = np.zeros(n) if bias is None else np.asarray(bias, dtype=F64)
    return a64 * w_scale, a64 * bias64 + b64


def forward_folded(acc: np.ndarray, x_scale: np.ndarray, fs: np.ndarray, fb: np.ndarray) -> np.ndarray:
    """Right-hand side of Eq. 9 after folding: z[m, n] = acc[m, n] S_x[m] fs[n] + fb[n]."""
    return (np.asarray(acc, dtype=F64) * np.asarray(x_scale, dtype=F64)[:, None]
            * np.asarray(fs, dtype=F64)[None, :] + np.asarray(fb, dtype=F64)[None, :])


def fold_integer_offset(alpha, beta, S_x: float, S_W, S_r: float):
    """Eq. 10-11 as printed (static per-tensor S_x, S_r):
    M' = alpha S_x S_W / S_r  and the accumulator offset round(beta / (alpha S_x S_W))."""
    alpha = np.asarray(alpha, dtype=F64)
    beta = np.asarray(beta, dtype=F64)
    S_W = np.asarray(S_W, dtype=F64)
    Mp = alpha * S_x * S_W / S_r
    off = np.rint(beta / (alpha * S_x * S_W)).astype(np.int64)
    return Mp, off


def requant_static(acc, Mp, off, Z_r: int = 0, qmax: int = 127) -> np.ndarray:
    """Eq. 10 as printed, for an engine with static scales: r_q = Z_r + M' (acc + offset), rounded and clipped,

        r_q[m, n] = clip(round(M'[n] * (acc[m, n] + off[n])) + Z_r, -qmax, qmax).

    `acc` is the integer bracket of Eq. 7 (here W_q x_q, zero-points 0) and `off` the rounded
    beta / (alpha S_x S_W) of Eq. 10; their sum is exact integer arithmetic.  The product with the
    multiplier M' (Eq. 11) is formed in float32 (the code is an integer decision taken in the
    precision of the kernels): float32(acc + off) * float32(M').  Returns int8.
    """
    t = (np.asarray(acc, dtype=np.int64) + np.asarray(off, dtype=np.int64)[None, :]).astype(F32)
    prod = (t * np.asarray(Mp, dtype=F32)[None, :]).astype(F32)
    return np.clip(np.rint(prod) + Z_r, -qmax, qmax).astype(np.int8)


# =========================================================================== output stage

def requant_per_token(z: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 1-2 applied to the layer output with z = 0 and one dynamic scale per token
    (the S_r, Z_r = 0 of Eq. 7):  y_scale[m] = max_n |z[m, n]| / 127,
    Yq = clip(round(z / y_scale[m]), -127, 127).  z is first rounded to float32 and the
    quotient is formed in float32.  Returns (Yq int8, y_scale float32)."""
    z32 = np.asarray(z, dtype=F64).astype(F32)
    return quantize_rows_sym(z32, 127)


def to_bf16_bits(z: np.ndarray) -> np.ndarray:
    """float32(z) rounded to bfloat16 by round-to-nearest-even, returned as the 16-bit
    patterns (uint16).  bfloat16 = the upper 16 bits of IEEE binary32."""
    u = np.asarray(z, dtype=F64).astype(F32).view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = (u + 0x7FFF + lsb) >> 16
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(F32)


# =========================================================================== whole layer

def qlinear_cwac_reference(Xq, x_scale, Wq, w_scale, bias, a, b) -> np.ndarray:
    """Unfolded path: integer product -> Eq. 6 dequant (+bias) -> CWAC.  float64 [M, N]."""
    return cwac_apply(dequant(int_matmul(Xq, Wq), x_scale, w_scale, bias), a, b)


def linear_fp(X: np.ndarray, W: np.ndarray, bias: Optional[np.ndarray]) -> np.ndarray:
    """The full-precision module M_full of Section 3.3: X W^T + bias in float64."""
    y = np.asarray(X, dtype=F64) @ np.asarray(W, dtype=F64).T
    if bias is not None:
        y = y + np.asarray(bias, dtype=F64)[None, :]
    return y
