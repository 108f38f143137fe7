"""Tolerances of the parity tests.

FP32 outputs: the kernel forms z with three FP32 roundings (int->float is exact below 2^24, the row-scale product,
the fused multiply-add), the oracle in float64: |d| <= 1e-5 |ref| + 1e-6 leaves two orders of magnitude of room.
INT8 codes: both sides round an FP32 quotient; they may disagree where it lies within a few 1e-6 of a half-integer,
which is rare (about one code in a million measured): at most 1 LSB on at most 0.01 % of the elements.
BF16 outputs: the bits of bf16_rne(float32(z_oracle)), except that the kernel rounds ITS FP32 z, which may sit on the
other side of a bf16 rounding boundary: at most one bf16 ulp on at most 0.01 % of the elements.  Where z nearly
cancels (|z| below 1e-4, i.e. a hundred times the FP32 absolute tolerance) an FP32 error of 1e-9 already moves several
bf16 ulps of that tiny number; those elements are held to the FP32 tolerance instead.
CWAC a, b: FP32 results of float64 sums, 1e-5 relative (b with an absolute floor of 1e-6 of the channel's scale)."""
import numpy as np

FP32_REL = 1e-5      # dequantized + compensated outputs: |d| <= 1e-5 |ref| + 1e-6
FP32_ABS = 1e-6
CODE_MAX_LSB = 1     # requantized INT8 codes: at most 1 LSB ...
CODE_MAX_FRAC = 1e-4  # ... on at most 0.01 % of the elements
AB_REL = 1e-5        # CWAC a, b


def assert_fp32_close(got, ref, what="z"):
    ref = np.asarray(ref, dtype=np.float64)
    d = np.abs(np.asarray(got, dtype=np.float64) - ref)
    lim = FP32_REL * np.abs(ref) + FP32_ABS
    bad = d > lim
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside tolerance, worst excess {np.max(d - lim):.3e}"


def assert_codes_close(got, ref, what="codes"):
    d = np.abs(got.astype(np.int32) - ref.astype(np.int32))
    assert d.max(initial=0) <= CODE_MAX_LSB, f"{what}: a code differs by {d.max()} LSB"
    frac = np.count_nonzero(d) / max(d.size, 1)
    # tiny outputs: allow a single element
    assert frac <= CODE_MAX_FRAC or np.count_nonzero(d) <= 1, f"{what}: {frac:.3e} of the codes differ"


def assert_ab_close(a, b, a_ref, b_ref, scale_b):
    """a: plain relative.  b: relative with an absolute floor of 1e-6 x the channel's natural scale."""
    a_ref = np.asarray(a_ref, dtype=np.float64)
    b_ref = np.asarray(b_ref, dtype=np.float64)
    da = np.abs(a - a_ref)
    assert np.all(da <= AB_REL * np.abs(a_ref)), f"a: worst rel {np.max(da / np.maximum(np.abs(a_ref), 1e-30)):.3e}"
    db = np.abs(b - b_ref)
    lim = AB_REL * np.abs(b_ref) + 1e-6 * np.asarray(scale_b)
    assert np.all(db <= lim), f"b: worst excess {np.max(db - lim):.3e}"


BF16_TINY = 1e-4     # |z| below this: compared as values (the FP32 tolerance), not as bf16 bit patterns


def assert_bf16_close(bits, z_ref, to_bf16_bits, bf16_bits_to_f32, what="bf16"):
    """bits: uint16 patterns from the kernel; z_ref: float64 oracle values; the two converters are the oracle's."""
    z_ref = np.asarray(z_ref, dtype=np.float64)
    bits = np.asarray(bits).astype(np.uint16)
    ref_bits = to_bf16_bits(z_ref)
    d = np.abs(bits.astype(np.int32) - ref_bits.astype(np.int32))
    tiny = np.abs(z_ref) < BF16_TINY
    big = ~tiny
    assert d[big].max(initial=0) <= 1, f"{what}: {d[big].max()} bf16 ulps off"
    assert np.count_nonzero(d[big]) <= max(1, int(1e-4 * d.size)), f"{what}: {np.count_nonzero(d[big])} elements differ"
    if tiny.any():
        got = bf16_bits_to_f32(bits[tiny]).astype(np.float64)
        err = np.abs(got - z_ref[tiny])
        assert np.all(err <= 2.0 ** -8 * np.abs(z_ref[tiny]) + FP32_ABS), f"{what}: tiny element off by {err.max():.3e}"
