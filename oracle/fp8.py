"""FP8 E4M3 (the "fn" variant: finite only) for quantised K/V slabs.

Test infrastructure only.  Written from the format's definition: 1 sign bit, 4 exponent bits
(bias 7), 3 mantissa bits; exponent field 0 holds the subnormals m/8 * 2^-6; there are no
infinities, and S.1111.111 is the only NaN, so the largest finite value is 1.75 * 2^8 = 448.

The paper names quantisation as a complement to budget allocation without fixing a scheme; the
scheme here: one fp32 scale per (layer, KV head) for K and one for V, a row element x is stored as
code = encode(fl32(x) * fl32(1 / scale)) with round-to-nearest-even and saturation to +-448, and
stands for the value decode(code) * scale in every later step.
"""
import numpy as np

MAX_FINITE = 448.0


def decode(codes):
    """uint8 codes -> float64 values (NaN for 0x7f / 0xff)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    normal = (1.0 + m / 8.0) * np.exp2(e.astype(np.float64) - 7.0)
    subnormal = (m / 8.0) * 2.0 ** -6
    val = np.where(e == 0, subnormal, normal)
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return sign * val


def encode(x):
    """float values -> uint8 codes: round to nearest representable value, ties to the even mantissa,
    magnitudes beyond 448 saturate to 448 (no infinities).  Exact arithmetic on the given values."""
    x = np.asarray(x, dtype=np.float64)
    a = np.minimum(np.abs(x), MAX_FINITE)
    # spacing of the grid around a: 2^(floor(log2 a) - 3) for normals, 2^-9 below 2^-6
    with np.errstate(divide="ignore"):
        ex = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    ex = np.clip(ex, -6, 8)
    step = np.exp2(ex - 3.0)
    q = a / step                                   # exact: a power-of-two division
    r = np.floor(q)
    frac = q - r
    up = (frac > 0.5) | ((frac == 0.5) & (np.mod(r, 2) == 1))
    n = r + up                                     # multiples of `step`: 0 .. 16
    val = n * step                                 # may have carried into the next binade: still on the grid
    val = np.minimum(val, MAX_FINITE)
    # value -> fields
    with np.errstate(divide="ignore"):
        e2 = np.floor(np.log2(np.where(val > 0, val, 1.0)))
    is_sub = val < 2.0 ** -6
    efield = np.where(is_sub, 0, e2 + 7).astype(np.int64)
    mfield = np.where(is_sub, np.rint(val * 2.0 ** 9), np.rint((val / np.exp2(e2) - 1.0) * 8.0)).astype(np.int64)
    code = (efield << 3) | mfield
    code = np.where(np.signbit(x), code | 0x80, code)
    return code.astype(np.uint8)


def quantise_rows(rows, scale, inv_scale):
    """rows (any float array) -> (codes uint8, dequantised float64 values) under one scale.
    The product with the inverse scale is taken in float32, as the stored code is defined."""
    x32 = np.asarray(rows, dtype=np.float32) * np.float32(inv_scale)
    codes = encode(x32.astype(np.float64))
    return codes, decode(codes) * float(np.float32(scale))
