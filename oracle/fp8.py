"""The FP8 verifier cache's number format (test infrastructure).

The paper names no FP8 cache; the serving variant stores the target's K/V as e4m3 bytes with one scale per
(page, KV head) so that the bytes Eq. 2's beta L d term counts are halved.  What an element stands for is fixed
by the library's contract, restated here from its definition:

    value = fp16( e4m3(byte) * fp16(scale) )            (both roundings to nearest, ties to even)

e4m3 ("fn" flavour): 1 sign bit, 4 exponent bits (bias 7), 3 mantissa bits; exponent field 0 holds subnormals
m/8 * 2^-6; there are no infinities, and the one NaN pattern is S.1111.111; the largest finite value is 448.
Attention over such a cache is then the plain definition (oracle.verify_attend) on the dequantised values, with
q rounded to fp16 as well.
"""
import numpy as np


def e4m3_to_f64(bits):
    """Exact value of each e4m3 byte as float64 (NaN for the NaN pattern)."""
    b = np.asarray(bits, dtype=np.uint8).astype(np.int64)
    sign = np.where(b & 0x80, -1.0, 1.0)
    e = (b >> 3) & 0xF
    m = b & 0x7
    normal = (1.0 + m / 8.0) * np.exp2(e.astype(np.float64) - 7.0)
    sub = (m / 8.0) * 2.0 ** -6
    val = np.where(e == 0, sub, normal)
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return sign * val


def fp16_round(x):
    """Round float64 values to fp16 (nearest, ties to even; subnormals kept) and return them as float64."""
    return np.asarray(x, dtype=np.float64).astype(np.float16).astype(np.float64)


def dequantize_e4m3(bits, scale):
    """fp16(e4m3(byte) * fp16(scale)); `scale` broadcasts against `bits`.  The product of an e4m3 value (4
    significant bits) and an fp16 value (11) is exact in float64, so only the final rounding acts."""
    return fp16_round(e4m3_to_f64(bits) * fp16_round(scale))
