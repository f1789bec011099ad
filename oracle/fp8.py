"""CPU oracle for the FP8 (e4m3) K/V cache variant (test infrastructure, not the product).

The paper keeps its dual cache in the model's dtype; an 8-bit cache is an extension (it halves the
cache footprint) with no passage to cite.  What the variant computes is fixed here: a cached value is
    bf16( decode_e4m3(code) * scale[sequence, kv head] )         (product and rounding in fp32 -> bf16)
and the attention over those values is the masked attention of Section 3.3 unchanged.

e4m3 ("FN" flavour, the one CUDA and torch implement): 1 sign bit, 4 exponent bits with bias 7,
3 mantissa bits; exponent field 0 = subnormals (mantissa / 8 * 2^-6); no infinities; the code with
all exponent and mantissa bits set (0x7f / 0xff) is NaN; the largest finite value is 448.
"""
import numpy as np


def decode_e4m3(codes):
    """uint8 codes -> float64 values, from the format definition."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    normal = (1.0 + m / 8.0) * np.exp2(e.astype(np.float64) - 7.0)
    sub = (m / 8.0) * 2.0 ** -6
    v = np.where(e == 0, sub, normal)
    v = np.where((e == 15) & (m == 7), np.nan, v)
    return sign * v


def bf16_round(x32):
    """float32 -> the nearest bf16 (ties to even), returned as float32."""
    x32 = np.ascontiguousarray(x32, dtype=np.float32)
    bits = x32.view(np.uint32).astype(np.uint64)
    rounded = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32)


def dequant_cache(codes, scale=None):
    """codes uint8 [S, Nc, Hkv, d], scale fp32 [S, Hkv] (None = 1) -> the cache the attention sees,
    as float32 holding bf16 values."""
    v = decode_e4m3(codes).astype(np.float32)       # every e4m3 value is exact in fp32
    if scale is not None:
        v = v * np.asarray(scale, dtype=np.float32)[:, None, :, None]
    return bf16_round(v)
