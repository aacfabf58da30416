"""CPU checker for 8-bit expert storage on the host link.  TEST INFRASTRUCTURE ONLY.

The paper names bit-width adaptation only as the earlier route to cheaper expert offloading
(Section 2.3, first paragraph; Section 5, "Inference Efficiency"); it defines no format.  The
reading taken here: an expert's packed rows are kept on the host as FP8 E4M3 codes (the OCP
8-bit floating point format: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no
infinities, S.1111.111 = NaN, largest finite value 448) with one fp32 scale per row, and are
widened back to bf16 on the device before the layer reads them.

    scale = max|w| / 448          (fp32; 1 if the row is all zeros)
    code  = e4m3_rne(w / scale)   (fp32 division, round to nearest even, saturating)
    w'    = bf16_rne(e4m3_value(code) * scale)   (fp32 product)

Every decision that picks an integer code is taken in fp32, as on the device.  Shares no code
with the CUDA sources; numpy only.

Pinned by tests: e4m3_decode (the format's published code points), e4m3_encode (round trip of
all finite codes, ties to even, saturation, subnormals), quantize_rows / dequantize_rows
(error bound of half a unit in the last place of the code, exact powers of two).
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0


def e4m3_decode(code) -> np.ndarray:
    """Value of an E4M3 code (uint8) as fp32: (-1)^s * 2^(e-7) * (1 + m/8) for e > 0,
    (-1)^s * 2^-6 * (m/8) for e = 0; S.1111.111 is NaN."""
    c = np.asarray(code, dtype=np.uint8).astype(np.int32)
    s = (c >> 7) & 1
    e = (c >> 3) & 15
    m = c & 7
    mag = np.where(e == 0, m.astype(np.float64) / 8.0 * 2.0 ** -6,
                   (1.0 + m.astype(np.float64) / 8.0) * np.exp2(e.astype(np.float64) - 7.0))
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return (np.where(s == 1, -mag, mag)).astype(np.float32)


def e4m3_encode(x) -> np.ndarray:
    """fp32 -> E4M3 code, round to nearest even, magnitudes beyond 448 saturate to 448
    (no infinity exists in the format); NaN -> 0x7F.  Written out from the format: find the
    spacing of representable values at |x| (2^(e-7-3) above the subnormal range, 2^-9 inside
    it), round |x| / spacing to an integer with ties to even, re-normalise."""
    x = np.asarray(x, dtype=np.float32)
    a = np.abs(x).astype(np.float64)
    sign = np.signbit(x).astype(np.uint8) << 7
    out = np.zeros(x.shape, dtype=np.uint8)
    nan = np.isnan(x)
    a = np.where(nan, 0.0, a)
    a = np.minimum(a, E4M3_MAX)
    # exponent of the binade, clamped to the subnormal range's spacing
    with np.errstate(divide="ignore"):
        ex = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    ex = np.maximum(ex, -6.0)                      # below 2^-6 the spacing stays 2^-9
    step = np.exp2(ex - 3.0)
    q = a / step                                   # exact: a is fp32, step a power of two
    r = np.rint(q)                                 # numpy rounds halves to even
    val = r * step                                 # may have carried into the next binade
    val = np.minimum(val, E4M3_MAX)
    # re-derive the fields from the rounded value
    with np.errstate(divide="ignore"):
        e2 = np.floor(np.log2(np.where(val > 0, val, 1.0)))
    sub = val < 2.0 ** -6
    efield = np.where(sub, 0, e2 + 7).astype(np.int32)
    mfield = np.where(sub, np.rint(val / 2.0 ** -9), np.rint((val / np.exp2(e2) - 1.0) * 8.0)).astype(np.int32)
    out = (sign | (efield.astype(np.uint8) << 3) | mfield.astype(np.uint8)).astype(np.uint8)
    out = np.where(val == 0, sign, out).astype(np.uint8)
    out = np.where(nan, np.uint8(0x7F), out).astype(np.uint8)
    return out


def _bf16_rne_bits(v32: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit pattern (uint16), round to nearest even (finite inputs)."""
    b = np.asarray(v32, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (b >> 16) & 1
    return ((b + 0x7FFF + lsb) >> 16).astype(np.uint16)


def quantize_rows(w_bits: np.ndarray):
    """w_bits: [..., n] bf16 bit patterns (uint16).  One scale per last-axis row.
    Returns (codes uint8 [..., n], scales fp32 [...])."""
    w = (np.asarray(w_bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)
    amax = np.max(np.abs(w), axis=-1)
    scale = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    q = (w / scale[..., None]).astype(np.float32)
    return e4m3_encode(q), scale


def dequantize_rows(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """bf16 bit patterns of e4m3_value(code) * scale (fp32 product, one rounding to bf16)."""
    v = (e4m3_decode(codes) * np.asarray(scales, dtype=np.float32)[..., None]).astype(np.float32)
    return _bf16_rne_bits(v)
