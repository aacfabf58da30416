"""Pins of the 8-bit storage checker (oracle/fp8_oracle.py) against what the E4M3 format itself fixes and against
torch's own float8_e4m3fn conversion (a library special case: finite, in-range values)."""
import numpy as np
import pytest
import torch

from oracle import fp8_oracle as Q


def test_decode_published_code_points():
    want = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x38: 1.0, 0x39: 1.125, 0x3C: 1.5,
            0x40: 2.0, 0x77: 240.0, 0x78: 256.0, 0x7E: 448.0, 0xC0: -2.0, 0xB8: -1.0, 0x81: -(2.0 ** -9)}
    for c, v in want.items():
        assert float(Q.e4m3_decode(np.uint8(c))) == v, hex(c)
    assert np.isnan(Q.e4m3_decode(np.uint8(0x7F))) and np.isnan(Q.e4m3_decode(np.uint8(0xFF)))
    # monotone over the positive finite codes
    pos = Q.e4m3_decode(np.arange(0, 0x7F, dtype=np.uint8))
    assert np.all(np.diff(pos) > 0)


def test_encode_round_trips_every_finite_code():
    codes = np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8)
    assert np.array_equal(Q.e4m3_encode(Q.e4m3_decode(codes)), codes)


def test_encode_ties_to_even_saturation_and_subnormals():
    enc = lambda v: int(Q.e4m3_encode(np.float32(v)))
    assert enc(1.0625) == 0x38            # halfway between 1.0 (m = 0) and 1.125 (m = 1): even mantissa
    assert enc(1.1875) == 0x3A            # halfway between 1.125 and 1.25 (m = 2)
    assert enc(1.0626) == 0x39
    assert enc(2.0 ** -10) == 0x00        # half of the smallest subnormal: tie to even = 0
    assert enc(1.5 * 2.0 ** -9) == 0x02   # tie between 1 and 2 subnormal steps
    assert enc(2.0 ** -9 * 7.5) == 0x08   # ties up into the normal range (7.5 -> 8 steps = 2^-6)
    assert enc(1000.0) == 0x7E and enc(-1e9) == 0xFE and enc(464.0) == 0x7E
    assert enc(-0.0) == 0x80 and enc(float("nan")) == 0x7F


def test_encode_matches_torch_float8_on_in_range_values():
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.normal(0, 1, 20000), rng.normal(0, 100, 20000), rng.uniform(-2 ** -6, 2 ** -6, 20000)])
    x = x[np.abs(x) <= 448.0].astype(np.float32)
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = Q.e4m3_encode(x)
    same = got == want
    zero = (got & 0x7F) == 0              # the sign of a value that rounds to zero may differ between libraries
    assert np.all(same | (zero & ((want & 0x7F) == 0)))


def test_quantize_rows_error_bound_and_exact_cases():
    rng = np.random.default_rng(6)
    w32 = rng.normal(0, 0.03, (64, 512)).astype(np.float32)
    bits = (w32.view(np.uint32) >> 16).astype(np.uint16)           # truncate to bf16 bit patterns
    w = (bits.astype(np.uint32) << 16).view(np.float32)
    codes, scales = Q.quantize_rows(bits)
    assert codes.shape == bits.shape and scales.shape == (64,)
    assert np.allclose(scales, np.max(np.abs(w), axis=1) / 448.0, rtol=1e-7)
    assert np.all(np.max(np.abs(Q.e4m3_decode(codes)), axis=1) == 448.0)   # the largest element maps to the top code
    back = (Q.dequantize_rows(codes, scales).astype(np.uint32) << 16).view(np.float32)
    # half a unit in the last place of the code (relative 2^-4 of the value's binade, at least half a subnormal step)
    # plus the bf16 rounding of the result
    q = np.abs(w / scales[:, None])
    half_ulp = np.where(q < 2.0 ** -6, 2.0 ** -10, np.exp2(np.floor(np.log2(np.maximum(q, 1e-30))) - 4.0))
    bound = half_ulp * scales[:, None] * (1 + 2.0 ** -7) + np.abs(w) * 2.0 ** -8
    assert np.all(np.abs(back - w) <= bound)
    # a row of powers of two within 2^9 of its largest element comes back exactly
    row = np.float32([2.0 ** -k for k in range(8)])[None] * np.float32(0.4375)   # 0.4375 * 2^-k, max maps to 448
    rb = (row.view(np.uint32) >> 16).astype(np.uint16)
    c, s = Q.quantize_rows(rb)
    assert np.array_equal(Q.dequantize_rows(c, s), rb)
    # an all-zero row: scale 1, codes 0
    c, s = Q.quantize_rows(np.zeros((1, 16), dtype=np.uint16))
    assert float(s[0]) == 1.0 and not c.any()


def test_a_planted_mistake_fails_a_pin():
    """Truncation instead of round-to-nearest-even would pass the round trip of exact codes: the tie cases catch it."""
    def enc_trunc(v):
        a = abs(float(v))
        ex = max(np.floor(np.log2(a)), -6.0)
        return np.floor(a / 2.0 ** (ex - 3)) * 2.0 ** (ex - 3)
    assert enc_trunc(1.1875) != float(Q.e4m3_decode(Q.e4m3_encode(np.float32(1.1875))))
