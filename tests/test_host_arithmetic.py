"""Host-side checks of arithmetic choices the CUDA kernels rely on (no GPU needed).

The quantise kernel divides in fp32 (IEEE, round to nearest) and rounds the quotient to
the nearest-even integer.  These tests show, over every bf16 magnitude and a dense sample
of scales, that this gives the integer the exact-rational definition gives, and that the
cheaper reciprocal-multiply would not - unless, as the kernel does, every quotient that comes
within 2^-13 of a half-integer is sent back to the division.
"""
import numpy as np

from oracle import w4a8_oracle as onp


def all_positive_bf16():
    bits = np.arange(0x0001, 0x7F80, dtype=np.uint16)          # every positive finite bf16
    return bits, onp.bf16_bits_to_f64(bits)


def test_fp32_scale_equals_exact_scale_for_every_bf16_amax():
    _, amax = all_positive_bf16()
    exact = np.minimum(amax / 127.0, 65504.0).astype(np.float16)                    # fp64 quotient, one rounding
    q32 = (amax.astype(np.float32) / np.float32(127.0))
    gpu = np.minimum(q32, np.float32(65504.0)).astype(np.float16)                   # what the kernel does
    assert np.array_equal(exact.view(np.uint16), gpu.view(np.uint16))


def test_fp32_division_rounds_like_exact_division():
    bits, x = all_positive_bf16()
    rng = np.random.default_rng(0)
    # scales: every 37th fp16 value plus the scales that real rows produce
    s_bits = np.concatenate([np.arange(1, 0x7C00, 37, dtype=np.uint16),
                             onp.f64_to_fp16_bits(np.minimum(x[rng.integers(0, len(x), 300)] / 127.0, 65504.0))])
    s_bits = s_bits[s_bits != 0]
    recip_mismatch = 0
    for sb in s_bits:
        s64 = float(onp.fp16_bits_to_f64(np.array([sb]))[0])
        sel = x <= 128.0 * s64                       # quotients beyond 128 clamp in every variant
        xs = x[sel]
        exact = np.clip(np.rint(xs / s64), -127, 127)
        q32 = xs.astype(np.float32) / np.float32(s64)
        assert np.array_equal(np.clip(np.rint(q32), -127, 127), exact), hex(int(sb))
        with np.errstate(over="ignore"):
            r32 = xs.astype(np.float32) * (np.float32(1.0) / np.float32(s64))
        recip_mismatch += int(np.count_nonzero(np.clip(np.rint(r32), -127, 127) != exact))
    assert recip_mismatch > 0          # the shortcut the kernel must not take does break ties


def test_reciprocal_with_tie_fallback_rounds_like_exact_division():
    """The kernel's fast path, step by step in fp32: t = x * (1 / s); y = t + 1.5 * 2^23 rounds t to an integer
    (ties to even) in y's low mantissa bits; n = y - 1.5 * 2^23; |t - n| > 1/2 - 2^-13 marks a quotient that may be
    an exact tie, and only those take the IEEE division.  A quotient of a bf16 by an fp16 that is not a tie is at
    least 2^-12 away from one, t is within 2^-16 of it: the fast path can never be on the wrong side."""
    bits, x = all_positive_bf16()
    rng = np.random.default_rng(1)
    s_bits = np.concatenate([np.arange(1, 0x7C00, 37, dtype=np.uint16),
                             onp.f64_to_fp16_bits(np.minimum(x[rng.integers(0, len(x), 300)] / 127.0, 65504.0))])
    s_bits = s_bits[s_bits != 0]
    magic = np.float32(12582912.0)
    slow = 0
    total = 0
    for sb in s_bits:
        s64 = float(onp.fp16_bits_to_f64(np.array([sb]))[0])
        # a row's values never exceed its maximum, and the scale is the maximum / 127 rounded to fp16:
        # quotients stay below 127 * (1 + 2^-11) unless the scale saturated (those rows take the division)
        xs = x[x <= 127.0 * (1.0 + 2.0 ** -10) * s64]
        exact = np.rint(xs / s64)
        s32 = np.float32(s64)
        with np.errstate(over="ignore"):
            t = xs.astype(np.float32) * (np.float32(1.0) / s32)
        y = t + magic
        n = y - magic
        code_fast = (y.view(np.uint32) & 0xFF).astype(np.int64)            # the low mantissa byte is the code
        suspect = np.abs(t - n) > np.float32(0.5 - 2.0 ** -13)
        code = np.where(suspect, np.rint(xs.astype(np.float32) / s32).astype(np.int64), code_fast)
        assert np.array_equal(code, exact.astype(np.int64)), hex(int(sb))
        assert exact.max(initial=0) <= 127
        # every exact tie must have been sent to the division
        ties = (2.0 * xs / s64) % 2.0 == 1.0
        assert np.all(suspect[ties])
        slow += int(suspect.sum())
        total += len(xs)
    assert slow < total / 200          # the division is the rare path


def test_zero_point_byte_trick():
    """((q | 0x80) - z) ^ 0x80 is q - z as a signed byte for q, z in 0..15 (no borrow between bytes)."""
    for q in range(16):
        for z in range(16):
            v = (((q | 0x80) - z) ^ 0x80) & 0xFF
            assert np.int8(np.uint8(v)) == q - z
    q = np.uint32(0x000F0F00)
    zz = np.uint32(0x0F000F0F)
    out = ((q | np.uint32(0x80808080)) - zz) ^ np.uint32(0x80808080)
    assert np.array([out], dtype=np.uint32).view(np.int8).tolist() == [-15, 0, 15, -15]     # little-endian bytes


def test_drain_integer_range_fits_fp32_exactly():
    assert 128 * 15 * 127 < 2 ** 24
