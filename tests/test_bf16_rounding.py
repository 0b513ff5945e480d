"""The two bfloat16 helpers of the harness, pinned bit by bit.

Gradients may be handed to the library as bfloat16.  The harness rounds the fp32 draw once, to
nearest with ties to even (inputs.f32_to_bf16_bits), both sides then read the same 16-bit patterns,
and the oracle widens them exactly (oracle.bf16_to_f64).  bfloat16 is the upper half of an IEEE
binary32 word (1 sign, 8 exponent, 7 fraction bits), so every expected value below follows from the
format alone and is written out by hand.
"""
import numpy as np
import pytest

import oracle
from paper_2104_11981_b200 import inputs


def _f32(bits):
    return np.array(bits, dtype=np.uint32).view(np.float32)


# (fp32 bit pattern, expected bf16 bit pattern, why)
ROUNDING_CASES = [
    (0x3F800000, 0x3F80, "1.0 is representable"),
    (0x3F808000, 0x3F80, "tie, kept half is even (..80): rounds down to even"),
    (0x3F818000, 0x3F82, "tie, kept half is odd (..81): rounds up to even"),
    (0x3F808001, 0x3F81, "just above a tie: up"),
    (0x3F807FFF, 0x3F80, "just below a tie: down"),
    (0x3FFF8000, 0x4000, "tie on an all-ones fraction: carry into the exponent (1.9960938 -> 2.0)"),
    (0x3FFFFFFF, 0x4000, "largest fp32 below 2.0: carries into the exponent"),
    (0x00000000, 0x0000, "+0"),
    (0x80000000, 0x8000, "-0 keeps its sign"),
    (0x7F7F0000, 0x7F7F, "largest finite bfloat16 stays"),
    (0x7F7F7FFF, 0x7F7F, "below the tie above the largest finite bfloat16"),
    (0x7F7F8000, 0x7F80, "tie above the largest finite value, kept half odd: overflows to +inf"),
    (0x7F7FFFFF, 0x7F80, "largest finite fp32 overflows to +inf"),
    (0xFF7FFFFF, 0xFF80, "and to -inf on the negative side"),
    (0x7F800000, 0x7F80, "+inf stays"),
    (0xBF808000, 0xBF80, "negative tie to even: sign does not matter"),
    (0xBF818000, 0xBF82, "negative tie, odd kept half"),
    (0x00008000, 0x0000, "subnormal tie to even (zero)"),
    (0x00018000, 0x0002, "subnormal tie, odd kept half"),
    (0x3A83126F, 0x3A83, "1e-3 (a typical gradient magnitude): low half 0x126F is below the tie"),
]


@pytest.mark.parametrize("bits32,bits16,why", ROUNDING_CASES)
def test_f32_to_bf16_bits_hand_picked(bits32, bits16, why):
    got = int(inputs.f32_to_bf16_bits(_f32([bits32]))[0])
    assert got == bits16, (hex(bits32), hex(got), hex(bits16), why)


def test_f32_to_bf16_bits_is_nearest_and_even_on_random_values():
    """Against the definition, in exact integer arithmetic: the result is one of the two neighbouring
    bfloat16 values, no farther from the input than the other, and even on a tie."""
    rng = np.random.Generator(np.random.Philox(5))
    u = rng.integers(0, 0x7F000000, size=200_000, dtype=np.uint64)          # positive finite, far from overflow
    u[:1000] = (u[:1000] & ~np.uint64(0xFFFF)) | np.uint64(0x8000)           # plant exact ties
    got = inputs.f32_to_bf16_bits(u.astype(np.uint32).view(np.float32)).astype(np.uint64)
    lo = u >> np.uint64(16)
    hi = lo + np.uint64(1)
    assert np.all((got == lo) | (got == hi))
    # for positive floats the integer bit patterns are ordered like the values and, within one binade or
    # across a carry, distances between neighbours are proportional to bit-pattern distances
    d_got = np.abs((got << np.uint64(16)).astype(np.int64) - u.astype(np.int64))
    d_other = np.abs((np.where(got == lo, hi, lo) << np.uint64(16)).astype(np.int64) - u.astype(np.int64))
    assert np.all(d_got <= d_other)
    ties = d_got == d_other
    assert ties.sum() >= 1000 and np.all(got[ties] % 2 == 0)


def test_bf16_to_f64_hand_picked():
    cases = [(0x3F80, 1.0), (0xBF80, -1.0), (0x4000, 2.0), (0x3F81, 1.0078125), (0x3A83, 0.0009994506835937500),
             (0x0000, 0.0), (0x7F7F, 3.3895313892515355e38), (0x0080, 2.0 ** -126), (0x0001, 2.0 ** -133),
             (0xC2F7, -123.5)]
    bits = np.array([c[0] for c in cases], dtype=np.uint16)
    got = oracle.bf16_to_f64(bits)
    assert got.dtype == np.float64
    for (b, want), g in zip(cases, got):
        assert g == want, (hex(b), g, want)
    assert np.signbit(oracle.bf16_to_f64(np.array([0x8000], dtype=np.uint16))[0])
    assert np.isinf(oracle.bf16_to_f64(np.array([0x7F80], dtype=np.uint16))[0])


def test_round_then_widen_is_within_half_an_ulp():
    """Composition: |widen(round(v)) - v| <= 2^-8 |v| (half a unit in the last of bfloat16's 8
    significant bits is 2^-8 of the leading bit), and values that are already bfloat16 come back unchanged."""
    v = inputs.normal_np((4096,), 1e-3, 17)
    back = oracle.bf16_to_f64(inputs.f32_to_bf16_bits(v))
    assert np.all(np.abs(back - v.astype(np.float64)) <= 2.0 ** -8 * np.abs(v.astype(np.float64)))
    again = oracle.bf16_to_f64(inputs.f32_to_bf16_bits(back.astype(np.float32)))
    assert np.array_equal(again, back)
    assert np.array_equal(inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(v)).astype(np.float64), back)


def test_torch_conversion_matches_the_harness_rounding():
    """Full-size gradients are rounded on the device by torch's float32 -> bfloat16 conversion; here
    the same conversion on the CPU is held against the pinned helper, ties included."""
    import torch
    pats = np.array([c[0] for c in ROUNDING_CASES if c[0] & 0x7F800000 != 0x7F800000 or c[0] == 0x7F800000],
                    dtype=np.uint32)
    rnd = inputs.normal_np((100_000,), 1e-3, 23).view(np.uint32)
    ties = (rnd[:2000] & np.uint32(0xFFFF0000)) | np.uint32(0x8000)
    allbits = np.concatenate([pats, rnd, ties])
    f = allbits.view(np.float32)
    got = torch.from_numpy(f.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, inputs.f32_to_bf16_bits(f))
