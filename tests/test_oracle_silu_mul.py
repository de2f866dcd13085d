"""Pins of the oracle's gated-MLP activation (h = silu(G) * U rounded once to BF16) against what
the mathematics fixes: special values, the identity silu(g) - silu(-g) = g, the limits, values
computed with Python's math module, and the BF16 rounding helper against exactly representable
values, ties and the float32 route where that one is exact."""
import math
import struct

import numpy as np

import oracle


def _bf16(v):
    """BF16 bit pattern of a value that BF16 represents exactly."""
    b = struct.unpack("<I", struct.pack("<f", v))[0]
    assert b & 0xFFFF == 0, v
    return b >> 16


def _row(gs, us):
    return np.array([[_bf16(g) for g in gs] + [_bf16(u) for u in us]], dtype=np.uint16)


def test_special_values_and_limits():
    h = oracle.silu_mul_f64(_row([0.0, 32.0, -32.0, 1.0], [3.0, 0.5, 2.0, 0.0]))[0]
    assert h[0] == 0.0                                   # silu(0) = 0
    assert abs(h[1] - 16.0) < 16.0 * 1e-13               # silu(g) -> g for large g
    assert abs(h[2]) < 1e-11                             # silu(g) -> 0 for very negative g
    assert h[3] == 0.0                                   # times up = 0


def test_identity_silu_minus_silu_of_negative_is_identity():
    gs = [0.125, 0.5, 1.0, 2.5, 7.0, 0.0078125]
    hp = oracle.silu_mul_f64(_row(gs, [1.0] * len(gs)))[0]
    hn = oracle.silu_mul_f64(_row([-g for g in gs], [1.0] * len(gs)))[0]
    for g, a, b in zip(gs, hp, hn):
        assert abs((a - b) - g) <= 1e-15 * max(1.0, g), (g, a, b)


def test_against_python_math():
    gs = [1.0, -1.0, 0.75, -3.5, 5.0, -0.0625]
    us = [2.0, 1.5, -4.0, 0.25, -1.0, 8.0]
    h = oracle.silu_mul_f64(_row(gs, us))[0]
    for g, u, v in zip(gs, us, h):
        want = g / (1.0 + math.exp(-g)) * u
        assert abs(v - want) <= 4e-16 * abs(want), (g, u, v, want)
    # a transposed operand or a swapped half would change these
    assert abs(h[0] - 2.0 * 0.7310585786300049) < 1e-15
    assert abs(h[3] - (-3.5 / (1.0 + math.exp(3.5))) * 0.25) < 1e-16


def test_bf16_rounding_helper():
    exact = np.array([1.0, -2.5, 0.0078125, 448.0, 3.0e-3 * 0 + 0.0], dtype=np.float64)
    bits = oracle.f64_to_bf16(exact)
    assert [int(b) for b in bits[:4]] == [_bf16(1.0), _bf16(-2.5), _bf16(0.0078125), _bf16(448.0)]
    assert int(bits[4]) == 0
    # ties go to the even mantissa: 1 + 2^-8 is half way between 1 and 1 + 2^-7
    assert int(oracle.f64_to_bf16(np.array([1.0 + 2.0 ** -8]))[0]) == _bf16(1.0)
    assert int(oracle.f64_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0]) == _bf16(1.0 + 2.0 ** -6)
    # just above a tie rounds up although rounding to float32 first would land on the tie
    assert int(oracle.f64_to_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0]) == _bf16(1.0 + 2.0 ** -7)
    # mantissa carry into the exponent
    assert int(oracle.f64_to_bf16(np.array([2.0 - 2.0 ** -9]))[0]) == _bf16(2.0)
    # agrees with the float32 route on float32 inputs (no double rounding there)
    rng = np.random.default_rng(3)
    x32 = rng.standard_normal(4096).astype(np.float32)
    assert np.array_equal(oracle.f64_to_bf16(x32.astype(np.float64)), oracle.f32_to_bf16(x32))


def test_rounded_result_is_the_nearest_bf16():
    rng = np.random.default_rng(5)
    gu = oracle.f32_to_bf16(rng.standard_normal((3, 64)).astype(np.float32) * 2.0)
    h64 = oracle.silu_mul_f64(gu)
    hb = oracle.bf16_to_f32(oracle.silu_mul(gu)).astype(np.float64)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(h64), 1e-30))) - 7)
    assert np.all(np.abs(hb - h64) <= 0.5 * ulp * (1 + 1e-12))
