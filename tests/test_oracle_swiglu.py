"""Pins of the oracle's gated activation h = Swish(gate) * up, rounded once to bf16 (CPU only).

The function is held to things it does not compute itself: closed forms of Swish, the reflection identity
Swish(g) - Swish(-g) = g, its limits, and a brute-force nearest-bf16 search for the rounding."""
import numpy as np
import pytest

from paper_2601_22347_b200 import inputs


def bits_of(values):
    return inputs.f32_to_bf16_bits(np.asarray(values, np.float32))


def vals_of(bits):
    return inputs.bf16_to_f64(np.asarray(bits, np.uint16))


ALL_FINITE = np.array([b for b in range(0x10000) if (b & 0x7F80) != 0x7F80], np.uint16)      # every finite bf16
ALL_VALUES = vals_of(ALL_FINITE)


def nearest_bf16_brute_force(v: float) -> int:
    """Nearest finite bf16 to v by search over all of them; ties to the even bit pattern."""
    dist = np.abs(ALL_VALUES - v)
    best = dist.min()
    cand = ALL_FINITE[dist == best]
    if cand.size == 1:
        return int(cand[0])
    cand = [int(c) for c in cand if (np.signbit(vals_of([c])[0]) == np.signbit(v)) or v == 0.0] or [int(c) for c in cand]
    even = [c for c in cand if c % 2 == 0]
    return even[0] if even else cand[0]


def test_swish_closed_forms(oracle):
    one = bits_of([[1.0]])
    # Swish(0) * u = 0 for every u; Swish(g) * 0 = 0
    g = bits_of([[0.0, 0.0, 3.0, -2.0]])
    u = bits_of([[5.0, -7.0, 0.0, 0.0]])
    assert np.all(vals_of(oracle.swiglu(g, u)) == 0.0)
    # Swish(1) = 1 / (1 + e^-1), rounded to bf16 by brute force
    got = int(oracle.swiglu(one, one)[0, 0])
    assert got == nearest_bf16_brute_force(1.0 / (1.0 + np.exp(-1.0)))
    # far out: Swish(g) = g up to far less than a bf16 rounding for g >= 40, and 0 (to bf16 subnormal precision) for g <= -110
    big = bits_of([[40.0, 64.0, 100.0]])
    assert np.array_equal(oracle.swiglu(big, bits_of([[1.0, 1.0, 1.0]])), big)
    neg = bits_of([[-110.0, -200.0]])
    assert np.all(vals_of(oracle.swiglu(neg, bits_of([[1.0, 1.0]]))) == 0.0)


def test_swish_reflection_identity_and_gating(oracle):
    """Swish(g) - Swish(-g) = g: checked on the oracle's outputs with up = 2^k (a power of two only shifts the
    exponent, so the only error is the one rounding of each term, below 2^-8 relative)."""
    rng = np.random.default_rng(5)
    g = (rng.standard_normal((64, 256)) * 3.0).astype(np.float32)
    gb = bits_of(g)
    gv = vals_of(gb)
    ones = bits_of(np.ones_like(g))
    pos = vals_of(oracle.swiglu(gb, ones))
    neg = vals_of(oracle.swiglu(bits_of(-vals_of(gb).astype(np.float32)), ones))
    assert np.all(np.abs((pos - neg) - gv) <= 2.0 ** -8 * (np.abs(pos) + np.abs(neg)) + 1e-30)
    # the second operand multiplies: with up = 4 the result is exactly 4 x the result with up = 1 (same rounding)
    four = bits_of(np.full_like(g, 4.0))
    assert np.array_equal(vals_of(oracle.swiglu(gb, four)), 4.0 * pos)
    # sign of up flips the sign
    assert np.array_equal(vals_of(oracle.swiglu(gb, bits_of(np.full_like(g, -1.0)))), -pos)


def test_rounding_is_one_round_to_nearest_even_against_brute_force(oracle):
    rng = np.random.default_rng(6)
    g = bits_of(rng.standard_normal((8, 64)) * 4.0)
    u = bits_of(rng.standard_normal((8, 64)) * 2.0)
    h = oracle.swiglu(g, u)
    gv, uv = vals_of(g), vals_of(u)
    exact = gv / (1.0 + np.exp(-gv)) * uv
    for t in range(8):
        for i in range(0, 64, 3):
            assert int(h[t, i]) == nearest_bf16_brute_force(float(exact[t, i])), (t, i)
    # magnitudes in the subnormal range of bf16 and below it
    tiny = bits_of([[2.0 ** -60, 2.0 ** -70, 2.0 ** -100]])
    tu = bits_of([[2.0 ** -64, 2.0 ** -64, 2.0 ** -60]])
    ht = oracle.swiglu(tiny, tu)
    tv, tuv = vals_of(tiny), vals_of(tu)
    ex = tv / (1.0 + np.exp(-tv)) * tuv
    for i in range(3):
        assert int(ht[0, i]) == nearest_bf16_brute_force(float(ex[0, i]))


def test_exact_ties_round_to_even(oracle):
    """Swish(g) * u lands exactly on a bf16 tie only by construction: g large enough that Swish(g) = g in fp64
    (g >= 40), u chosen so that g * u is halfway between two bf16 values."""
    g = bits_of([[64.0, 64.0, 64.0, 64.0]])
    # 64 * u with u = 1 + k/128: exact bf16; products with a 9-bit significand need two 8-bit factors:
    # g = 1.5 * 64 = 96, u = 1.0078125 (1 + 2^-7): 96.75 = 1.51171875 * 64 -> significand 1.1000001 1 -> a tie at 9 bits
    g = bits_of([[96.0, 96.0]])
    u = bits_of([[1.0 + 2.0 ** -7, 1.0 + 3.0 * 2.0 ** -7]])
    exact = vals_of(g) * vals_of(u)                       # 96.75 and 98.25
    h = oracle.swiglu(g, u)
    for i in range(2):
        v = float(exact[0, i])
        lo = nearest_bf16_brute_force(v - 1e-9)
        hi = nearest_bf16_brute_force(v + 1e-9)
        assert lo != hi                                    # a genuine tie
        assert int(h[0, i]) in (lo, hi) and int(h[0, i]) % 2 == 0


def test_chain_equals_two_steps(oracle):
    """The fused operation is the rotate+quantize path applied to the stored h."""
    rng = np.random.default_rng(7)
    g = bits_of(rng.standard_normal((16, 1024)) * 2.0)
    u = bits_of(rng.standard_normal((16, 1024)))
    h = oracle.swiglu(g, u)
    assert h.dtype == np.uint16 and h.shape == g.shape
    a = oracle.rotate_quantize(h, None, 32, 1, 32)
    b = oracle.rotate_quantize(oracle.swiglu(g, u), None, 32, 1, 32)
    assert np.array_equal(a["codes"], b["codes"]) and np.array_equal(a["scales"], b["scales"])
