"""Pins for the oracle's bfloat16 format model and its single rounded operations.

What fixes the expected values: the paper's format facts (Appendix A table,
Section 3.1 remark, Section 2.2), the definition of round-to-nearest-even
checked through exact neighbour distances, torch's own float32->bfloat16
conversion (an independent library routine), and exact rational arithmetic.
"""
import random
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from conftest import bf16_window, bits_to_f64, neighbours, ulp_f64
import exact_rational as R


def test_format_facts_from_the_paper():
    # Appendix A table: 8 exponent bits, 7 mantissa bits, ulp(1) = 2^-7
    assert oracle.widen(0x3F80) == 1.0
    assert oracle.widen(0x3F81) - oracle.widen(0x3F80) == 2.0 ** -7
    # Section 3.1: 0.1 is not representable and rounds to 0.1001
    assert oracle.round_to_bf16(0.1) == 0x3DCD
    assert oracle.widen(0x3DCD) == 0.10009765625
    assert f"{oracle.widen(0x3DCD):.4f}" == "0.1001"
    # Section 2.2: 0.999 rounds to 1.0
    assert oracle.round_to_bf16(0.999) == 0x3F80
    # Section 3.1 remark: ulp(200) = 1 and 200 (+) 0.1 = 200
    b200 = oracle.round_to_bf16(200.0)
    assert oracle.widen(b200) == 200.0
    assert oracle.widen(b200 + 1) - 200.0 == 1.0
    got = oracle.binary_op(oracle.OP_ADD, np.array([b200], np.uint16), np.array([0x3DCD], np.uint16))
    assert int(got[0]) == b200
    # Appendix D: 1 (-) 1.2e-5 is lost; the least effective decrement is ulp(1)/2 = 2^-8
    one = np.array([0x3F80], np.uint16)
    tiny = np.array([oracle.round_to_bf16(1.2e-5)], np.uint16)
    assert int(oracle.binary_op(oracle.OP_SUB, one, tiny)[0]) == 0x3F80
    # below one the spacing is 2^-8, so a decrement of 2^-9 is a tie that goes back to the even 1.0 ...
    tie = np.array([oracle.round_to_bf16(2.0 ** -9)], np.uint16)
    assert int(oracle.binary_op(oracle.OP_SUB, one, tie)[0]) == 0x3F80
    # ... and above one a step of ulp(1)/2 = 2^-8 ~ 0.0039 is the tie that is lost too
    assert abs(2.0 ** -7 / 2 - 0.0039) < 1e-4
    half_ulp = np.array([oracle.round_to_bf16(2.0 ** -8)], np.uint16)
    assert int(oracle.binary_op(oracle.OP_ADD, one, half_ulp)[0]) == 0x3F80
    just_more = np.array([oracle.round_to_bf16(2.0 ** -8) + 1], np.uint16)
    assert int(oracle.binary_op(oracle.OP_ADD, one, just_more)[0]) == 0x3F81


def test_every_finite_pattern_round_trips():
    bits = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    finite = ((bits >> 7) & 0xFF) != 0xFF
    vals = oracle.widen(bits[finite])
    assert np.array_equal(oracle.round_to_bf16(vals), bits[finite])
    assert np.array_equal(vals, bits_to_f64(bits[finite]))
    # infinities and NaN class
    assert oracle.round_to_bf16(float("inf")) == 0x7F80
    assert oracle.round_to_bf16(float("-inf")) == 0xFF80
    nan = oracle.round_to_bf16(float("nan"))
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x7F) != 0
    assert oracle.round_to_bf16(-0.0) == 0x8000 and oracle.round_to_bf16(0.0) == 0x0000


def test_ties_go_to_even_and_overflow_goes_to_infinity():
    # midpoints between consecutive bfloat16 values across normal, subnormal and top binades
    lows = np.concatenate([
        bf16_window(-126, -120, signs=(0,)), bf16_window(-3, 3, signs=(0, 1)),
        bf16_window(120, 127, signs=(0,)), np.arange(0, 128, dtype=np.uint16)])
    lows = lows[(lows & 0x7FFF) < 0x7F7F]
    up, _ = neighbours(lows)
    mid = (bits_to_f64(lows) + bits_to_f64(up)) / 2.0          # exact in double
    got = oracle.round_to_bf16(mid)
    even = np.where((lows & 1) == 0, lows, up)
    assert np.array_equal(got, even)
    # nudging the midpoint by one double ulp decides the direction
    assert np.array_equal(oracle.round_to_bf16(np.nextafter(mid, np.sign(mid) * np.inf)), up)
    assert np.array_equal(oracle.round_to_bf16(np.nextafter(mid, 0.0)), lows)
    # overflow threshold: max finite + half an ulp rounds to infinity (tie to even = 2^128)
    top = bits_to_f64(np.array([0x7F7F], np.uint16))[0]
    assert oracle.round_to_bf16(top + 2.0 ** 119) == 0x7F80
    assert oracle.round_to_bf16(np.nextafter(top + 2.0 ** 119, 0.0)) == 0x7F7F
    # smallest subnormal: half of it ties to zero (even), just above goes up
    assert oracle.round_to_bf16(2.0 ** -134) == 0x0000
    assert oracle.round_to_bf16(np.nextafter(2.0 ** -134, 1.0)) == 0x0001
    assert oracle.round_to_bf16(-(2.0 ** -134) * 3) == 0x8002      # 1.5 quanta: tie to even = 2


def test_rounder_agrees_with_torch_conversion():
    g = torch.Generator().manual_seed(11)
    raw = torch.randint(-2 ** 31, 2 ** 31 - 1, (1 << 22,), dtype=torch.int64, generator=g).to(torch.int32)
    f32 = raw.view(torch.float32)
    f32 = f32[torch.isfinite(f32)]
    want = f32.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.round_to_bf16(f32.double().numpy())
    assert np.array_equal(got, want)
    # float32 subnormals and the last binade, densely
    edge = torch.cat([torch.arange(0, 1 << 20, dtype=torch.int32),
                      torch.arange(0x7F000000, 0x7F7FFFFF, 37, dtype=torch.int64).to(torch.int32)]).view(torch.float32)
    want = edge.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.round_to_bf16(edge.double().numpy()), want)


def test_rounder_agrees_with_exact_rationals():
    rnd = random.Random(5)
    for _ in range(4000):
        e = rnd.randint(-140, 130)
        x = rnd.uniform(1.0, 2.0) * 2.0 ** e * rnd.choice((-1, 1))
        assert oracle.round_to_bf16(x) == R.rn(Fraction(x))


def _assert_nearest_even(result, dist_of, finite_mask=None):
    """result is a nearest bfloat16 (ties to even) given an exact distance function of a candidate."""
    up, down = neighbours(result)
    d0, du, dd = dist_of(result), dist_of(up), dist_of(down)
    ok = (d0 <= du) & (d0 <= dd)
    tie = (d0 == du) | (d0 == dd)
    nonzero = (result & 0x7FFF) != 0
    ok &= ~(tie & nonzero) | ((result & 1) == 0)
    if finite_mask is not None:
        ok |= ~finite_mask
    assert ok.all(), f"{(~ok).sum()} results are not the nearest-even value"


@pytest.mark.parametrize("op", ["add", "sub"])
def test_add_sub_exhaustive_window(op):
    # all pairs with exponents in [-8, 8], both signs: the exact sum fits a double
    w = bf16_window(-8, 8)
    a = np.repeat(w, w.size)
    b = np.tile(w, w.size)
    code = oracle.OP_ADD if op == "add" else oracle.OP_SUB
    r = oracle.binary_op(code, a, b)
    exact = bits_to_f64(a) + (bits_to_f64(b) if op == "add" else -bits_to_f64(b))
    _assert_nearest_even(r, lambda c: np.abs(exact - bits_to_f64(c)))
    # exact zero results are +0 under round-to-nearest
    assert np.all(r[exact == 0.0] == 0)


def test_mul_exhaustive_significands_and_exponent_edges():
    # all 128 x 128 significands, signs, exponents chosen to hit normal, subnormal and overflow results
    w = np.concatenate([bf16_window(e, e) for e in (-126, -70, -64, -1, 0, 1, 63, 64, 127)])
    a = np.repeat(w, w.size)
    b = np.tile(w, w.size)
    r = oracle.binary_op(oracle.OP_MUL, a, b)
    exact = bits_to_f64(a) * bits_to_f64(b)                     # 16-bit product: exact in double
    finite = (r & 0x7F80) != 0x7F80
    _assert_nearest_even(r, lambda c: np.abs(exact - bits_to_f64(c)), finite)
    top = bits_to_f64(np.array([0x7F7F], np.uint16))[0]
    assert np.all(np.abs(exact[~finite]) >= top + 2.0 ** 119)   # infinity only past the overflow threshold
    assert np.all(np.abs(exact[finite]) < top + 2.0 ** 119)


def test_div_exhaustive_significands():
    # the quotient is decided exactly by cross-multiplication: |a - c*b| for candidate c
    w = np.concatenate([bf16_window(e, e) for e in (-60, -1, 0, 1, 60)])
    a = np.repeat(w, w.size)
    b = np.tile(w, w.size)
    r = oracle.binary_op(oracle.OP_DIV, a, b)
    fa, fb = bits_to_f64(a), bits_to_f64(b)
    _assert_nearest_even(r, lambda c: np.abs(fa - bits_to_f64(c) * fb))


def test_div_subnormal_results_against_rationals():
    rnd = random.Random(7)
    for _ in range(3000):
        a = rnd.randrange(0x0001, 0x0800)           # tiny numerators incl. subnormals
        b = rnd.randrange(0x3F80, 0x4700)
        a |= rnd.choice((0, 0x8000))
        got = int(oracle.binary_op(oracle.OP_DIV, np.array([a], np.uint16), np.array([b], np.uint16))[0])
        assert got == R.div(a, b)


def test_sqrt_all_positive_finite_values():
    bits = np.arange(1, 0x7F80, dtype=np.uint16)
    r = oracle.binary_op(oracle.OP_SQRT, bits)
    x = bits_to_f64(bits)
    up, down = neighbours(r)
    c, cu, cd = bits_to_f64(r), bits_to_f64(up), bits_to_f64(down)
    hi_mid, lo_mid = (c + cu) / 2, (c + cd) / 2            # 9-bit midpoints, squares exact in double
    assert np.all(lo_mid * lo_mid <= x) and np.all(x <= hi_mid * hi_mid)
    # a square root is never a tie except trivially; check strictness where it is not exact
    inexact = c * c != x
    assert np.all((lo_mid * lo_mid < x)[inexact]) and np.all((x < hi_mid * hi_mid)[inexact])
    assert int(oracle.binary_op(oracle.OP_SQRT, np.array([0x8000], np.uint16))[0]) == 0x8000
    assert int(oracle.binary_op(oracle.OP_SQRT, np.array([0x0000], np.uint16))[0]) == 0x0000
    for b in random.Random(3).sample(range(1, 0x7F80), 300):
        assert int(r[b - 1]) == R.sqrt(b)


def test_fma_single_rounding_window():
    # a*b + c with exponents in a window: exact in double, one rounding
    w = bf16_window(-3, 3)
    rng = np.random.default_rng(9)
    a, b, c = (rng.choice(w, 2_000_000) for _ in range(3))
    r = oracle.binary_op(oracle.OP_FMA, a, b, c)
    exact = bits_to_f64(a) * bits_to_f64(b) + bits_to_f64(c)
    _assert_nearest_even(r, lambda k: np.abs(exact - bits_to_f64(k)))
    # a case where fused and unfused differ: the product's low bits survive only when fused
    a1 = np.array([0x3F81], np.uint16)                     # 1 + 2^-7
    prod = oracle.binary_op(oracle.OP_MUL, a1, a1)         # (1+2^-7)^2 = 1 + 2^-6 + 2^-14 -> 1 + 2^-6
    neg = prod ^ np.uint16(0x8000)
    fused = oracle.binary_op(oracle.OP_FMA, a1, a1, neg)
    assert bits_to_f64(fused)[0] == 2.0 ** -14
    assert int(oracle.binary_op(oracle.OP_ADD, prod, neg)[0]) == 0


def test_fma_is_one_rounding_even_when_the_addend_is_far_below_the_product():
    # a*b lands exactly on a midpoint of two bfloat16 values; an addend 60 binades below decides the direction.
    # Rounding the sum to double first would lose the addend and fall back to ties-to-even.
    a = np.array([0x3F81], np.uint16)                      # 1 + 2^-7
    b = np.array([0x3FC0], np.uint16)                      # 1.5 -> product 1.5 + 1.5*2^-7 = 1.51171875 (midpoint)
    lo, hi = 0x3FC1, 0x3FC2                                # neighbours 1.5078125 and 1.515625
    assert bits_to_f64(a)[0] * bits_to_f64(b)[0] == (bits_to_f64(np.array([lo], np.uint16))[0] +
                                                     bits_to_f64(np.array([hi], np.uint16))[0]) / 2
    tiny = oracle.round_to_bf16(2.0 ** -70)
    up = oracle.binary_op(oracle.OP_FMA, a, b, np.array([tiny], np.uint16))
    down = oracle.binary_op(oracle.OP_FMA, a, b, np.array([tiny | 0x8000], np.uint16))
    tie = oracle.binary_op(oracle.OP_FMA, a, b, np.array([0], np.uint16))
    assert (int(up[0]), int(down[0]), int(tie[0])) == (hi, lo, hi)           # tie itself goes to even (0x3FC2)
    # brute force against exact rationals over wide exponent ranges, subnormals included
    rnd = random.Random(23)
    pool = [int(x) for x in np.concatenate([bf16_window(-126, 100), np.arange(1, 128, dtype=np.uint16)])]
    trip = [(rnd.choice(pool), rnd.choice(pool), rnd.choice(pool)) for _ in range(20000)]
    trip = [(x, y, z) for x, y, z in trip if abs(R.decode(x) * R.decode(y)) < 2 ** 120]
    A, B, C = (np.array(t, np.uint16) for t in zip(*trip))
    got = oracle.binary_op(oracle.OP_FMA, A, B, C)
    for (x, y, z), g in zip(trip, got):
        want = R.fma(x, y, z)
        assert int(g) == want or ((int(g) | want) & 0x7FFF) == 0, (hex(x), hex(y), hex(z), hex(int(g)), hex(want))


def test_ulp_helper_matches_definition():
    # Def. 3.1 with the paper's examples: ulp(1) = 2^-7, ulp(200) = 1, subnormals share 2^-133
    assert ulp_f64(np.array([0x3F80], np.uint16))[0] == 2.0 ** -7
    assert ulp_f64(np.array([oracle.round_to_bf16(200.0)], np.uint16))[0] == 1.0
    assert ulp_f64(np.array([0x0001], np.uint16))[0] == 2.0 ** -133
    w = bf16_window(-20, 20, signs=(0,))
    up, _ = neighbours(w)
    assert np.array_equal(bits_to_f64(up) - bits_to_f64(w), ulp_f64(w))
