"""Pins for the oracle's MCF primitives: the invariants the paper states, evaluated exactly.

Theorem 4.1 (Fast2Sum: a+b = x+y, |y| <= ulp(x)/2), Appendix C (TwoSum gives
the same expansion without ordering; TwoProdFMA gives the same result as the
Split-based TwoProd), Def. 2.1 (non-overlapping components), Algorithm 1
(Grow), Algorithms Scaling and Mul, and brute force against exact rationals.
"""
import random
from fractions import Fraction

import numpy as np

import oracle
from conftest import bf16_window, bits_to_f64, ulp_f64
import exact_rational as R


def _pairs(w):
    return np.repeat(w, w.size), np.tile(w, w.size)


def test_fast_two_sum_invariant_exhaustive_window():
    # Theorem 4.1 on every ordered pair |a| >= |b| of a 17-binade window, both signs, plus zeros
    w = bf16_window(-8, 8, with_zero=True)
    a, b = _pairs(w)
    keep = np.abs(bits_to_f64(a)) >= np.abs(bits_to_f64(b))
    a, b = a[keep], b[keep]
    x, y = oracle.fast_two_sum(a, b)
    fa, fb, fx, fy = map(bits_to_f64, (a, b, x, y))
    assert np.array_equal(fa + fb, fx + fy)                  # both sides exact in double on this window
    assert np.all(np.abs(fy) <= ulp_f64(x) / 2)              # the bound is attained at ties, so <=
    assert np.any(np.abs(fy) == ulp_f64(x) / 2)
    # x is the rounded sum itself
    assert np.array_equal(x, oracle.binary_op(oracle.OP_ADD, a, b))


def test_fast_two_sum_needs_the_ordering_and_two_sum_does_not():
    w = bf16_window(-8, 8, with_zero=True)
    a, b = _pairs(w)
    x, y = oracle.two_sum(a, b)
    fa, fb, fx, fy = map(bits_to_f64, (a, b, x, y))
    assert np.array_equal(fa + fb, fx + fy)                  # exact for every pair, any order
    assert np.all(np.abs(fy) <= ulp_f64(x) / 2)
    # where |a| >= |b| the two algorithms produce the same expansion (values; zero signs may differ)
    keep = np.abs(fa) >= np.abs(fb)
    fx2, fy2 = oracle.fast_two_sum(a[keep], b[keep])
    assert np.array_equal(bits_to_f64(fx2), fx[keep]) and np.array_equal(bits_to_f64(fy2), fy[keep])
    # and Fast2Sum applied with the wrong order is not error-free in general
    fx3, fy3 = oracle.fast_two_sum(a[~keep], b[~keep])
    broken = bits_to_f64(fx3) + bits_to_f64(fy3) != fa[~keep] + fb[~keep]
    assert broken.any()


def test_two_prod_is_error_free_and_matches_dekker():
    # every significand pair, both signs, a few exponent combinations that stay clear of underflow
    w = np.concatenate([bf16_window(e, e) for e in (-20, -1, 0, 1, 20)])
    a, b = _pairs(w)
    x, e = oracle.two_prod(a, b)
    fa, fb, fx, fe = map(bits_to_f64, (a, b, x, e))
    assert np.array_equal(fa * fb, fx + fe)                  # 16-bit product: exact in double
    assert np.all(np.abs(fe) <= ulp_f64(x) / 2)
    xd, ed = oracle.two_prod_dekker(a, b)
    assert np.array_equal(x, xd)
    assert np.array_equal(fe, bits_to_f64(ed))               # Appendix C: "the same results"


def test_split_halves():
    w = bf16_window(-10, 10)
    hi, lo = oracle.split(w)
    fw, fh, fl = map(bits_to_f64, (w, hi, lo))
    assert np.array_equal(fh + fl, fw)
    # each half fits in 4 significant bits: scaled by its own leading power of two it is a multiple of 1/8
    for part in (fh, fl):
        nz = part != 0
        mant, _ = np.frexp(part[nz])
        assert np.all(mant * 16 == np.round(mant * 16))


def test_grow_invariants():
    rng = np.random.default_rng(21)
    w = bf16_window(-6, 6)
    x = rng.choice(w, 3_000_000)
    a = rng.choice(bf16_window(-14, -6), x.size)            # |a| < |x|
    # y: a valid low component, |y| <= ulp(x)/2
    y = oracle.round_to_bf16(bits_to_f64(x) * 0 + rng.uniform(-0.5, 0.5, x.size) * ulp_f64(x))
    u, v = oracle.grow(x, y, a)
    fx, fy, fa, fu, fv = map(bits_to_f64, (x, y, a, u, v))
    assert np.all(np.abs(fv) <= ulp_f64(u) / 2)             # Def. 2.1: non-overlapping output
    # exact when the low component starts at zero
    u0, v0 = oracle.grow(x, np.zeros_like(x), a)
    assert np.array_equal(bits_to_f64(u0) + bits_to_f64(v0), fx + fa)
    # otherwise the only rounding is the one addition y (+) v of Algorithm 1 line 3
    s1, e1 = oracle.fast_two_sum(x, a)
    t = oracle.binary_op(oracle.OP_ADD, y, e1)
    err = np.abs((fu + fv) - (fx + fy + fa))
    assert np.all(err <= ulp_f64(t) / 2)
    assert np.array_equal(fu + fv, bits_to_f64(s1) + bits_to_f64(t))


def test_grow_keeps_what_plain_bf16_loses():
    # Section 3.1 remark + Section 4: 1.0 (+) 2^-10 is lost in bfloat16; Grow keeps it in the second component
    one = np.array([0x3F80], np.uint16)
    inc = np.array([oracle.round_to_bf16(2.0 ** -10)], np.uint16)
    plain = one.copy()
    hi, lo = one.copy(), np.zeros(1, np.uint16)
    seen = []
    for _ in range(8):
        plain = oracle.binary_op(oracle.OP_ADD, plain, inc)
        hi, lo = oracle.grow(hi, lo, inc)
        seen.append((int(hi[0]), float(bits_to_f64(lo)[0])))
    assert int(plain[0]) == 0x3F80                           # eight lost additions
    total = [bits_to_f64(np.array([h], np.uint16))[0] + l for h, l in seen]
    assert total == [1.0 + k * 2.0 ** -10 for k in range(1, 9)]     # the expansion holds the exact sum
    assert seen[3] == (0x3F80, 2.0 ** -8)                    # half an ulp is still carried below (tie kept)
    assert seen[4][0] == 0x3F81 and seen[4][1] < 0           # then it rolls into the first component
    assert seen[7] == (0x3F81, 0.0)


def test_renormalize_is_fast_two_sum():
    w = bf16_window(-5, 5)
    rng = np.random.default_rng(2)
    hi = rng.choice(w, 200_000)
    lo = rng.choice(bf16_window(-12, -5), hi.size)
    rh, rl = oracle.renormalize(hi, lo)
    assert np.array_equal(bits_to_f64(rh) + bits_to_f64(rl), bits_to_f64(hi) + bits_to_f64(lo))
    assert np.all(np.abs(bits_to_f64(rl)) <= ulp_f64(rh) / 2)
    fh, fl = oracle.fast_two_sum(hi, lo)
    assert np.array_equal(rh, fh) and np.array_equal(rl, fl)


def _valid_expansions(rng, n, e_lo, e_hi):
    hi = rng.choice(bf16_window(e_lo, e_hi), n)
    lo = oracle.round_to_bf16(rng.uniform(-0.5, 0.5, n) * ulp_f64(hi))
    return hi, lo


def test_mul_and_scaling_accuracy():
    rng = np.random.default_rng(33)
    n = 1_000_000
    a1, a2 = _valid_expansions(rng, n, -3, 3)
    b1, b2 = _valid_expansions(rng, n, -3, 3)
    x, e = oracle.mul(a1, a2, b1, b2)
    exact = (bits_to_f64(a1) + bits_to_f64(a2)) * (bits_to_f64(b1) + bits_to_f64(b2))
    got = bits_to_f64(x) + bits_to_f64(e)
    # a length-2 bfloat16 expansion carries ~16 bits; the dropped a2*b2 term and three roundings of
    # second-order terms leave a relative error of a few 2^-16 (worst seen: 4.2)
    assert np.all(np.abs(got - exact) <= 6 * 2.0 ** -16 * np.abs(exact))
    assert np.all(np.abs(bits_to_f64(e)) <= ulp_f64(x) / 2)
    # with zero low parts Mul reduces to the error-free product
    z = np.zeros(n, np.uint16)
    x0, e0 = oracle.mul(a1, z, b1, z)
    assert np.array_equal(bits_to_f64(x0) + bits_to_f64(e0), bits_to_f64(a1) * bits_to_f64(b1))
    # Scaling
    v = rng.choice(bf16_window(-3, 3), n)
    xs, es = oracle.scaling(v, a1, a2)
    exact = bits_to_f64(v) * (bits_to_f64(a1) + bits_to_f64(a2))
    assert np.all(np.abs(bits_to_f64(xs) + bits_to_f64(es) - exact) <= 3 * 2.0 ** -16 * np.abs(exact))
    xs0, es0 = oracle.scaling(v, a1, z)
    assert np.array_equal(bits_to_f64(xs0) + bits_to_f64(es0), bits_to_f64(v) * bits_to_f64(a1))


def test_beta2_decay_needs_the_expansion():
    # Section 4.2: beta2 = 0.999 rounds to 1.0, so v (*) beta2 does not decay in plain bfloat16,
    # while Mul with the expansion (1, -0.001) decays by the right factor
    v = bf16_window(-30, -10, signs=(0,))
    z = np.zeros_like(v)
    b2h = np.full_like(v, 0x3F80)
    b2l = np.full_like(v, oracle.round_to_bf16(0.999 - 1.0))
    plain = oracle.binary_op(oracle.OP_MUL, b2h, v)
    assert np.array_equal(plain, v)
    x, e = oracle.mul(b2h, b2l, v, z)
    got = bits_to_f64(x) + bits_to_f64(e)
    want = 0.999 * bits_to_f64(v)
    assert np.all(np.abs(got - want) <= 2.0 ** -15 * want)
    assert np.all(got < bits_to_f64(v))


def test_primitives_against_exact_rationals_on_random_tiny_inputs():
    rnd = random.Random(17)
    pool = [int(b) for b in bf16_window(-12, 4, with_zero=True)]
    a = [rnd.choice(pool) for _ in range(1500)]
    b = [rnd.choice(pool) for _ in range(1500)]
    c = [rnd.choice(pool) for _ in range(1500)]
    d = [rnd.choice(pool) for _ in range(1500)]
    A, B, C, D = (np.array(t, np.uint16) for t in (a, b, c, d))
    f2 = oracle.fast_two_sum(A, B)
    tp = oracle.two_prod(A, B)
    gr = oracle.grow(A, B, C)
    ml = oracle.mul(A, B, C, D)
    sc = oracle.scaling(A, B, C)

    def same(got_bits, want_bits):
        # identical bits, except that the rational model does not track the sign of an exact zero sum
        return got_bits == want_bits or ((got_bits | want_bits) & 0x7FFF) == 0

    for i in range(len(a)):
        assert all(map(same, (int(f2[0][i]), int(f2[1][i])), R.fast_two_sum(a[i], b[i])))
        assert all(map(same, (int(tp[0][i]), int(tp[1][i])), R.two_prod(a[i], b[i])))
        assert all(map(same, (int(gr[0][i]), int(gr[1][i])), R.grow(a[i], b[i], c[i])))
        assert all(map(same, (int(ml[0][i]), int(ml[1][i])), R.mcf_mul(a[i], b[i], c[i], d[i])))
        assert all(map(same, (int(sc[0][i]), int(sc[1][i])), R.scaling(a[i], b[i], c[i])))


def test_zero_signs_follow_ieee():
    P0, N0 = np.array([0x0000], np.uint16), np.array([0x8000], np.uint16)
    x = np.array([0x3F80], np.uint16)
    assert int(oracle.binary_op(oracle.OP_SUB, x, x)[0]) == 0x0000           # x - x = +0
    assert int(oracle.binary_op(oracle.OP_ADD, P0, N0)[0]) == 0x0000
    assert int(oracle.binary_op(oracle.OP_ADD, N0, N0)[0]) == 0x8000
    assert int(oracle.binary_op(oracle.OP_MUL, N0, x)[0]) == 0x8000
    assert int(oracle.binary_op(oracle.OP_DIV, N0, x)[0]) == 0x8000
    nan = int(oracle.binary_op(oracle.OP_DIV, P0, P0)[0])
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x7F)
    assert int(oracle.binary_op(oracle.OP_DIV, x, P0)[0]) == 0x7F80
