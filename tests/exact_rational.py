"""bfloat16 arithmetic on exact rationals (``fractions.Fraction``), for brute force on tiny inputs.

A second, slow model of "one operation, one rounding to nearest-even" that
uses only integer/rational arithmetic: no floating point of the host, no code
of the oracle, no code of the CUDA library.  The tests run tiny cases through
this model and through the oracle and demand identical bits.
"""
from __future__ import annotations

from fractions import Fraction

TWO = Fraction(2)


def decode(bits: int) -> Fraction:
    """Value of a finite bfloat16 bit pattern (1 sign, 8 exponent, 7 mantissa bits)."""
    sign = -1 if bits & 0x8000 else 1
    field = (bits >> 7) & 0xFF
    man = bits & 0x7F
    assert field != 0xFF, "finite values only"
    if field == 0:
        return sign * Fraction(man, 2 ** 133)
    return sign * Fraction(128 + man, 128) * TWO ** (field - 127)


def rn(x: Fraction, negative_zero: bool = False) -> int:
    """Nearest bfloat16 to the rational x, ties to even, gradual underflow, overflow to infinity."""
    if x == 0:
        return 0x8000 if negative_zero else 0
    sign = 0x8000 if x < 0 else 0
    ax = -x if x < 0 else x
    e = ax.numerator.bit_length() - ax.denominator.bit_length()
    if TWO ** e > ax:
        e -= 1
    assert TWO ** e <= ax < TWO ** (e + 1)
    e = max(e, -126)
    scaled = ax / TWO ** (e - 7)
    whole = scaled.numerator // scaled.denominator
    rest = scaled - whole
    if rest > Fraction(1, 2) or (rest == Fraction(1, 2) and whole % 2 == 1):
        whole += 1
    if whole == 256:
        whole, e = 128, e + 1
    if whole < 128:
        return sign | whole
    if e + 127 >= 255:
        return sign | 0x7F80
    return sign | ((e + 127) << 7) | (whole - 128)


def add(a: int, b: int) -> int:
    return rn(decode(a) + decode(b), negative_zero=bool(a & b & 0x8000) and decode(a) == 0 == decode(b))


def sub(a: int, b: int) -> int:
    return add(a, b ^ 0x8000)


def mul(a: int, b: int) -> int:
    p = decode(a) * decode(b)
    return rn(p, negative_zero=bool((a ^ b) & 0x8000))


def fma(a: int, b: int, c: int) -> int:
    return rn(decode(a) * decode(b) + decode(c))


def div(a: int, b: int) -> int:
    return rn(decode(a) / decode(b), negative_zero=bool((a ^ b) & 0x8000))


def sqrt(a: int) -> int:
    """Correctly rounded square root of a non-negative finite bfloat16, decided with exact squares."""
    x = decode(a)
    assert x >= 0
    if x == 0:
        return a
    lo, hi = 0, 0x7F7F          # positive bit patterns are ordered like their values
    while lo < hi:              # largest pattern c with c*c <= x
        mid = (lo + hi + 1) // 2
        if decode(mid) ** 2 <= x:
            lo = mid
        else:
            hi = mid - 1
    below, above = lo, lo + 1
    if decode(below) ** 2 == x or above > 0x7F7F:
        return below
    half = (decode(below) + decode(above)) / 2
    if x > half * half:
        return above
    if x < half * half:
        return below
    return below if below % 2 == 0 else above


def fast_two_sum(a, b):
    x = add(a, b)
    return x, sub(b, sub(x, a))


def two_prod(a, b):
    x = mul(a, b)
    return x, fma(a, b, x ^ 0x8000)


def grow(x, y, a):
    u, v = fast_two_sum(x, a)
    return fast_two_sum(u, add(y, v))


def mcf_mul(a1, a2, b1, b2):
    x, e = two_prod(a1, b1)
    e = add(e, add(mul(a1, b2), mul(a2, b1)))
    return fast_two_sum(x, e)


def scaling(v, a1, a2):
    x, e = two_prod(a1, v)
    e = add(mul(a2, v), e)
    return fast_two_sum(x, e)


def value_unchanged(th_old, dth_old, th_new, dth_new) -> bool:
    """Is the effective update of Eq. 2, (theta' + dtheta') - (theta + dtheta), exactly zero?"""
    return decode(th_new) + decode(dth_new) == decode(th_old) + decode(dth_old)


def components_unchanged(th_old, dth_old, th_new, dth_new) -> bool:
    """The other candidate reading of "not updated": every stored component kept its value."""
    return decode(th_new) == decode(th_old) and decode(dth_new) == decode(dth_old)


def is_normalised(hi, lo) -> bool:
    """|lo| <= ulp(hi)/2 (Def. 3.1 with 7 stored bits), the invariant Grow maintains."""
    field = (hi >> 7) & 0xFF
    ulp = TWO ** (max(field - 127, -126) - 7)
    return abs(decode(lo)) <= ulp / 2


def two_sum(a, b):
    x = add(a, b)
    bv = sub(x, a)
    av = sub(x, bv)
    return x, add(sub(a, av), sub(b, bv))


def grow_two_sum(x, y, a):
    u, v = two_sum(x, a)
    return two_sum(u, add(y, v))


def adamw_element_variant(th, dth, m, v, dv, g, sc, strategy, twosum_grow=False, split_decay=False):
    """Step variants: strategy 3 = BF16-Kahan (dth holds c); TwoSum-based Grow; decay by its own addition."""
    m = add(mul(sc["b1"], m), mul(sc["c1"], g))
    tv = mul(sc["c2"], mul(g, g))
    if strategy == 2:
        p, e = mcf_mul(sc["b2h"], sc["b2l"], v, dv)
        v, dv = grow(p, e, tv)
    else:
        v = add(mul(sc["b2"], v), tv)
    r = div(div(m, sc["bc1"]), add(sqrt(div(v, sc["bc2"])), sc["eps"]))
    w = mul(sc["lam"], th)
    nega = sc["a"] ^ 0x8000
    decay = mul(nega, w)
    delta = mul(nega, r) if split_decay else mul(nega, add(r, w))

    def apply(th, dth, upd):
        if strategy == 0:
            return add(th, upd), dth
        return grow_two_sum(th, dth, upd) if twosum_grow else grow(th, dth, upd)

    if strategy == 3:
        comp = add(delta, dth)
        new = add(th, comp)
        th, dth = new, sub(comp, sub(new, th))
    else:
        if split_decay:
            th, dth = apply(th, dth, decay)
        th, dth = apply(th, dth, delta)
    return th, dth, m, v, dv, delta


def adamw_element(th, dth, m, v, dv, g, sc, strategy, eps_inside=False):
    """Algorithm 2 lines 8-13 for one parameter; sc = dict of bfloat16 scalars. Returns new state and the update."""
    m = add(mul(sc["b1"], m), mul(sc["c1"], g))
    tv = mul(sc["c2"], mul(g, g))
    if strategy == 2:
        p, e = mcf_mul(sc["b2h"], sc["b2l"], v, dv)
        v, dv = grow(p, e, tv)
    else:
        v = add(mul(sc["b2"], v), tv)
    mhat = div(m, sc["bc1"])
    vhat = div(v, sc["bc2"])
    den = sqrt(add(vhat, sc["eps"])) if eps_inside else add(sqrt(vhat), sc["eps"])
    r = div(mhat, den)
    delta = mul(sc["a"] ^ 0x8000, add(r, mul(sc["lam"], th)))
    if strategy == 0:
        th = add(th, delta)
    else:
        th, dth = grow(th, dth, delta)
    return th, dth, m, v, dv, delta


def scalars(lr, beta1, beta2, eps, wd, t):
    """Scalar preparation with rationals: the decimal hypers are taken as exact decimals."""
    f = lambda s: Fraction(str(s))
    b2h = rn(f(beta2))
    return {
        "b1": rn(f(beta1)), "c1": rn(1 - f(beta1)), "b2": b2h, "c2": rn(1 - f(beta2)),
        "b2h": b2h, "b2l": rn(f(beta2) - decode(b2h)),
        "bc1": rn(1 - f(beta1) ** t), "bc2": rn(1 - f(beta2) ** t),
        "a": rn(f(lr)), "lam": rn(f(wd)), "eps": rn(f(eps)),
    }
