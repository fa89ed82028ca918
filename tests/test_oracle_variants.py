"""Pins for the oracle's comparator and variant steps: BF16-Kahan (Appendix B), Grow on TwoSum
(Appendix C), weight decay applied by its own addition (Appendix D).

Fixed by: the error-free-sum invariant the paper states for the Kahan variable ("essentially
Fast2Sum given |theta| >= |delta|"), its equivalence with Collage-light from a zero compensation,
exactness of TwoSum for any ordering, the lost-update worked case, and exact rationals.
"""
import numpy as np
import pytest

import oracle
from conftest import bf16_window, bits_to_f64, ulp_f64
import exact_rational as R
from paper_2405_03637_b200 import workloads as W

HYP = dict(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)


def _state(theta, strategy):
    th = np.array(theta, dtype=np.uint16)
    z = lambda: np.zeros_like(th)
    return dict(x_hi=th, x_lo=z() if strategy in (1, 2, 3) else None, m=z(), v_hi=z(), v_lo=z() if strategy == 2 else None)


def _step(st, g, t, strategy, hyp=HYP, **kw):
    return oracle.adamw_step(st["x_hi"], st["x_lo"], st["m"], st["v_hi"], st["v_lo"], g, step=t, strategy=strategy,
                             **hyp, **kw)


def test_kahan_compensation_is_the_rounding_error_of_the_addition():
    # Appendix D "Equivalence": with |theta| >= |update| the Kahan variable is the Fast2Sum error, so
    # theta' + c' == theta + (delta (+) c) exactly
    n = 1 << 15
    th0 = W.bits(W.stress_weights(n, 2))
    st = _state(th0.copy(), 3)
    for t in range(1, 41):
        g = W.bits(W.stress_grads(n, 2, t))
        before_th, before_c = st["x_hi"].copy(), st["x_lo"].copy()
        _, d = _step(st, g, t, 3, hyp=W.HYPERS_STRESS, want_delta=True)
        comp = oracle.binary_op(oracle.OP_ADD, d, before_c)
        lhs = bits_to_f64(st["x_hi"]) + bits_to_f64(st["x_lo"])
        rhs = bits_to_f64(before_th) + bits_to_f64(comp)
        assert np.array_equal(lhs, rhs)
        assert np.all(np.abs(bits_to_f64(st["x_lo"])) <= ulp_f64(st["x_hi"]) / 2)


def test_kahan_first_step_equals_collage_light_first_step():
    # from a zero compensation both are Fast2Sum(theta, delta): same theta, and c == dtheta wherever the
    # second Fast2Sum of Grow leaves theta alone (its input is at most half an ulp)
    n = 1 << 16
    th0 = W.bits(W.flat_weights(n, 0))
    g = W.bits(W.flat_grads(n, 0, 1))
    k, l = _state(th0.copy(), 3), _state(th0.copy(), 1)
    _step(k, g, 1, 3)
    _step(l, g, 1, 1)
    same_theta = k["x_hi"] == l["x_hi"]
    assert same_theta.mean() > 0.999
    assert np.array_equal(bits_to_f64(k["x_lo"])[same_theta], bits_to_f64(l["x_lo"])[same_theta])
    for key in ("m", "v_hi"):
        assert np.array_equal(k[key], l[key])


def test_kahan_keeps_what_plain_bf16_loses():
    # 200 (+) 0.1 is lost (Section 3.1 remark); with the compensation it arrives after a few steps
    th = np.full(64, oracle.round_to_bf16(200.0), np.uint16)
    hyp = dict(HYP, weight_decay=0.0, lr=0.1)
    plain, kahan = _state(th.copy(), 0), _state(th.copy(), 3)
    g = np.full(64, oracle.round_to_bf16(1e-3), np.uint16)
    shadow = bits_to_f64(th).copy()
    bound = np.zeros(64)
    for t in range(1, 31):
        sp, _ = _step(plain, g, t, 0, hyp=hyp)
        before_c = kahan["x_lo"].copy()
        sk, d = _step(kahan, g, t, 3, hyp=hyp, want_delta=True)
        shadow += bits_to_f64(d)
        bound += ulp_f64(oracle.binary_op(oracle.OP_ADD, d, before_c)) / 2
        assert sp["edq"] == 0.0 and sp["lost"] == 64
    assert np.all(plain["x_hi"] == th)
    held = bits_to_f64(kahan["x_hi"]) + bits_to_f64(kahan["x_lo"])
    assert np.all(np.abs(held - shadow) <= bound)
    assert np.all(bits_to_f64(kahan["x_hi"]) < 200.0)               # the updates did reach theta
    assert abs(float(bits_to_f64(kahan["x_hi"])[0]) - float(shadow[0])) <= 1.0


def test_kahan_edq_counts_theta_only():
    # Eq. 2 as printed: the effective update is F(theta (+) update) - theta; the compensation is not part of it
    n = 4096
    th0 = W.bits(W.flat_weights(n, 3))
    st = _state(th0.copy(), 3)
    g = W.bits(W.flat_grads(n, 3, 1))
    sums, d = _step(st, g, 1, 3, want_delta=True)
    eff = bits_to_f64(st["x_hi"]) - bits_to_f64(th0)
    dd = bits_to_f64(d)
    assert sums["dot"] == pytest.approx(float(np.sum(dd * eff)), rel=1e-12)
    assert sums["lost"] == int(np.sum((dd != 0) & (eff == 0)))
    # at t = 1 (c = 0) that is exactly plain bfloat16's EDQ
    plain = _state(th0.copy(), 0)
    sp, _ = _step(plain, g, 1, 0)
    assert sp == sums


def test_grow_on_two_sum_is_exact_for_any_ordering():
    rng = np.random.default_rng(4)
    n = 500_000
    th = rng.choice(bf16_window(-12, -4), n)                 # small parameters
    big = rng.choice(bf16_window(-6, 0), n)                  # updates larger than the parameter
    z = np.zeros(n, np.uint16)
    # through the step: lr and gradients chosen freely is awkward, so check the primitive through two steps
    # of pure Grow using the library of primitives: TwoSum twice
    u1, v1 = oracle.two_sum(th, big)
    t = oracle.binary_op(oracle.OP_ADD, z, v1)
    u2, v2 = oracle.two_sum(u1, t)
    assert np.array_equal(bits_to_f64(u2) + bits_to_f64(v2), bits_to_f64(th) + bits_to_f64(big))
    # Fast2Sum-based Grow is not exact there
    g1, g2 = oracle.grow(th, z, big)
    assert np.any(bits_to_f64(g1) + bits_to_f64(g2) != bits_to_f64(th) + bits_to_f64(big))


@pytest.mark.parametrize("strategy", [1, 2])
def test_two_sum_grow_flag_matches_default_where_theta_dominates_and_fixes_the_rest(strategy):
    n = 1 << 16
    th0 = W.bits(W.flat_weights(n, 0))
    g = W.bits(W.flat_grads(n, 0, 1))
    a, b = _state(th0.copy(), strategy), _state(th0.copy(), strategy)
    sa, d = _step(a, g, 1, strategy, want_delta=True)
    sb, _ = _step(b, g, 1, strategy, flags=oracle.FLAG_TWOSUM_GROW)
    dominated = np.abs(bits_to_f64(th0)) >= np.abs(bits_to_f64(d))
    va = bits_to_f64(a["x_hi"]) + bits_to_f64(a["x_lo"])
    vb = bits_to_f64(b["x_hi"]) + bits_to_f64(b["x_lo"])
    assert np.array_equal(va[dominated], vb[dominated])
    exact = bits_to_f64(th0) + bits_to_f64(d)
    assert np.array_equal(vb, exact)                         # TwoSum: exact for every element
    assert (~dominated).sum() > 0 and np.any(va[~dominated] != exact[~dominated])
    assert sb["edq"] == pytest.approx(float(np.sqrt(np.sum(bits_to_f64(d) ** 2))), rel=1e-12)


def test_split_decay_applies_the_decay_that_the_summed_form_absorbs():
    # with |r| ~ 1 the term lam*theta is absorbed in r (+) lam*theta (bfloat16 keeps 8 bits), so the summed form
    # barely decays; applied on its own the decay reaches the expansion exactly
    n = 1 << 14
    th0 = np.full(n, oracle.round_to_bf16(0.02), np.uint16)
    g = W.bits(W.flat_grads(n, 8, 1))
    summed, split = _state(th0.copy(), 1), _state(th0.copy(), 1)
    _, d1 = _step(summed, g, 1, 1, want_delta=True)
    ss, d2 = _step(split, g, 1, 1, want_delta=True, flags=oracle.FLAG_DECAY_BY_GROW)
    sc = oracle.derive_scalars(**{k: HYP[k] for k in ("lr", "beta1", "beta2", "eps")}, wd=HYP["weight_decay"], step=1)
    decay = oracle.binary_op(oracle.OP_MUL, np.full(n, sc["a"] ^ 0x8000, np.uint16),
                             oracle.binary_op(oracle.OP_MUL, np.full(n, sc["lam"], np.uint16), th0))
    got = bits_to_f64(split["x_hi"]) + bits_to_f64(split["x_lo"])
    want = bits_to_f64(th0) + bits_to_f64(decay) + bits_to_f64(d2)
    assert np.all(np.abs(got - want) <= ulp_f64(split["x_lo"]) / 2 + 1e-300)
    intended = bits_to_f64(decay) + bits_to_f64(d2)
    assert ss["sumsq"] == pytest.approx(float(np.sum(intended ** 2)), rel=1e-12)
    # the summed form moved theta by the Adam part only (decay absorbed for most elements)
    moved = (bits_to_f64(summed["x_hi"]) + bits_to_f64(summed["x_lo"])) - bits_to_f64(th0)
    assert np.mean(np.abs(moved - bits_to_f64(d2)) < np.abs(bits_to_f64(decay)) / 2) > 0.5


def test_variants_against_exact_rationals():
    rng = np.random.default_rng(12)
    thetas = rng.choice(bf16_window(-9, 1), 24)
    hyp = dict(lr=2e-3, beta1=0.9, beta2=0.98, eps=1e-8, weight_decay=0.01)
    cases = [(3, 0), (1, oracle.FLAG_TWOSUM_GROW), (2, oracle.FLAG_TWOSUM_GROW), (0, oracle.FLAG_DECAY_BY_GROW),
             (1, oracle.FLAG_DECAY_BY_GROW), (2, oracle.FLAG_DECAY_BY_GROW | oracle.FLAG_TWOSUM_GROW)]
    for strategy, flags in cases:
        st = _state(thetas.copy(), strategy)
        ref = [(int(b), 0, 0, 0, 0) for b in thetas]
        for t in range(1, 7):
            g = rng.choice(bf16_window(-14, -6), thetas.size)
            _, d = _step(st, g, t, strategy, hyp=hyp, want_delta=True, flags=flags)
            sc = R.scalars("2e-3", "0.9", "0.98", "1e-8", "0.01", t)
            for i in range(thetas.size):
                *ref_i, delta = R.adamw_element_variant(*ref[i], int(g[i]), sc, strategy,
                                                        twosum_grow=bool(flags & oracle.FLAG_TWOSUM_GROW),
                                                        split_decay=bool(flags & oracle.FLAG_DECAY_BY_GROW))
                got = (int(st["x_hi"][i]), int(st["x_lo"][i]) if st["x_lo"] is not None else 0, int(st["m"][i]),
                       int(st["v_hi"][i]), int(st["v_lo"][i]) if strategy == 2 else 0)
                same = all(a == b or ((a | b) & 0x7FFF) == 0 for a, b in zip(got, ref_i))
                assert same and int(d[i]) == delta, (strategy, flags, t, i, got, ref_i)
                ref[i] = got
