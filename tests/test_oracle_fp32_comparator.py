"""Pins for the oracle's option-D comparator (float optimizer states, float master weights; Table 2,
Section 5.1) and its D^-MW form.

Fixed by: agreement with AdamW in double to float accuracy, the invariant theta == RN_bf16(master),
the master weight keeping updates that the bfloat16 parameter cannot show (Section 2.1, master
weights), and a numpy float32 evaluation of the same operation order (checks that the C++ floats
are plain IEEE single operations with no contraction or extended precision).
"""
import numpy as np
import pytest

import oracle
from conftest import bits_to_f64
from paper_2405_03637_b200 import workloads as W

HYP = dict(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)


def _fresh(n, seed, with_master=True):
    theta = W.bits(W.flat_weights(n, seed))
    master = bits_to_f64(theta).astype(np.float32) if with_master else None
    return theta, master, np.zeros(n, np.float32), np.zeros(n, np.float32)


def test_master_weights_follow_fp64_adamw_to_float_accuracy():
    n, T = 1 << 14, 60
    theta, master, m, v = _fresh(n, 0)
    th64 = bits_to_f64(theta).copy(); m64 = np.zeros(n); v64 = np.zeros(n)
    moved = np.zeros(n)
    for t in range(1, T + 1):
        g = W.bits(W.flat_grads(n, 0, t))
        oracle.adamw_fp32_step(theta, master, m, v, g, step=t, **HYP)
        d = oracle.adamw_fp64(th64, m64, v64, bits_to_f64(g), step=t, want_delta=True, **HYP)
        moved += np.abs(d)
        assert np.array_equal(theta, oracle.round_to_bf16(master.astype(np.float64)))      # theta = RN(master)
    assert np.all(np.abs(master - th64) <= 2e-6 * moved + 4 * T * 2.0 ** -24 * np.abs(th64))
    assert np.allclose(m, m64, rtol=1e-5, atol=1e-9) and np.allclose(v, v64, rtol=1e-5, atol=1e-15)


def test_master_weight_keeps_updates_below_half_an_ulp_of_the_bf16_parameter():
    n = 512
    theta = np.full(n, oracle.round_to_bf16(200.0), np.uint16)
    master = np.full(n, 200.0, np.float32)
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    g = np.full(n, oracle.round_to_bf16(1e-3), np.uint16)
    hyp = dict(HYP, lr=0.1, weight_decay=0.0)
    for t in range(1, 4):
        s = oracle.adamw_fp32_step(theta, master, m, v, g, step=t, **hyp)
        assert s["lost"] == 0 and s["edq"] == pytest.approx(np.sqrt(s["sumsq"]), rel=2e-4)   # float ulp at 200 is 1.5e-5 of an update of 0.1
    assert np.all(theta == oracle.round_to_bf16(200.0))          # 200 - 0.3 still rounds to 200 in bfloat16
    assert np.all(np.abs(master - 199.7) < 1e-3)                 # the master weight did move
    for t in range(4, 8):
        oracle.adamw_fp32_step(theta, master, m, v, g, step=t, **hyp)
    assert np.all(bits_to_f64(theta) == 199.0)                   # ... and theta follows once it crosses half an ulp
    # without master weights every one of these updates is lost
    theta2 = np.full(n, oracle.round_to_bf16(200.0), np.uint16)
    m2, v2 = np.zeros(n, np.float32), np.zeros(n, np.float32)
    for t in range(1, 8):
        s = oracle.adamw_fp32_step(theta2, None, m2, v2, g, step=t, **hyp)
        assert s["lost"] == n and s["edq"] == 0.0
    assert np.all(theta2 == oracle.round_to_bf16(200.0))


@pytest.mark.parametrize("with_master", [True, False])
@pytest.mark.parametrize("flags", [0, 1])
def test_every_operation_is_one_ieee_single_operation(with_master, flags):
    n = 1 << 13
    theta, master, m, v = _fresh(n, 5, with_master)
    f = np.float32
    hyp = dict(lr=3e-3, beta1=0.9, beta2=0.98, eps=1e-6, weight_decay=0.01)
    th_np = theta.copy()
    w_np = master.copy() if with_master else None
    m_np, v_np = m.copy(), v.copy()
    for t in range(1, 6):
        gb = W.bits(W.flat_grads(n, 5, t))
        oracle.adamw_fp32_step(theta, master, m, v, gb, step=t, flags=flags, **hyp)
        g = bits_to_f64(gb).astype(f)
        b1, c1 = f(hyp["beta1"]), f(1.0 - hyp["beta1"])
        b2, c2 = f(hyp["beta2"]), f(1.0 - hyp["beta2"])
        bc1, bc2 = f(1.0 - hyp["beta1"] ** t), f(1.0 - hyp["beta2"] ** t)
        m_np = b1 * m_np + c1 * g
        v_np = b2 * v_np + c2 * (g * g)
        vhat = v_np / bc2
        den = np.sqrt(vhat + f(hyp["eps"])) if flags else np.sqrt(vhat) + f(hyp["eps"])
        w_old = w_np if with_master else bits_to_f64(th_np).astype(f)
        delta = f(-f(hyp["lr"])) * ((m_np / bc1) / den + f(hyp["weight_decay"]) * w_old)
        w_new = w_old + delta
        assert w_new.dtype == np.float32
        th_np = oracle.round_to_bf16(w_new.astype(np.float64))
        if with_master:
            w_np = w_new
            assert np.array_equal(master.view(np.uint32), w_np.view(np.uint32))
        assert np.array_equal(theta, th_np)
        assert np.array_equal(m.view(np.uint32), m_np.view(np.uint32))
        assert np.array_equal(v.view(np.uint32), v_np.view(np.uint32))


def test_no_master_weights_rounds_the_float_sum_to_bf16():
    n = 4096
    theta, _, m, v = _fresh(n, 9, with_master=False)
    before = theta.copy()
    g = W.bits(W.flat_grads(n, 9, 1))
    s = oracle.adamw_fp32_step(theta, None, m, v, g, step=1, **HYP)
    eff = bits_to_f64(theta) - bits_to_f64(before)
    assert s["lost"] == int(np.sum(eff == 0))                     # every update is non-zero here
    # at t = 1 the update is -lr * (sign(g) * |g|/(|g|+eps) + wd*theta) up to float rounding
    gf = bits_to_f64(g)
    want = bits_to_f64(before) - 1e-4 * (gf / (np.abs(gf) + 1e-8) + 0.1 * bits_to_f64(before))
    assert np.mean(theta == oracle.round_to_bf16(want)) > 0.999      # all but float-vs-double near-ties


# ---- variant: float arithmetic in registers on the Collage-plus storage ---------------------------

def _pair_state(n, seed):
    theta = W.bits(W.flat_weights(n, seed))
    z = lambda: np.zeros(n, np.uint16)
    return dict(x_hi=theta, x_lo=z(), m=z(), v_hi=z(), v_lo=z())


def test_register_variant_stores_normalised_pairs_and_tracks_fp64_adamw():
    n, T = 1 << 14, 50
    hyp = dict(HYP, beta2=0.95)
    st = _pair_state(n, 0)
    strict = {k: v.copy() for k, v in st.items()}
    th64 = bits_to_f64(st["x_hi"]).copy(); m64 = np.zeros(n); v64 = np.zeros(n)
    moved = np.zeros(n)
    for t in range(1, T + 1):
        g = W.bits(W.flat_grads(n, 0, t))
        s = oracle.adamw_fp32_register_step(st["x_hi"], st["x_lo"], st["m"], st["v_hi"], st["v_lo"], g, step=t, **hyp)
        oracle.adamw_step(strict["x_hi"], strict["x_lo"], strict["m"], strict["v_hi"], strict["v_lo"], g, step=t,
                          strategy=oracle.STRATEGY_PLUS, **hyp)
        moved += np.abs(oracle.adamw_fp64(th64, m64, v64, bits_to_f64(g), step=t, want_delta=True, **hyp))
        # the split is a normalised expansion (Def. 2.1): |lo| <= ulp(hi)/2, for theta and for v
        from conftest import ulp_f64
        assert np.all(np.abs(bits_to_f64(st["x_lo"])) <= ulp_f64(st["x_hi"]) / 2)
        assert np.all(np.abs(bits_to_f64(st["v_lo"])) <= ulp_f64(st["v_hi"]) / 2)
        assert s["lost"] <= n // 100                          # updates below the ~2^-17 resolution of the pair
    held = bits_to_f64(st["x_hi"]) + bits_to_f64(st["x_lo"])
    held_strict = bits_to_f64(strict["x_hi"]) + bits_to_f64(strict["x_lo"])
    err, err_strict = np.abs(held - th64), np.abs(held_strict - th64)
    # a bfloat16 pair resolves ~2^-16 of theta per step; m is stored in bfloat16 (2^-9 relative), which bounds
    # how far the update can drift from the double one
    assert np.all(err <= 0.01 * moved + T * 2.0 ** -16 * np.abs(th64))
    # and float arithmetic in registers sits closer to the double trajectory than strict bfloat16 arithmetic
    assert err.sum() < 0.5 * err_strict.sum()
    vv = bits_to_f64(st["v_hi"]) + bits_to_f64(st["v_lo"])
    assert np.all(np.abs(vv - v64) <= 2.0 ** -14 * v64 + 1e-30)


def test_register_variant_matches_a_numpy_float32_evaluation():
    n = 1 << 12
    f = np.float32
    hyp = dict(lr=3e-3, beta1=0.9, beta2=0.98, eps=1e-6, weight_decay=0.01)
    st = _pair_state(n, 4)
    ref = {k: v.copy() for k, v in st.items()}
    w = lambda b: bits_to_f64(b).astype(f)
    rn = lambda x: oracle.round_to_bf16(x.astype(np.float64))
    for t in range(1, 6):
        gb = W.bits(W.flat_grads(n, 4, t))
        oracle.adamw_fp32_register_step(st["x_hi"], st["x_lo"], st["m"], st["v_hi"], st["v_lo"], gb, step=t, **hyp)
        g = w(gb)
        x = w(ref["x_hi"]) + w(ref["x_lo"])
        vv = w(ref["v_hi"]) + w(ref["v_lo"])
        m_new = f(hyp["beta1"]) * w(ref["m"]) + f(1.0 - hyp["beta1"]) * g
        v_new = f(hyp["beta2"]) * vv + f(1.0 - hyp["beta2"]) * (g * g)
        den = np.sqrt(v_new / f(1.0 - hyp["beta2"] ** t)) + f(hyp["eps"])
        delta = f(-f(hyp["lr"])) * ((m_new / f(1.0 - hyp["beta1"] ** t)) / den + f(hyp["weight_decay"]) * x)
        x_new = x + delta
        ref["x_hi"] = rn(x_new); ref["x_lo"] = rn(x_new - w(ref["x_hi"]))
        ref["m"] = rn(m_new)
        ref["v_hi"] = rn(v_new); ref["v_lo"] = rn(v_new - w(ref["v_hi"]))
        for k in st:
            assert np.array_equal(st[k], ref[k]), (t, k)
