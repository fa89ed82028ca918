"""GPU parity of the comparator and variant steps (BF16-Kahan, TwoSum-based Grow, decay by its own
addition) against the oracle: every state array bit for bit, EDQ within 1e-5."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import EdqBuffers, Guarded, assert_same_bits, edq_close, oracle_step
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import workloads as W

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("step_kernel")]
KEYS = ("x_hi", "x_lo", "m", "v_hi", "v_lo")

CASES = [
    (B.KAHAN, 0), (B.KAHAN, B.FLAG_EPS_INSIDE_SQRT),
    (B.LIGHT, B.FLAG_TWOSUM_GROW), (B.PLUS, B.FLAG_TWOSUM_GROW),
    (B.BF16, B.FLAG_DECAY_BY_GROW), (B.LIGHT, B.FLAG_DECAY_BY_GROW), (B.PLUS, B.FLAG_DECAY_BY_GROW),
    (B.PLUS, B.FLAG_DECAY_BY_GROW | B.FLAG_TWOSUM_GROW | B.FLAG_EPS_INSIDE_SQRT),
]


def _state(theta, strategy):
    z = lambda: np.zeros_like(theta)
    return dict(x_hi=theta.copy(), x_lo=z() if strategy >= 1 else None, m=z(), v_hi=z(), v_lo=z() if strategy == 2 else None)


@pytest.mark.parametrize("strategy,flags", CASES)
@pytest.mark.parametrize("n,misalign", [(1 << 20, 0), (100_003, 0), (4097, 3), (9, 0)])
def test_variant_steps_bitwise(strategy, flags, n, misalign):
    hyp = dict(W.HYPERS, beta2=0.98)
    theta = W.bits(W.flat_weights(n, 60))
    theta[::11] = W.bits(W.flat_grads(n, 61, 1))[::11]         # some parameters as small as their updates
    st = _state(theta, strategy)
    dev = {k: (Guarded(v, misalign) if v is not None else None) for k, v in st.items()}
    t_ = lambda g: g.t if g is not None else None
    e = EdqBuffers()
    for t in (1, 2, 3, 4):
        g = W.bits(W.flat_grads(n, 62, t))
        G = Guarded(g, misalign)
        B.adamw_step(t_(dev["x_hi"]), t_(dev["x_lo"]), t_(dev["m"]), t_(dev["v_hi"]), t_(dev["v_lo"]), G.t, n,
                     e.hyper(hyp, flags), t, strategy)
        torch.cuda.synchronize()
        want = oracle_step(st, g, t, strategy, hyp, flags=flags)
        for k in KEYS:
            if st[k] is not None:
                assert_same_bits(dev[k].bits(), st[k], f"strategy {strategy} flags {flags} step {t} {k}")
                assert dev[k].guards_intact()
        edq_close(e.read(), want)
    assert B.pipeline_fault() == 0


def test_kahan_multi_tensor_and_stress_values():
    # the comparator through the one-launch multi-tensor step, on the lost-arithmetic stress distributions
    shapes = [("a", 300_001), ("b", 4096), ("c", 7), ("d", 65_536)]
    hyp = W.HYPERS_STRESS
    host, dev, grads, rows = [], [], [], []
    for i, (_, n) in enumerate(shapes):
        st = _state(W.bits(W.stress_weights(n, 70 + i)), B.KAHAN)
        host.append(st)
        d = {k: (Guarded(v) if v is not None else None) for k, v in st.items()}
        dev.append(d)
        grads.append(Guarded(np.zeros(n, np.uint16)))
        rows.append((d["x_hi"].t, d["x_lo"].t, d["m"].t, d["v_hi"].t, None, grads[-1].t, n))
    plan = B.plan_create(rows)
    e = EdqBuffers()
    for t in range(1, 11):
        tot = dict(dot=0.0, sumsq=0.0, lost=0)
        for i, (_, n) in enumerate(shapes):
            g = W.bits(W.stress_grads(n, 70 + i, t))
            grads[i].t.copy_(W.from_bits(g, "cuda"))
            s = oracle_step(host[i], g, t, B.KAHAN, hyp)
            tot["dot"] += s["dot"]; tot["sumsq"] += s["sumsq"]; tot["lost"] += s["lost"]
        B.adamw_step_multi(plan, e.hyper(hyp), t, B.KAHAN)
        torch.cuda.synchronize()
        tot["edq"] = tot["dot"] / np.sqrt(tot["sumsq"]) if tot["sumsq"] > 0 else 0.0
        for i in range(len(shapes)):
            for k in ("x_hi", "x_lo", "m", "v_hi"):
                assert_same_bits(dev[i][k].bits(), host[i][k], f"tensor {i} {k} step {t}")
        edq_close(e.read(), tot)
    B.plan_destroy(plan)


def test_flag_combinations_that_mean_nothing_are_rejected():
    z = lambda: torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    a = [z() for _ in range(5)]
    with pytest.raises(B.CollageError) as err:
        B.adamw_step(a[0], None, a[1], a[2], None, a[3], 64, B.make_hyper(**W.HYPERS, flags=B.FLAG_TWOSUM_GROW), 1, B.BF16)
    assert err.value.status == B.ERR_ARG
    with pytest.raises(B.CollageError) as err:
        B.adamw_step(a[0], a[4], a[1], a[2], None, a[3], 64, B.make_hyper(**W.HYPERS, flags=B.FLAG_TWOSUM_GROW), 1, B.KAHAN)
    assert err.value.status == B.ERR_ARG


@pytest.mark.parametrize("n,misalign,flags", [(1 << 20, 0, 0), (100_003, 0, 1), (4097, 3, 0), (9, 0, 0)])
def test_float_arithmetic_in_registers_variant_bitwise(n, misalign, flags):
    # option C's storage, float arithmetic, results split back into bfloat16 pairs
    hyp = dict(W.HYPERS, beta2=0.98)
    theta = W.bits(W.flat_weights(n, 90))
    z = lambda: np.zeros(n, np.uint16)
    st = dict(x_hi=theta.copy(), x_lo=z(), m=z(), v_hi=z(), v_lo=z())
    dev = {k: Guarded(v, misalign) for k, v in st.items()}
    e = EdqBuffers()
    for t in (1, 2, 3, 4):
        g = W.bits(W.flat_grads(n, 91, t))
        G = Guarded(g, misalign)
        B.adamw_step(dev["x_hi"].t, dev["x_lo"].t, dev["m"].t, dev["v_hi"].t, dev["v_lo"].t, G.t, n,
                     e.hyper(hyp, flags), t, B.PLUS_FP32_REGISTERS)
        torch.cuda.synchronize()
        want = oracle.adamw_fp32_register_step(st["x_hi"], st["x_lo"], st["m"], st["v_hi"], st["v_lo"], g, step=t,
                                               flags=flags, **hyp)
        for k in KEYS:
            assert_same_bits(dev[k].bits(), st[k], f"register variant step {t} {k}")
            assert dev[k].guards_intact()
        edq_close(e.read(), want)
    assert B.pipeline_fault() == 0


VARIANT_HYPERS = [
    # lr, beta1, beta2, eps, weight_decay, step
    (1e-4, 0.9, 0.999, 1e-8, 0.1, 1_000_000),
    (0.0, 0.9, 0.999, 1e-8, 0.1, 3),
    (1.0, 0.0, 0.5, 1e-8, 0.0, 2),
    (3e-3, 0.5, 0.95, 1e-6, 0.5, 7),
    (1e-2, 0.999, 0.9999, 1e-3, 1.0, 12345),
]


@pytest.mark.parametrize("strategy,flags", [(1, B.FLAG_TWOSUM_GROW), (2, B.FLAG_TWOSUM_GROW), (2, B.FLAG_DECAY_BY_GROW),
                                            (2, B.FLAG_TWOSUM_GROW | B.FLAG_DECAY_BY_GROW | B.FLAG_EPS_INSIDE_SQRT),
                                            (0, B.FLAG_DECAY_BY_GROW), (4, 0)])
def test_variants_over_a_sweep_of_hyper_parameters(strategy, flags):
    # three steps from zero moments for every row: the flag paths and the register variant derive their scalars
    # from the same host code as the default path, the oracle derives them on its own
    n = 30_011
    for lr, b1, b2, eps, wd, t0 in VARIANT_HYPERS:
        hyp = dict(lr=lr, beta1=b1, beta2=b2, eps=eps, weight_decay=wd)
        theta = W.bits(W.flat_weights(n, 95))
        z = lambda: np.zeros(n, np.uint16)
        st = dict(x_hi=theta.copy(), x_lo=z() if strategy else None, m=z(), v_hi=z(), v_lo=z() if strategy in (2, 4) else None)
        dev = {k: (Guarded(v) if v is not None else None) for k, v in st.items()}
        ptr = lambda k: dev[k].t if dev[k] is not None else None
        e = EdqBuffers()
        for t in (t0, t0 + 1, t0 + 2):
            g = W.bits(W.flat_grads(n, 96, t % 1000))
            G = Guarded(g)
            B.adamw_step(ptr("x_hi"), ptr("x_lo"), ptr("m"), ptr("v_hi"), ptr("v_lo"), G.t, n, e.hyper(hyp, flags), t, strategy)
            torch.cuda.synchronize()
            if strategy == 4:
                want = oracle.adamw_fp32_register_step(st["x_hi"], st["x_lo"], st["m"], st["v_hi"], st["v_lo"], g, step=t,
                                                       flags=flags, **hyp)
            else:
                want, _ = oracle.adamw_step(st["x_hi"], st["x_lo"], st["m"], st["v_hi"], st["v_lo"], g, step=t,
                                            strategy=strategy, flags=flags, **hyp)
            for k in KEYS:
                if st[k] is not None:
                    assert_same_bits(dev[k].bits(), st[k], f"{hyp} step {t} strategy {strategy} flags {flags} {k}")
            edq_close(e.read(), want)
