"""GPU parity of the fused AdamW step against the oracle: every state array bit for bit, EDQ within 1e-5."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import EdqBuffers, Guarded, assert_same_bits, edq_close, oracle_state, oracle_step
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import workloads as W

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("step_kernel")]

KEYS = ("x_hi", "x_lo", "m", "v_hi", "v_lo")


def _device_state(st: dict, misalign=0):
    return {k: (Guarded(v, misalign) if v is not None else None) for k, v in st.items()}


def _t(g):
    return g.t if g is not None else None


def _compare(dev: dict, st: dict, what):
    for k in KEYS:
        if st[k] is not None:
            assert_same_bits(dev[k].bits(), st[k], f"{what} {k}")
            assert dev[k].guards_intact(), f"{what} {k}: guard band overwritten"


@pytest.mark.parametrize("strategy", [0, 1, 2])
def test_config0_ten_steps_bitwise_with_edq(strategy):
    # 1,048,576 parameters, theta ~ N(0, 0.02^2), fresh gradient ~ N(0, (1e-3)^2) per step, 10 steps
    n, hyp = 1 << 20, W.HYPERS
    theta = W.bits(W.flat_weights(n, 0))
    st = oracle_state(theta, strategy)
    dev = _device_state(st)
    e = EdqBuffers()
    for t in range(1, 11):
        g = W.bits(W.flat_grads(n, 0, t))
        G = Guarded(g)
        B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n,
                     e.hyper(hyp), t, strategy)
        torch.cuda.synchronize()
        want = oracle_step(st, g, t, strategy, hyp)
        _compare(dev, st, f"strategy {strategy} step {t}")
        assert np.array_equal(G.bits(), g) and G.guards_intact()
        got = e.read()
        edq_close(got, want)
        assert got["n"] == n


@pytest.mark.parametrize("strategy", [0, 1, 2])
@pytest.mark.parametrize("n,misalign", [(1, 0), (7, 0), (8, 0), (9, 0), (4095, 0), (4097, 0), (16384, 0), (16385, 0),
                                        (100_003, 0), (4097, 1), (65_536, 3), (33, 5), (2_000_001, 0)])
def test_ragged_sizes_and_misaligned_pointers(strategy, n, misalign):
    hyp = dict(W.HYPERS, beta2=0.95)
    theta = W.bits(W.flat_weights(n, 40 + n % 7))
    st = oracle_state(theta, strategy)
    dev = _device_state(st, misalign)
    e = EdqBuffers()
    for t in (1, 2, 3):
        g = W.bits(W.flat_grads(n, 41, t))
        G = Guarded(g, misalign)
        B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n,
                     e.hyper(hyp), t, strategy)
        torch.cuda.synchronize()
        want = oracle_step(st, g, t, strategy, hyp, threads=1)
        _compare(dev, st, f"n={n} misalign={misalign} step {t}")
        edq_close(e.read(), want)


def test_mixed_alignment_between_arrays():
    # only one array off its 16-byte boundary: the whole tensor must take the element-wise path
    n, strategy, hyp = 50_000, 2, W.HYPERS
    theta = W.bits(W.flat_weights(n, 9))
    st = oracle_state(theta, strategy)
    dev = {k: Guarded(v, 4 if k == "m" else 0) for k, v in st.items()}
    g = W.bits(W.flat_grads(n, 9, 1))
    G = Guarded(g)
    e = EdqBuffers()
    B.adamw_step(dev["x_hi"].t, dev["x_lo"].t, dev["m"].t, dev["v_hi"].t, dev["v_lo"].t, G.t, n, e.hyper(hyp), 1, strategy)
    torch.cuda.synchronize()
    want = oracle_step(st, g, 1, strategy, hyp)
    _compare(dev, st, "mixed alignment")
    edq_close(e.read(), want)


@pytest.mark.parametrize("strategy", [0, 2])
def test_eps_inside_sqrt_flag_and_no_edq(strategy):
    n, hyp = 300_000, dict(lr=3e-3, beta1=0.9, beta2=0.98, eps=1e-6, weight_decay=0.01)
    theta = W.bits(W.flat_weights(n, 12))
    st = oracle_state(theta, strategy)
    dev = _device_state(st)
    for t in (1, 2):
        g = W.bits(W.flat_grads(n, 12, t))
        G = Guarded(g)
        h = B.make_hyper(**hyp, flags=B.FLAG_EPS_INSIDE_SQRT)        # edq_out NULL: no reduction, no workspace
        B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n, h, t, strategy)
        torch.cuda.synchronize()
        oracle_step(st, g, t, strategy, hyp, flags=oracle.FLAG_EPS_INSIDE_SQRT)
        _compare(dev, st, f"eps inside, step {t}")


def test_special_values_propagate_like_ieee():
    # zeros of both signs, subnormals, huge values, infinities and NaNs in every input array
    rng = np.random.default_rng(77)
    special = np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x007F, 0x0080, 0x7F7F, 0xFF7F, 0x7F80, 0xFF80, 0x7FC0, 0xFFC1,
                        0x3F80, 0xBF80, 0x0200, 0x7E00, 0x1234, 0x6789], dtype=np.uint16)
    n = 200_000
    for strategy in (0, 1, 2):
        st = {k: rng.choice(special, n) for k in KEYS}
        if strategy < 1: st["x_lo"] = None
        if strategy < 2: st["v_lo"] = None
        g = rng.choice(special, n)
        dev = _device_state(st)
        G = Guarded(g)
        h = B.make_hyper(**W.HYPERS)
        B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n, h, 3, strategy)
        torch.cuda.synchronize()
        oracle_step(st, g, 3, strategy, W.HYPERS)
        _compare(dev, st, f"special values strategy {strategy}")


def test_stress_lost_arithmetic_config_short():
    # config-2 distributions (theta = +-U(0.5,4), log-uniform gradients, lr 1e-5): 1M-element slice, 30 steps, C and A
    n, hyp = 1 << 20, W.HYPERS_STRESS
    theta = W.bits(W.stress_weights(n, 2))
    edq_hist = {}
    for strategy in (2, 0):
        st = oracle_state(theta, strategy)
        dev = _device_state(st)
        e = EdqBuffers()
        hist = []
        for t in range(1, 31):
            g = W.bits(W.stress_grads(n, 2, t))
            G = Guarded(g)
            B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n,
                         e.hyper(hyp), t, strategy)
            torch.cuda.synchronize()
            want = oracle_step(st, g, t, strategy, hyp)
            got = e.read()
            edq_close(got, want)
            hist.append(got)
        _compare(dev, st, f"stress strategy {strategy}")
        edq_hist[strategy] = hist
    # plain bfloat16 loses most updates here (Def. 3.2: |update| <= ulp(theta)/2).  Collage-plus loses only those
    # below the reach of its second component: a length-2 bfloat16 expansion resolves about 2^-17 |theta|
    # (|dtheta| <= ulp(theta)/2 = 2^-9 |theta|, and dtheta has 8 bits of its own), and with lr 1e-5 and gradients
    # down to 1e-8 a few per cent of the updates are smaller than that; hence 5 %, not 0
    assert edq_hist[0][-1]["lost"] > 0.5 * n
    assert edq_hist[2][-1]["lost"] < 0.05 * n
    assert edq_hist[2][-1]["edq"] > edq_hist[0][-1]["edq"]


def test_checkpoint_resume_is_bit_identical():
    # the library keeps no state between calls: 6 steps == 3 steps, copy everything out and back, 3 steps
    n, strategy, hyp = 123_457, 2, W.HYPERS
    theta = W.bits(W.flat_weights(n, 21))
    grads = [W.bits(W.flat_grads(n, 21, t)) for t in range(1, 7)]

    def run(dev, t):
        G = Guarded(grads[t - 1])
        B.adamw_step(dev["x_hi"].t, dev["x_lo"].t, dev["m"].t, dev["v_hi"].t, dev["v_lo"].t, G.t, n,
                     B.make_hyper(**hyp), t, strategy)
        torch.cuda.synchronize()

    a = _device_state(oracle_state(theta, strategy))
    for t in range(1, 7):
        run(a, t)
    b = _device_state(oracle_state(theta, strategy))
    for t in range(1, 4):
        run(b, t)
    saved = {k: b[k].bits() for k in KEYS}
    c = {k: Guarded(v, 2) for k, v in saved.items()}          # resume in different, differently aligned buffers
    for t in range(4, 7):
        run(c, t)
    for k in KEYS:
        assert np.array_equal(a[k].bits(), c[k].bits()), k


def test_wrong_device_arguments_are_rejected():
    z = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    h = B.make_hyper(**W.HYPERS)
    with pytest.raises(B.CollageError) as err:
        B.adamw_step(z, None, z, z.clone(), None, z.clone(), 64, h, 1, B.BF16)      # m aliases x_hi
    assert err.value.status == B.ERR_ALIAS
    with pytest.raises(B.CollageError) as err:
        B.adamw_step(z, None, z.clone(), z.clone(), None, z.clone(), 64, h, 0, B.BF16)
    assert err.value.status == B.ERR_ARG
    B.adamw_step(z, None, z.clone(), z.clone(), None, z.clone(), 0, h, 1, B.BF16)    # n == 0: fine, no-op
    torch.cuda.synchronize()


@pytest.mark.parametrize("strategy", [0, 2])
def test_host_resident_state_is_staged_with_identical_results(strategy):
    # state in pinned host memory, streamed through a small device buffer so that the step takes many slabs
    n, hyp = 300_007, W.HYPERS
    theta = W.bits(W.flat_weights(n, 31))
    st = oracle_state(theta, strategy)
    host = {k: (W.from_bits(v).pin_memory() if v is not None else None) for k, v in st.items()}
    staging = torch.empty(256 + B.workspace_bytes() + 2 * 6 * 2 * 16384 * 2 + 4096, dtype=torch.uint8, device="cuda")
    import ctypes
    rec = (ctypes.c_uint8 * 64)()
    for t in (1, 2, 3):
        g = W.bits(W.flat_grads(n, 31, t))
        G = W.from_bits(g).pin_memory()
        h = B.make_hyper(**hyp)
        h.edq_out = ctypes.addressof(rec)
        B.adamw_step_host(host["x_hi"], host["x_lo"], host["m"], host["v_hi"], host["v_lo"], G, n, h, t, strategy, staging)
        torch.cuda.synchronize()
        want = oracle_step(st, g, t, strategy, hyp)
        for k in KEYS:
            if st[k] is not None:
                assert_same_bits(W.bits(host[k]), st[k], f"host step {t} {k}")
        got = B.Edq.from_buffer_copy(bytes(rec)[:B.EDQ_RECORD_BYTES])
        edq_close(dict(dot=got.dot, sumsq=got.sumsq, edq=got.edq, lost=int(got.lost)), want)
        assert int(got.n) == n
    with pytest.raises(B.CollageError) as err:
        B.adamw_step_host(host["x_hi"], host["x_lo"], host["m"], host["v_hi"], host["v_lo"], G, n, B.make_hyper(**hyp), 1,
                          strategy, staging[:1024])
    assert err.value.status == B.ERR_WORKSPACE


@pytest.mark.parametrize("eps", [0.0, 1e-40, 1e-20, 1e30])
@pytest.mark.parametrize("flags", [0, 1])
def test_unusual_epsilon_takes_the_guarded_arithmetic_chain(eps, flags):
    # outside 2^-54 <= eps <= 2^60 the kernel cannot assume a normal denominator: zero and subnormal moments,
    # zero denominators (0/0 -> NaN, x/0 -> Inf) must all come out as IEEE says
    n, strategy = 100_000, 2
    hyp = dict(W.HYPERS, eps=eps)
    rng = np.random.default_rng(5)
    theta = W.bits(W.flat_weights(n, 50))
    st = oracle_state(theta, strategy)
    st["v_hi"] = rng.choice(np.array([0x0000, 0x0001, 0x0040, 0x0080, 0x1000, 0x3000], np.uint16), n)
    st["m"] = rng.choice(np.array([0x0000, 0x8000, 0x0003, 0x2000, 0xB000], np.uint16), n)
    dev = _device_state(st)
    for t in (1, 2):
        g = W.bits(W.flat_grads(n, 50, t))
        g[::3] = 0
        G = Guarded(g)
        B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n,
                     B.make_hyper(**hyp, flags=flags), t, strategy)
        torch.cuda.synchronize()
        oracle_step(st, g, t, strategy, hyp, flags=flags)
        _compare(dev, st, f"eps={eps} flags={flags} step {t}")


def test_zero_and_subnormal_moments_on_the_lean_chain():
    # default epsilon (lean chain): parameters that never saw a gradient, subnormal moments, huge moments
    n, strategy, hyp = 100_000, 2, W.HYPERS
    rng = np.random.default_rng(6)
    theta = W.bits(W.flat_weights(n, 51))
    st = oracle_state(theta, strategy)
    st["v_hi"] = rng.choice(np.array([0x0000, 0x0001, 0x007F, 0x0080, 0x0100, 0x3000, 0x7F00, 0x7F7F], np.uint16), n)
    st["m"] = rng.choice(np.array([0x0000, 0x8000, 0x0001, 0x8003, 0x0080, 0x2000, 0xB000, 0x7F00, 0xFF7F], np.uint16), n)
    dev = _device_state(st)
    e = EdqBuffers()
    for t in (1, 2, 3):
        g = W.bits(W.flat_grads(n, 51, t))
        g[::2] = 0
        G = Guarded(g)
        B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n,
                     e.hyper(hyp), t, strategy)
        torch.cuda.synchronize()
        oracle_step(st, g, t, strategy, hyp)
        _compare(dev, st, f"lean chain step {t}")


def test_negative_second_moment_gives_nan_not_a_flushed_zero():
    # invalid state (v < 0, including negative subnormals) must come out NaN exactly as IEEE says
    n, hyp = 8192, W.HYPERS
    for strategy in (0, 2):
        rng = np.random.default_rng(9)
        theta = W.bits(W.flat_weights(n, 52))
        st = oracle_state(theta, strategy)
        st["v_hi"] = rng.choice(np.array([0x8001, 0x807F, 0x8080, 0xB000, 0x0001, 0x3000], np.uint16), n)
        dev = _device_state(st)
        g = np.zeros(n, np.uint16)
        G = Guarded(g)
        B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n,
                     B.make_hyper(**hyp), 5, strategy)
        torch.cuda.synchronize()
        oracle_step(st, g, 5, strategy, hyp)
        _compare(dev, st, f"negative v, strategy {strategy}")


@pytest.mark.parametrize("strategy", [0, 1, 2])
def test_sparse_rare_lanes_between_ordinary_ones_keep_state_edq_and_lost_exact(strategy):
    # Ordinary training state with about one lane in a hundred that the lean chain cannot answer by itself
    # (subnormal or zero first moments, huge or subnormal second moments: tiny and tied quotients), and as many
    # parameters whose update is lost even as a pair (theta = 2^31 with delta-theta = +-2^20, zeros of either
    # sign beside them).  Vectors with and without such a lane alternate inside every tile; several tiles and
    # a ragged tail.  State bit for bit, EDQ sums within tolerance, the lost count exactly.
    n, hyp = 300_007, dict(W.HYPERS, weight_decay=0.0)
    rng = np.random.default_rng(1234 + strategy)
    st = oracle_state(W.bits(W.flat_weights(n, 61)), strategy)
    dev = _device_state(st)
    e = EdqBuffers()

    def step(t):
        g = W.bits(W.flat_grads(n, 61, t))
        g[rng.random(n) < 0.01] = 0
        G = Guarded(g)
        B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n,
                     e.hyper(hyp), t, strategy)
        torch.cuda.synchronize()
        want = oracle_step(st, g, t, strategy, hyp)
        edq_close(e.read(), want)
        _compare(dev, st, f"sparse rare lanes, strategy {strategy}, step {t}")
        return want

    step(1)
    # poke the rare lanes into the (identical) host and device copies
    where = lambda p: np.flatnonzero(rng.random(n) < p)
    i = where(0.01)
    st["m"][i] = rng.choice(np.array([0x0000, 0x8000, 0x0001, 0x8003, 0x0080], np.uint16), i.size)
    i = where(0.01)
    st["v_hi"][i] = rng.choice(np.array([0x7F00, 0x7F7F, 0x0001, 0x007F, 0x0000], np.uint16), i.size)
    i = where(0.01)
    st["x_hi"][i] = rng.choice(np.array([0x4F00, 0xCF00], np.uint16), i.size)
    if strategy >= 1:
        st["x_lo"][i] = rng.choice(np.array([0x4980, 0xC980, 0x0000, 0x8000], np.uint16), i.size)
    dev = _device_state(st)
    lost = [step(t)["lost"] for t in (2, 3, 4)]
    assert min(lost) > 0        # the poked parameters do lose updates, so the exact count is exercised


HYPER_SWEEP = [
    # lr, beta1, beta2, eps, weight_decay, step
    (1e-4, 0.9, 0.999, 1e-8, 0.1, 1),
    (1e-4, 0.9, 0.999, 1e-8, 0.1, 1_000_000),        # bias corrections round to 1
    (1e-4, 0.9, 0.999, 1e-8, 0.1, 10 ** 9),
    (0.0, 0.9, 0.999, 1e-8, 0.1, 3),                 # zero learning rate: every update is a signed zero
    (1.0, 0.0, 0.5, 1e-8, 0.0, 2),                   # no momentum, fast second moment, huge steps
    (3e-3, 0.5, 0.95, 1e-6, 0.5, 7),
    (1e-5, 0.99, 0.9999, 1e-10, 0.01, 1000),
    (6e-4, 0.9, 0.95, 1e-5, 0.1, 50),
    (1e-2, 0.999, 0.9999, 1e-3, 1.0, 12345),
    (2.5e-4, 0.8, 0.0, 1.0, 0.0, 4),                 # beta2 = 0: v is the last squared gradient; eps = 1
]


@pytest.mark.parametrize("strategy", [0, 1, 2, 3])
def test_hyper_parameter_and_step_sweep(strategy):
    # one step from a mid-training state for every row of the sweep: scalars derived on both sides independently
    n = 70_001
    rng = np.random.default_rng(40 + strategy)
    for lr, b1, b2, eps, wd, t in HYPER_SWEEP:
        hyp = dict(lr=lr, beta1=b1, beta2=b2, eps=eps, weight_decay=wd)
        st = oracle_state(W.bits(W.flat_weights(n, 90)), strategy)
        st["m"] = W.bits(W.normal_bf16(n, 1e-3, 91))
        v = W.normal_bf16(n, 1e-3, 92).float().square().to(torch.bfloat16)
        st["v_hi"] = W.bits(v)
        if st["x_lo"] is not None:
            st["x_lo"] = W.bits(W.normal_bf16(n, 2e-5, 93))
        if st["v_lo"] is not None:              # a second component well below the first, either sign
            st["v_lo"] = W.bits((v.float() * 1.5e-3 * torch.sign(W.normal_bf16(n, 1.0, 94).float())).to(torch.bfloat16))
        g = W.bits(W.flat_grads(n, 90, 1))
        g[rng.random(n) < 0.02] = 0
        dev = _device_state(st)
        e = EdqBuffers()
        G = Guarded(g)
        B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n,
                     e.hyper(hyp), t, strategy)
        torch.cuda.synchronize()
        want = oracle_step(st, g, t, strategy, hyp)
        _compare(dev, st, f"hypers {hyp} step {t} strategy {strategy}")
        edq_close(e.read(), want)


@pytest.mark.parametrize("strategy", [1, 2])
def test_lost_counts_values_that_did_not_move_on_planted_resplit_pairs(strategy):
    # Pairs on which Grow hands back the same value over other components, planted densely: the count
    # follows the value (Eq. 2's effective update is zero), not the stored bit patterns.  beta1 = beta2 = 0,
    # no decay and g = -+1 make the update exactly +-RN(lr) at step 1, so the planted update is what the step applies.
    from gpu_util import resplit_pairs
    a_bits = 0x35AB
    lr = float(oracle.widen(a_bits))
    hyp = dict(lr=lr, beta1=0.0, beta2=0.0, eps=1e-8, weight_decay=0.0)
    xp, yp = resplit_pairs(a_bits)                       # update +a
    xm, ym = resplit_pairs(a_bits | 0x8000)              # update -a
    assert xp.size > 500 and xm.size > 500
    rng = np.random.default_rng(99)
    n = 300_011
    th = W.bits(W.stress_weights(n, 5)); dth = np.zeros(n, np.uint16)
    g = np.where(rng.integers(0, 2, n) == 1, np.uint16(0x3F80), np.uint16(0xBF80)).astype(np.uint16)
    planted = rng.random(n) < 0.5
    for sign_bits, (xs, ys) in ((0xBF80, (xp, yp)), (0x3F80, (xm, ym))):      # g = -1 gives +a, g = +1 gives -a
        idx = np.flatnonzero(planted & (g == sign_bits))
        k = rng.integers(0, xs.size, idx.size)
        th[idx], dth[idx] = xs[k], ys[k]
    st = oracle_state(th, strategy)
    st["x_lo"] = dth.copy()
    before = (st["x_hi"].copy(), st["x_lo"].copy())
    dev = _device_state(st)
    e = EdqBuffers()
    G = Guarded(g)
    B.adamw_step(_t(dev["x_hi"]), _t(dev["x_lo"]), _t(dev["m"]), _t(dev["v_hi"]), _t(dev["v_lo"]), G.t, n, e.hyper(hyp), 1, strategy)
    torch.cuda.synchronize()
    want = oracle_step(st, g, 1, strategy, hyp)
    _compare(dev, st, f"planted resplit pairs, strategy {strategy}")
    got = e.read()
    edq_close(got, want)
    components_same = int(np.sum((st["x_hi"] == before[0]) & (st["x_lo"] == before[1])))
    assert got["lost"] >= int(planted.sum()) > n // 3            # every planted pair is counted ...
    assert got["lost"] - components_same >= int(planted.sum())   # ... and none of them kept its bit patterns
