"""Differential test on random bit patterns: every state array and the gradient drawn from all 2^16 bfloat16
patterns (NaN, infinities, subnormals, zeros of both signs included), random hyper-parameters and step numbers,
every strategy and flag combination; the device must reproduce the oracle bit for bit (NaNs as a class)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same_bits
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import workloads as W

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("step_kernel")]
CASES = [(0, 0), (1, 0), (2, 0), (3, 0), (1, 2), (2, 2), (2, 4), (2, 7), (0, 4), (0, 1), (2, 1), (3, 1)]


def _draw(rng, n, mode):
    if mode == 0:                         # any pattern
        return rng.integers(0, 1 << 16, n, dtype=np.uint16)
    if mode == 1:                         # finite, any exponent
        a = rng.integers(0, 1 << 16, n, dtype=np.uint16)
        a[(a & 0x7F80) == 0x7F80] &= 0x807F
        return a
    e = rng.integers(100, 140, n).astype(np.uint16)          # moderate exponents, both signs
    return ((rng.integers(0, 2, n).astype(np.uint16) << 15) | (e << 7) | rng.integers(0, 128, n).astype(np.uint16)).astype(np.uint16)


@pytest.mark.parametrize("case", range(len(CASES)))
def test_random_patterns_in_every_array(case):
    strategy, flags = CASES[case]
    rng = np.random.default_rng(7000 + case)
    n = 500_003
    for mode in (0, 1, 2):
        hyp = dict(lr=float(10 ** rng.uniform(-6, 0)), beta1=float(rng.choice([0.0, 0.5, 0.9, 0.99, 0.999])),
                   beta2=float(rng.choice([0.0, 0.5, 0.95, 0.999, 0.9999])), eps=float(10 ** rng.uniform(-12, -1)),
                   weight_decay=float(rng.choice([0.0, 0.01, 0.1, 1.0])))
        t = int(rng.choice([1, 2, 3, 10, 1000, 10 ** 6]))
        st = dict(x_hi=_draw(rng, n, mode), x_lo=_draw(rng, n, mode) if strategy >= 1 else None, m=_draw(rng, n, mode),
                  v_hi=_draw(rng, n, mode), v_lo=_draw(rng, n, mode) if strategy == 2 else None)
        if mode == 2:
            st["v_hi"] &= 0x7FFF                                 # a valid (non-negative) second moment
        g = _draw(rng, n, mode)
        dev = {k: (W.from_bits(v, "cuda") if v is not None else None) for k, v in st.items()}
        B.adamw_step(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], W.from_bits(g, "cuda"), n,
                     B.make_hyper(**hyp, flags=flags), t, strategy)
        torch.cuda.synchronize()
        oracle.adamw_step(st["x_hi"], st["x_lo"], st["m"], st["v_hi"], st["v_lo"], g, step=t, strategy=strategy,
                          flags=flags, threads=oracle.max_threads(), **hyp)
        for k, v in st.items():
            if v is not None:
                assert_same_bits(W.bits(dev[k]), v, f"strategy {strategy} flags {flags} mode {mode} {hyp} step {t}: {k}")
    assert B.pipeline_fault() == 0


def _same_f32(got: np.ndarray, want: np.ndarray) -> np.ndarray:
    nan = lambda a: ((a & 0x7F800000) == 0x7F800000) & ((a & 0x007FFFFF) != 0)
    return (got == want) | (nan(got) & nan(want))


@pytest.mark.parametrize("flags", [0, 1])
def test_random_patterns_register_variant(flags):
    rng = np.random.default_rng(7100 + flags)
    n = 300_007
    for mode in (0, 1, 2):
        hyp = dict(lr=float(10 ** rng.uniform(-6, 0)), beta1=float(rng.choice([0.0, 0.9, 0.999])),
                   beta2=float(rng.choice([0.0, 0.95, 0.9999])), eps=float(10 ** rng.uniform(-12, -1)),
                   weight_decay=float(rng.choice([0.0, 0.1, 1.0])))
        t = int(rng.choice([1, 3, 1000, 10 ** 6]))
        st = {k: _draw(rng, n, mode) for k in ("x_hi", "x_lo", "m", "v_hi", "v_lo")}
        g = _draw(rng, n, mode)
        dev = {k: W.from_bits(v, "cuda") for k, v in st.items()}
        B.adamw_step(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], W.from_bits(g, "cuda"), n,
                     B.make_hyper(**hyp, flags=flags), t, B.PLUS_FP32_REGISTERS)
        torch.cuda.synchronize()
        oracle.adamw_fp32_register_step(st["x_hi"], st["x_lo"], st["m"], st["v_hi"], st["v_lo"], g, step=t, flags=flags, **hyp)
        for k, v in st.items():
            assert_same_bits(W.bits(dev[k]), v, f"register variant flags {flags} mode {mode} {hyp} step {t}: {k}")


@pytest.mark.parametrize("with_master", [True, False])
def test_random_patterns_fp32_comparators(with_master):
    rng = np.random.default_rng(7200 + int(with_master))
    n = 300_007
    for mode in (0, 1):
        hyp = dict(lr=float(10 ** rng.uniform(-6, 0)), beta1=float(rng.choice([0.0, 0.9, 0.999])),
                   beta2=float(rng.choice([0.0, 0.95, 0.9999])), eps=float(10 ** rng.uniform(-12, -1)),
                   weight_decay=float(rng.choice([0.0, 0.1, 1.0])))
        t = int(rng.choice([1, 3, 1000, 10 ** 6]))
        f32 = lambda: rng.integers(0, 1 << 32, n, dtype=np.uint32) if mode == 0 else \
            ((rng.integers(0, 2, n).astype(np.uint32) << 31) | (rng.integers(90, 150, n).astype(np.uint32) << 23)
             | rng.integers(0, 1 << 23, n).astype(np.uint32))
        theta, g = _draw(rng, n, mode), _draw(rng, n, mode)
        m, v = f32().view(np.float32).copy(), f32().view(np.float32).copy()
        master = f32().view(np.float32).copy() if with_master else None
        d_theta, d_g = W.from_bits(theta, "cuda"), W.from_bits(g, "cuda")
        d_m, d_v = torch.from_numpy(m.copy()).cuda(), torch.from_numpy(v.copy()).cuda()
        d_w = torch.from_numpy(master.copy()).cuda() if with_master else None
        B.adamw_step_fp32(d_theta, d_w, d_m, d_v, d_g, n, B.make_hyper(**hyp), t)
        torch.cuda.synchronize()
        oracle.adamw_fp32_step(theta, master, m, v, g, step=t, **hyp)
        assert_same_bits(W.bits(d_theta), theta, f"fp32 comparator master={with_master} mode {mode} {hyp} step {t}: theta")
        pairs = [("m", d_m, m), ("v", d_v, v)] + ([("master", d_w, master)] if with_master else [])
        for name, d, h in pairs:
            ok = _same_f32(d.cpu().numpy().view(np.uint32), h.view(np.uint32))
            assert ok.all(), (name, mode, hyp, t, int((~ok).sum()), int(np.flatnonzero(~ok)[0]))
