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

pytestmark = pytest.mark.gpu
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
