"""Asynchrony of the step: calls only enqueue work on the caller's stream, keep nothing on the host that
a later call could disturb, and steps on different streams do not interfere."""
import numpy as np
import pytest
import torch

from gpu_util import EdqBuffers, assert_same_bits, edq_close, oracle_state, oracle_step
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import workloads as W

pytestmark = pytest.mark.gpu
KEYS = ("x_hi", "x_lo", "m", "v_hi", "v_lo")


def _check(dev, st, what):
    for k in KEYS:
        if st[k] is not None:
            assert_same_bits(W.bits(dev[k]), st[k], f"{what} {k}")


@pytest.mark.parametrize("strategy", [0, 2])
def test_steps_queued_back_to_back_without_synchronising(strategy):
    # five steps with different scalars and gradients enqueued on a side stream with no host synchronisation in
    # between: every call must have captured its scalars by value; the result is the oracle's fifth state
    n, hyp = 1_000_003, W.HYPERS
    st = oracle_state(W.bits(W.flat_weights(n, 71)), strategy)
    side = torch.cuda.Stream()
    grads = [W.bits(W.flat_grads(n, 71, t)) for t in range(1, 6)]
    e = EdqBuffers()
    torch.cuda.synchronize()                                     # the buffers above were made on the default stream
    with torch.cuda.stream(side):
        dev = {k: (W.from_bits(v, "cuda") if v is not None else None) for k, v in st.items()}
        gdev = [W.from_bits(g, "cuda") for g in grads]
        for t in range(1, 6):
            h = e.hyper(dict(hyp, lr=hyp["lr"] * t))            # a different struct, freed right after the call
            B.adamw_step(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], gdev[t - 1], n, h, t, strategy, side)
            del h
    side.synchronize()
    for t in range(1, 6):
        want = oracle_step(st, grads[t - 1], t, strategy, dict(hyp, lr=hyp["lr"] * t))
    _check(dev, st, f"queued steps, strategy {strategy}")
    edq_close(e.read(), want)                                    # the record holds the last step's sums
    assert B.pipeline_fault() == 0


def test_two_streams_step_different_tensors_at_the_same_time():
    # a long step on one stream and many short ones on another, each with its own EDQ record and workspace
    hyp = W.HYPERS
    big_n, small_n = 40_000_003, 50_001
    big = oracle_state(W.bits(W.flat_weights(big_n, 72)), 2)
    small = oracle_state(W.bits(W.flat_weights(small_n, 73)), 1)
    gb, gs = W.bits(W.flat_grads(big_n, 72, 1)), [W.bits(W.flat_grads(small_n, 73, t)) for t in range(1, 21)]
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    e1, e2 = EdqBuffers(), EdqBuffers()
    dbig = {k: W.from_bits(v, "cuda") for k, v in big.items()}
    dsmall = {k: (W.from_bits(v, "cuda") if v is not None else None) for k, v in small.items()}
    dgb, dgs = W.from_bits(gb, "cuda"), [W.from_bits(g, "cuda") for g in gs]
    torch.cuda.synchronize()
    for rep in range(3):                                          # three long steps, twenty short ones beside them
        B.adamw_step(dbig["x_hi"], dbig["x_lo"], dbig["m"], dbig["v_hi"], dbig["v_lo"], dgb, big_n, e1.hyper(hyp), rep + 1, B.PLUS, s1)
        for t in range(1, 21):
            if (t - 1) * 3 // 20 == rep:
                B.adamw_step(dsmall["x_hi"], dsmall["x_lo"], dsmall["m"], dsmall["v_hi"], None, dgs[t - 1], small_n,
                             e2.hyper(hyp), t, B.LIGHT, s2)
    torch.cuda.synchronize()
    for rep in range(3):
        want_big = oracle_step(big, gb, rep + 1, 2, hyp)
    for t in range(1, 21):
        want_small = oracle_step(small, gs[t - 1], t, 1, hyp)
    _check(dbig, big, "long step")
    _check(dsmall, small, "short steps")
    edq_close(e1.read(), want_big)
    edq_close(e2.read(), want_small)
    assert B.pipeline_fault() == 0
