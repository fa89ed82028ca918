"""Asynchrony of the step: calls only enqueue work on the caller's stream, keep nothing on the host that
a later call could disturb, and steps on different streams do not interfere."""
import numpy as np
import pytest
import torch

from gpu_util import EdqBuffers, assert_same_bits, edq_close, oracle_state, oracle_step
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import workloads as W

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("step_kernel")]
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


@pytest.mark.parametrize("api", ["flat", "multi"])
def test_steps_recorded_into_a_cuda_graph_replay_bit_identically(api):
    # the step only launches kernels on the given stream (no allocation, no synchronisation, no host round trip),
    # so three consecutive steps can be recorded once and replayed: same bits as the oracle, twice
    n, hyp, strategy = 300_011, W.HYPERS, 2
    st0 = oracle_state(W.bits(W.flat_weights(n, 74)), strategy)
    grads = [W.bits(W.flat_grads(n, 74, t)) for t in (1, 2, 3)]
    dev = {k: W.from_bits(v, "cuda") for k, v in st0.items()}
    gdev = [W.from_bits(g, "cuda") for g in grads]
    e = EdqBuffers()
    plans = [B.plan_create([(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], g, n)]) for g in gdev] if api == "multi" else None

    def enqueue(stream):
        for t in (1, 2, 3):
            if api == "multi":
                B.adamw_step_multi(plans[t - 1], e.hyper(hyp), t, strategy, stream)
            else:
                B.adamw_step(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], gdev[t - 1], n, e.hyper(hyp), t, strategy, stream)

    def restore():
        for k, v in st0.items():
            dev[k].copy_(W.from_bits(v, "cuda"))
        torch.cuda.synchronize()

    side = torch.cuda.Stream()
    enqueue(side)                                   # first use: per-device kernel attributes are set outside the recording
    side.synchronize()
    restore()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        enqueue(side)
    want = {k: v.copy() for k, v in st0.items()}
    for t in (1, 2, 3):
        sums = oracle_step(want, grads[t - 1], t, strategy, hyp)
    for rep in range(2):
        restore()
        graph.replay()
        torch.cuda.synchronize()
        _check(dev, want, f"graph replay {rep} ({api})")
        edq_close(e.read(), sums)
    if plans:
        for p in plans:
            B.plan_destroy(p)
    assert B.pipeline_fault() == 0


def test_fp32_comparator_step_recorded_into_a_cuda_graph():
    import oracle
    from conftest import bits_to_f64
    n, hyp = 200_003, W.HYPERS
    theta0 = W.bits(W.flat_weights(n, 75))
    grads = [W.bits(W.flat_grads(n, 75, t)) for t in (1, 2)]
    d_theta, d_master = W.from_bits(theta0, "cuda"), torch.from_numpy(bits_to_f64(theta0).astype(np.float32)).cuda()
    d_m, d_v = torch.zeros(n, dtype=torch.float32, device="cuda"), torch.zeros(n, dtype=torch.float32, device="cuda")
    gdev = [W.from_bits(g, "cuda") for g in grads]
    e = EdqBuffers()

    def enqueue(stream):
        for t in (1, 2):
            B.adamw_step_fp32(d_theta, d_master, d_m, d_v, gdev[t - 1], n, e.hyper(hyp), t, stream)

    def restore():
        d_theta.copy_(W.from_bits(theta0, "cuda"))
        d_master.copy_(torch.from_numpy(bits_to_f64(theta0).astype(np.float32)).cuda())
        d_m.zero_()
        d_v.zero_()
        torch.cuda.synchronize()

    side = torch.cuda.Stream()
    enqueue(side)
    side.synchronize()
    restore()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        enqueue(side)
    theta, master = theta0.copy(), bits_to_f64(theta0).astype(np.float32)
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    for t in (1, 2):
        want = oracle.adamw_fp32_step(theta, master, m, v, grads[t - 1], step=t, **hyp)
    restore()
    graph.replay()
    torch.cuda.synchronize()
    assert np.array_equal(W.bits(d_theta), theta)
    assert np.array_equal(d_master.cpu().numpy().view(np.uint32), master.view(np.uint32))
    assert np.array_equal(d_v.cpu().numpy().view(np.uint32), v.view(np.uint32))
    edq_close(e.read(), want)
    assert B.pipeline_fault() == 0


def test_a_wait_that_runs_out_is_reported_and_the_device_stays_usable():
    # the give-up path of the pipeline's bounded barrier waits, made on purpose with a barrier that nothing
    # completes and a 20 ms bound: the kernel returns normally, the code is reported once, work goes on
    assert B.pipeline_fault() == 0
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    B.wait_timeout_selftest(20)
    t1.record()
    torch.cuda.synchronize()
    assert 5.0 < t0.elapsed_time(t1) < 500.0          # bounded: tens of milliseconds, not seconds
    assert B.pipeline_fault() == 100
    assert B.pipeline_fault() == 0                    # reading clears the word
    with pytest.raises(B.CollageError):
        B.wait_timeout_selftest(0)
    with pytest.raises(B.CollageError):
        B.wait_timeout_selftest(5000)
    n, hyp = 20_011, W.HYPERS
    st = oracle_state(W.bits(W.flat_weights(n, 76)), 2)
    dev = {k: W.from_bits(v, "cuda") for k, v in st.items()}
    g = W.bits(W.flat_grads(n, 76, 1))
    e = EdqBuffers()
    B.adamw_step(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], W.from_bits(g, "cuda"), n, e.hyper(hyp), 1, 2)
    torch.cuda.synchronize()
    want = oracle_step(st, g, 1, 2, hyp)
    _check(dev, st, "step after a reported timeout")
    edq_close(e.read(), want)
    assert B.pipeline_fault() == 0
