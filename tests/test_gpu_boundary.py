"""GPU checks of the boundary's contract: host threads making their first calls together, the EDQ
workspace and its ticket, the fault word carried in the record, overlap checks against a plan."""
import subprocess
import sys
import textwrap
from pathlib import Path

import numpy as np
import pytest
import torch

from gpu_util import EdqBuffers, assert_same_bits, edq_close, oracle_state, oracle_step
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import workloads as W

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent
KEYS = ("x_hi", "x_lo", "m", "v_hi", "v_lo")


def test_two_host_threads_make_their_first_calls_at_the_same_time():
    # A fresh process, so that the calls below really are the library's first on the device: two threads
    # leave a barrier together and each runs, on a stream of its own, a flat step (different precision
    # options, hence different kernels); one of them goes on to the static EDQ.  Each must match the
    # oracle; the library's one-time set-up (kernel attributes, device facts, scratch address) is what
    # the threads race on.
    script = textwrap.dedent('''
        import sys, threading, ctypes
        sys.path.insert(0, %r); sys.path.insert(0, %r)
        import numpy as np, torch
        import oracle
        from gpu_util import assert_same_bits, edq_close, oracle_state, oracle_step
        from paper_2405_03637_b200 import binding as B, workloads as W
        torch.cuda.init(); torch.cuda.set_device(0)
        hyp, n, KEYS = W.HYPERS, 300_007, ("x_hi", "x_lo", "m", "v_hi", "v_lo")
        jobs = []
        for k, strategy in enumerate((2, 1)):
            st = oracle_state(W.bits(W.flat_weights(n, 90 + k)), strategy)
            g = W.bits(W.flat_grads(n, 90 + k, 1))
            dev = {key: (W.from_bits(v, "cuda") if v is not None else None) for key, v in st.items()}
            ws = torch.zeros(B.workspace_bytes(), dtype=torch.uint8, device="cuda")
            out, out2 = (torch.zeros(64, dtype=torch.uint8, device="cuda") for _ in range(2))
            old = {key: (v.clone() if v is not None else None) for key, v in dev.items()}
            jobs.append(dict(strategy=strategy, st=st, g=g, dev=dev, gd=W.from_bits(g, "cuda"), ws=ws, out=out, out2=out2,
                             old=old, stream=torch.cuda.Stream(), err=None))
        torch.cuda.synchronize()
        gate = threading.Barrier(2)

        def work(j):
            try:
                torch.cuda.set_device(0)
                d, s = j["dev"], j["stream"]
                h = B.make_hyper(**hyp, edq_out=j["out"], workspace=j["ws"])
                gate.wait()
                B.adamw_step(d["x_hi"], d["x_lo"], d["m"], d["v_hi"], d["v_lo"], j["gd"], n, h, 1, j["strategy"], s)
                if j["strategy"] == 2:          # the static scratch is one per device: only one thread may use it at a time
                    s.synchronize()
                    B.edq_static(j["old"]["x_hi"], j["old"]["x_lo"], d["x_hi"], d["x_lo"], j["gd"], n, j["out2"], s)
                s.synchronize()
            except Exception as exc:            # noqa: BLE001
                j["err"] = exc

        threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
        [t.start() for t in threads]; [t.join() for t in threads]
        for j in jobs:
            assert j["err"] is None, j["err"]
            want = oracle_step(j["st"], j["g"], 1, j["strategy"], hyp)
            for key in KEYS:
                if j["st"][key] is not None:
                    assert_same_bits(W.bits(j["dev"][key]), j["st"][key], "thread step " + key)
            edq_close(B.read_edq(j["out"]), want)
        assert B.read_edq(jobs[0]["out2"])["n"] == n
        assert B.pipeline_fault() == 0
        print("threads ok")
    ''') % (str(ROOT), str(ROOT / "tests"))
    proc = subprocess.run([sys.executable, "-c", script], capture_output=True, text=True, timeout=600)
    assert proc.returncode == 0 and "threads ok" in proc.stdout, proc.stdout[-2000:] + proc.stderr[-4000:]


def test_workspace_is_left_ready_by_every_call_and_a_torn_ticket_is_repaired():
    # one clearing, then many steps with different grid sizes through the same workspace; then the ticket word
    # overwritten with a value that cannot be a count (all ones): the kernel resets it and still reduces correctly
    hyp = W.HYPERS
    e = EdqBuffers()
    for n, strategy in ((1_000_003, 2), (777, 0), (50_000, 1), (4096, 2), (1, 1), (300_001, 0)):
        st = oracle_state(W.bits(W.flat_weights(n, 61)), strategy)
        dev = {k: (W.from_bits(v, "cuda") if v is not None else None) for k, v in st.items()}
        for t in (1, 2):
            g = W.bits(W.flat_grads(n, 61, t))
            B.adamw_step(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], W.from_bits(g, "cuda"), n,
                         e.hyper(hyp), t, strategy)
            torch.cuda.synchronize()
            edq_close(e.read(), oracle_step(st, g, t, strategy, hyp))
            assert e.read()["n"] == n
    ticket = e.ws[B.workspace_bytes() - 64:]
    assert int(ticket.view(torch.int32)[0].item()) == 0              # back at zero after every call
    ticket.fill_(0xFF)
    n, strategy = 2_000_003, 2
    st = oracle_state(W.bits(W.flat_weights(n, 62)), strategy)
    dev = {k: W.from_bits(v, "cuda") for k, v in st.items()}
    g = W.bits(W.flat_grads(n, 62, 1))
    B.adamw_step(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], W.from_bits(g, "cuda"), n, e.hyper(hyp), 1, strategy)
    torch.cuda.synchronize()
    edq_close(e.read(), oracle_step(st, g, 1, strategy, hyp))
    assert int(ticket.view(torch.int32)[0].item()) == 0


def test_a_recorded_fault_shows_in_the_next_edq_record():
    # the give-up path of a bounded wait, exercised without any fault (a wait on a barrier nothing completes,
    # 5 ms): the code it leaves in the device's fault word is carried by the record of the next step that
    # reduces EDQ, so a caller that reads the record needs no extra synchronising call to learn of it
    n, strategy, hyp = 100_003, 2, W.HYPERS
    assert B.pipeline_fault() == 0
    B.wait_timeout_selftest(5)
    st = oracle_state(W.bits(W.flat_weights(n, 63)), strategy)
    dev = {k: W.from_bits(v, "cuda") for k, v in st.items()}
    g = W.bits(W.flat_grads(n, 63, 1))
    e = EdqBuffers()
    B.adamw_step(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], W.from_bits(g, "cuda"), n, e.hyper(hyp), 1, strategy)
    torch.cuda.synchronize()
    got = e.read()
    assert got["fault"] == 100
    edq_close(got, oracle_step(st, g, 1, strategy, hyp))             # the step itself was not disturbed
    for k in KEYS:
        assert_same_bits(W.bits(dev[k]), st[k], k)
    assert B.pipeline_fault() == 100 and B.pipeline_fault() == 0     # read and cleared
    B.adamw_step(dev["x_hi"], dev["x_lo"], dev["m"], dev["v_hi"], dev["v_lo"], W.from_bits(g, "cuda"), n, e.hyper(hyp), 2, strategy)
    torch.cuda.synchronize()
    assert e.read()["fault"] == 0


def test_record_and_workspace_may_not_overlap_a_plan():
    n = 40_000
    x = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for _ in range(5)]
    plan = B.plan_create([(x[0], x[1], x[2], x[3], None, x[4], n)])
    e = EdqBuffers()
    hyp = W.HYPERS
    B.adamw_step_multi(plan, e.hyper(hyp), 1, B.LIGHT)               # fine
    inside = x[2].view(torch.uint8)
    with pytest.raises(B.CollageError) as err:                       # the record inside the first moment
        B.adamw_step_multi(plan, B.make_hyper(**hyp, edq_out=inside[1024:1088], workspace=e.ws), 1, B.LIGHT)
    assert err.value.status == B.ERR_ALIAS
    big = torch.zeros(n * 2 + B.workspace_bytes(), dtype=torch.uint8, device="cuda")
    y = big[:n * 2].view(torch.bfloat16)
    plan2 = B.plan_create([(y, x[1], x[2], x[3], None, x[4], n)])
    with pytest.raises(B.CollageError) as err:                       # the workspace begins inside theta's last bytes
        B.adamw_step_multi(plan2, B.make_hyper(**hyp, edq_out=e.out, workspace=big[n * 2 - 16:]), 1, B.LIGHT)
    assert err.value.status == B.ERR_ALIAS
    with pytest.raises(B.CollageError) as err:                       # the record inside the workspace
        B.adamw_step_multi(plan, B.make_hyper(**hyp, edq_out=e.ws[256:320], workspace=e.ws), 1, B.LIGHT)
    assert err.value.status == B.ERR_ALIAS
    # a registered replica of theta counts as an array of the plan
    rep = torch.zeros(n * 2 + 64, dtype=torch.uint8, device="cuda")
    B.plan_set_replicas(plan, [[rep[:n * 2].view(torch.bfloat16)]])
    with pytest.raises(B.CollageError) as err:
        B.adamw_step_multi(plan, B.make_hyper(**hyp, edq_out=rep[1024:1088], workspace=e.ws), 1, B.LIGHT)
    assert err.value.status == B.ERR_ALIAS
    B.plan_set_replicas(plan, [])
    B.adamw_step_multi(plan, B.make_hyper(**hyp, edq_out=rep[1024:1088], workspace=e.ws), 1, B.LIGHT)    # no longer a replica
    per = torch.zeros(B.EDQ_RECORD_BYTES, dtype=torch.uint8, device="cuda")
    cws = torch.empty(B.plan_workspace_bytes(plan), dtype=torch.uint8, device="cuda")
    B.adamw_step_multi_per_tensor(plan, B.make_hyper(**hyp), 2, B.LIGHT, per, 1, cws)
    with pytest.raises(B.CollageError) as err:                       # per-tensor records inside the gradient
        B.adamw_step_multi_per_tensor(plan, B.make_hyper(**hyp), 2, B.LIGHT, x[4].view(torch.uint8)[:B.EDQ_RECORD_BYTES], 1, cws)
    assert err.value.status == B.ERR_ALIAS
    torch.cuda.synchronize()
    B.plan_destroy(plan)
    B.plan_destroy(plan2)


def test_empty_inputs_still_write_their_record():
    # n == 0 and an empty plan launch no step kernel; the record must still say "nothing": zeros, not stale data
    e = EdqBuffers()
    e.out.fill_(0xAB)
    z = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    B.adamw_step(z, z.clone(), z.clone(), z.clone(), z.clone(), z.clone(), 0, e.hyper(W.HYPERS), 1, B.PLUS)
    torch.cuda.synchronize()
    assert e.read() == dict(dot=0.0, sumsq=0.0, edq=0.0, n=0, lost=0, fault=0)
    e.out.fill_(0xAB)
    plan = B.plan_create([(z, z.clone(), z.clone(), z.clone(), z.clone(), z.clone(), 0)])
    B.adamw_step_multi(plan, e.hyper(W.HYPERS), 1, B.PLUS)
    torch.cuda.synchronize()
    assert e.read() == dict(dot=0.0, sumsq=0.0, edq=0.0, n=0, lost=0, fault=0)
    B.plan_destroy(plan)


def test_build_flavor_of_the_library_under_test_is_the_product():
    assert B.build_flavor() == "product"
