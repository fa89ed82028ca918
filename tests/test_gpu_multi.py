"""GPU parity of the one-launch multi-tensor step (chunk table) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import EdqBuffers, Guarded, assert_same_bits, edq_close, oracle_state, oracle_step
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import workloads as W

pytestmark = pytest.mark.gpu
KEYS = ("x_hi", "x_lo", "m", "v_hi", "v_lo")


def _build(shapes, strategy, seed, misalign_of=lambda i: 0):
    """Per-tensor oracle state + guarded device copies + plan."""
    host, dev, grads = [], [], []
    for i, (_, n) in enumerate(shapes):
        theta = W.bits(W.flat_weights(n, seed * 1000 + i)) if n else np.zeros(0, np.uint16)
        st = oracle_state(theta, strategy)
        host.append(st)
        dev.append({k: (Guarded(v, misalign_of(i)) if v is not None else None) for k, v in st.items()})
        grads.append(Guarded(np.zeros(n, np.uint16), misalign_of(i)))
    rows = [(d["x_hi"].t, d["x_lo"].t if d["x_lo"] else None, d["m"].t, d["v_hi"].t, d["v_lo"].t if d["v_lo"] else None,
             g.t, s[1]) for d, g, s in zip(dev, grads, shapes)]
    return host, dev, grads, rows


def _set_grads(shapes, grads, seed, t):
    out = []
    for i, (_, n) in enumerate(shapes):
        g = W.bits(W.flat_grads(n, seed * 1000 + i, t)) if n else np.zeros(0, np.uint16)
        if n:
            grads[i].t.copy_(W.from_bits(g, "cuda"))
        out.append(g)
    return out


def _oracle_multi(host, gbits, t, strategy, hyp):
    tot = dict(dot=0.0, sumsq=0.0, lost=0)
    for st, g in zip(host, gbits):
        if g.size == 0:
            continue
        s = oracle_step(st, g, t, strategy, hyp)
        tot["dot"] += s["dot"]; tot["sumsq"] += s["sumsq"]; tot["lost"] += s["lost"]
    tot["edq"] = tot["dot"] / np.sqrt(tot["sumsq"]) if tot["sumsq"] > 0 else 0.0
    return tot


@pytest.mark.parametrize("strategy", [0, 1, 2])
@pytest.mark.parametrize("chunk", [0, 2048, 65536])
def test_ragged_tensor_set(strategy, chunk, step_kernel):
    shapes = W.ragged_shapes()
    hyp = W.HYPERS
    host, dev, grads, rows = _build(shapes, strategy, seed=3, misalign_of=lambda i: (0, 0, 1, 0, 0, 3)[i % 6])
    plan = B.plan_create(rows, chunk)
    assert B.plan_num_elements(plan) == sum(n for _, n in shapes)
    ce = chunk or 24576
    assert B.plan_num_chunks(plan) == sum(-(-n // ce) for _, n in shapes)
    e = EdqBuffers()
    for t in (1, 2, 3):
        gbits = _set_grads(shapes, grads, 3, t)
        B.adamw_step_multi(plan, e.hyper(hyp), t, strategy)
        torch.cuda.synchronize()
        want = _oracle_multi(host, gbits, t, strategy, hyp)
        for i, (st, d) in enumerate(zip(host, dev)):
            for k in KEYS:
                if st[k] is not None:
                    assert_same_bits(d[k].bits(), st[k], f"tensor {i} {k} step {t}")
                    assert d[k].guards_intact()
        got = e.read()
        edq_close(got, want)
        assert got["n"] == sum(n for _, n in shapes)
    B.plan_destroy(plan)


def test_gpt2_small_shaped_set_collage_light():
    # 148 tensors, 124,439,808 parameters: whole-array parity for the first steps
    shapes = W.gpt2_small_shapes()
    strategy, hyp = 1, W.HYPERS
    host, dev, grads, rows = _build(shapes, strategy, seed=1)
    plan = B.plan_create(rows)
    e = EdqBuffers()
    for t in (1, 2):
        gbits = _set_grads(shapes, grads, 1, t)
        B.adamw_step_multi(plan, e.hyper(hyp), t, strategy)
        torch.cuda.synchronize()
        want = _oracle_multi(host, gbits, t, strategy, hyp)
        for i, (st, d) in enumerate(zip(host, dev)):
            for k in ("x_hi", "x_lo", "m", "v_hi"):
                assert_same_bits(d[k].bits(), st[k], f"{shapes[i][0]} {k} step {t}")
        edq_close(e.read(), want)
    assert all(d[k].guards_intact() for d in dev for k in ("x_hi", "x_lo", "m", "v_hi"))
    B.plan_destroy(plan)


def test_plan_strategy_needs_its_components():
    n = 4096
    z = lambda: torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    keep = [z() for _ in range(4)]
    plan = B.plan_create([(keep[0], None, keep[1], keep[2], None, keep[3], n)])
    h = B.make_hyper(**W.HYPERS)
    B.adamw_step_multi(plan, h, 1, B.BF16)
    for s in (B.LIGHT, B.PLUS):
        with pytest.raises(B.CollageError) as err:
            B.adamw_step_multi(plan, h, 1, s)
        assert err.value.status == B.ERR_NULL
    torch.cuda.synchronize()
    B.plan_destroy(plan)
    empty = B.plan_create([])
    e = EdqBuffers()
    B.adamw_step_multi(empty, e.hyper(W.HYPERS), 1, B.BF16)
    torch.cuda.synchronize()
    assert e.read()["edq"] == 0.0 and e.read()["n"] == 0
    B.plan_destroy(empty)


@pytest.mark.parametrize("strategy", [0, 1, 2])
@pytest.mark.parametrize("chunk", [0, 2048])
def test_per_tensor_edq_matches_oracle_tensor_by_tensor(strategy, chunk, step_kernel):
    shapes = W.ragged_shapes() + [("big", 700_001)]
    hyp = W.HYPERS
    host, dev, grads, rows = _build(shapes, strategy, seed=7, misalign_of=lambda i: (0, 1, 0)[i % 3])
    plan = B.plan_create(rows, chunk)
    num = len(shapes)
    per = torch.zeros(num * B.EDQ_RECORD_BYTES, dtype=torch.uint8, device="cuda")
    cws = torch.empty(B.plan_workspace_bytes(plan), dtype=torch.uint8, device="cuda")
    assert B.plan_workspace_bytes(plan) >= 32 * B.plan_num_chunks(plan)
    total = torch.zeros(64, dtype=torch.uint8, device="cuda")
    for t in (1, 2, 3):
        gbits = _set_grads(shapes, grads, 7, t)
        h = B.make_hyper(**hyp, edq_out=total)
        B.adamw_step_multi_per_tensor(plan, h, t, strategy, per, num, cws)
        torch.cuda.synchronize()
        recs = B.read_edq_array(per, num)
        tot = dict(dot=0.0, sumsq=0.0, lost=0)
        for i, (st, g) in enumerate(zip(host, gbits)):
            if g.size == 0:
                assert recs[i] == dict(dot=0.0, sumsq=0.0, edq=0.0, n=0, lost=0, fault=0)
                continue
            want = oracle_step(st, g, t, strategy, hyp, threads=1)
            edq_close(recs[i], want)
            assert recs[i]["n"] == g.size
            for k in KEYS:
                if st[k] is not None:
                    assert_same_bits(dev[i][k].bits(), st[k], f"tensor {i} {k} step {t}")
                    assert dev[i][k].guards_intact()
            tot["dot"] += want["dot"]; tot["sumsq"] += want["sumsq"]; tot["lost"] += want["lost"]
        tot["edq"] = tot["dot"] / np.sqrt(tot["sumsq"])
        got = B.read_edq(total)
        edq_close(got, tot)
        assert got["n"] == sum(n for _, n in shapes)
    assert B.pipeline_fault() == 0
    # argument checks
    with pytest.raises(B.CollageError) as err:
        B.adamw_step_multi_per_tensor(plan, B.make_hyper(**hyp), 1, strategy, per, num - 1, cws)
    assert err.value.status == B.ERR_ARG
    with pytest.raises(B.CollageError) as err:
        B.adamw_step_multi_per_tensor(plan, B.make_hyper(**hyp), 1, strategy, per, num, cws[:64])
    assert err.value.status == B.ERR_WORKSPACE
    B.plan_destroy(plan)


@pytest.mark.parametrize("strategy", [0, 2])
def test_theta_replicas_are_written_by_the_step_itself(strategy, step_kernel):
    # sharded optimizer state needs theta everywhere: the step writes it to registered replicas (here two more
    # buffers on this GPU; on several GPUs they would be peers' memory) - ragged, unaligned and empty tensors included
    shapes = W.ragged_shapes() + [("big", 500_003)]
    hyp = W.HYPERS
    mis = lambda i: (0, 0, 1, 0, 3)[i % 5]
    host, dev, grads, rows = _build(shapes, strategy, seed=9, misalign_of=mis)
    plan = B.plan_create(rows)
    reps = [[Guarded(np.full(n, 0x7FC1, np.uint16), mis(i)) for i, (_, n) in enumerate(shapes)] for _ in range(2)]
    B.plan_set_replicas(plan, [[g.t if g.n else None for g in rep] for rep in reps])
    e = EdqBuffers()
    for t in (1, 2):
        gbits = _set_grads(shapes, grads, 9, t)
        B.adamw_step_multi(plan, e.hyper(hyp), t, strategy)
        torch.cuda.synchronize()
        want = _oracle_multi(host, gbits, t, strategy, hyp)
        for i, (st, d) in enumerate(zip(host, dev)):
            assert_same_bits(d["x_hi"].bits(), st["x_hi"], f"tensor {i} theta step {t}")
            for r, rep in enumerate(reps):
                assert_same_bits(rep[i].bits(), st["x_hi"], f"replica {r} tensor {i} step {t}")
                assert rep[i].guards_intact()
        edq_close(e.read(), want)
    # replicas must not overlap the plan's arrays, and must sit like their tensor modulo 16 bytes
    with pytest.raises(B.CollageError) as err:
        B.plan_set_replicas(plan, [[d["m"].t if d["m"].n else None for d in dev]])
    assert err.value.status == B.ERR_ALIAS
    bad = [[g.t if g.n else None for g in reps[0]]]
    big = len(shapes) - 1
    bad[0][big] = reps[0][big].raw[reps[0][big].lo + 1:].view(torch.bfloat16)
    with pytest.raises(B.CollageError) as err:
        B.plan_set_replicas(plan, bad)
    assert err.value.status == B.ERR_ARG
    B.plan_set_replicas(plan, [])                      # detach
    gbits = _set_grads(shapes, grads, 9, 3)
    before = [rep[-1].bits() for rep in reps]
    B.adamw_step_multi(plan, e.hyper(hyp), 3, strategy)
    torch.cuda.synchronize()
    assert all(np.array_equal(b, rep[-1].bits()) for b, rep in zip(before, reps))
    assert B.pipeline_fault() == 0
    B.plan_destroy(plan)


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_step_of_emulated_ranks_gathers_theta_everywhere(world, step_kernel):
    # ZeRO-1-style ownership on one device: every "rank" keeps its own full copy of theta (what its forward
    # pass would read) and the optimizer state of its slice only; its step writes the new theta of the slice
    # into every rank's copy.  The ranks' kernels do not wait on one another, so running them one after the
    # other is the same computation.  Afterwards every copy equals the oracle's theta of the unsharded step,
    # and the summed EDQ records equal its global EDQ.
    from paper_2405_03637_b200 import sharding as S
    shapes = [("a", 70_001), ("b", 4096), ("c", 33_333), ("d", 8), ("e", 250_000)]
    sizes = [n for _, n in shapes]
    strategy, hyp = 2, W.HYPERS
    theta = [W.bits(W.flat_weights(n, 300 + i)) for i, n in enumerate(sizes)]
    copies = [[W.from_bits(t, "cuda") for t in theta] for _ in range(world)]          # theta as each rank sees it
    full = [oracle_state(t, strategy) for t in theta]
    parts = S.partition(sizes, world)
    plans, states, grads_dev, edqs = [], [], [], []
    for r in range(world):
        z = lambda i: torch.zeros(sizes[i], dtype=torch.bfloat16, device="cuda")
        # state tensors of full length for simplicity; the rank touches its ranges only
        rows = [(copies[r][i], z(i), z(i), z(i), z(i), torch.zeros(sizes[i], dtype=torch.bfloat16, device="cuda"), sizes[i])
                for i in range(len(sizes))]
        mine = S.slice_rows(rows, parts[r])
        plan = B.plan_create(mine)
        peers = [copies[q] for q in range(world) if q != r]
        B.plan_set_replicas(plan, S.replica_rows(peers, parts[r]))
        plans.append(plan)
        states.append(rows)
        edqs.append(EdqBuffers())
    for t in (1, 2, 3):
        gbits = [W.bits(W.flat_grads(n, 400 + i, t)) for i, n in enumerate(sizes)]
        for r in range(world):
            for i in range(len(sizes)):
                states[r][i][5].copy_(W.from_bits(gbits[i], "cuda"))
        for r in range(world):
            B.adamw_step_multi(plans[r], edqs[r].hyper(hyp), t, strategy)
        torch.cuda.synchronize()
        sums = np.zeros(4)                                  # dot, sumsq, (unused), lost of the unsharded step
        for st, g in zip(full, gbits):
            w = oracle_step(st, g, t, strategy, hyp)
            sums += np.array([w["dot"], w["sumsq"], 0.0, w["lost"]])
        for r in range(world):
            for i in range(len(sizes)):
                assert_same_bits(W.bits(copies[r][i]), full[i]["x_hi"], f"world {world} step {t}: theta copy of rank {r}, tensor {i}")
        recs = [e.read() for e in edqs]
        got = S.allreduce_edq(torch.tensor([sum(x["dot"] for x in recs), sum(x["sumsq"] for x in recs),
                                            float(sum(x["lost"] for x in recs))], dtype=torch.float64))
        assert sum(x["n"] for x in recs) == sum(sizes)
        assert abs(got["dot"] - sums[0]) <= 1e-5 * abs(sums[0]) and abs(got["sumsq"] - sums[1]) <= 1e-5 * sums[1]
        assert got["lost"] == int(sums[3])
    for p in plans:
        B.plan_destroy(p)
    assert B.pipeline_fault() == 0
