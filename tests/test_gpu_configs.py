"""GPU parity on the benchmark's own configurations, including the full-size LLaMA-7B-shaped launch.

Full-size arrays are far beyond what the oracle can step in seconds, so the large cases compare
sampled windows (every element of a window bit for bit; elements are independent, so a window is a
complete check of the elements in it) and the small cases compare whole arrays.
"""
import numpy as np
import pytest
import torch

import bench
import oracle
from gpu_util import EdqBuffers, assert_same_bits, edq_close, oracle_step
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import workloads as W

pytestmark = pytest.mark.gpu
KEYS = ("x_hi", "x_lo", "m", "v_hi", "v_lo")


def _windows(n, rng, width, count):
    """Sample windows of one tensor: its first and last `width` elements and `count` random ones."""
    if n <= 2 * width:
        return [(0, n)]
    wins = [(0, width), (n - width, n)]
    for _ in range(count):
        lo = int(rng.integers(0, n - width))
        wins.append((lo, lo + width))
    return wins


def _gather(t, wins):
    return W.bits(torch.cat([t[lo:hi] for lo, hi in wins]))          # one device-to-host copy per call


def test_llama7b_full_size_launch_sampled_parity():
    # the exact launch bench.py times: 291 tensors, 6,738,415,616 parameters, Collage-plus with EDQ
    dev = torch.device("cuda")
    arrays, rows, n = bench.build_llama7b_state(torch, W, dev, seed=3, layers=32)
    assert n == 6_738_415_616 and len(rows) == 291
    plan = B.plan_create(rows)
    assert B.plan_num_elements(plan) == n
    e = EdqBuffers()
    rng = np.random.default_rng(0)
    samples = []                                   # (row index, windows, oracle state dict, gradient bits)
    for i, row in enumerate(rows):
        wins = _windows(row[6], rng, 98_304, 11)            # four 24,576-element chunks per window
        st = {k: _gather(row[j], wins) for j, k in enumerate(KEYS)}
        samples.append((i, wins, st, _gather(row[5], wins)))
    total = sum(sum(hi - lo for lo, hi in wins) for _, wins, _, _ in samples)
    assert total >= 2 ** 28
    hyp = W.HYPERS
    for t in (1, 2):
        # step 1 as bench.py launches it (at this size: the two-stage pipeline with 8192-element tiles), step 2
        # with the three-stage pipeline pinned, so that both are checked at full size
        B.adamw_step_multi(plan, e.hyper(hyp, flags=0 if t == 1 else B.FLAG_PIPELINE_KERNEL), t, B.PLUS)
        torch.cuda.synchronize()
        for i, wins, st, g in samples:
            oracle_step(st, g, t, 2, hyp)
            for j, k in enumerate(KEYS):
                assert_same_bits(_gather(rows[i][j], wins), st[k], f"step {t} tensor {i} {k}")
        got = e.read()
        assert got["n"] == n and 0 <= got["lost"] <= n
        assert np.isfinite(got["edq"]) and got["edq"] > 0 and got["sumsq"] > 0
        assert abs(got["edq"]) <= np.sqrt(got["sumsq"]) * 1.5          # projection of a nearby vector
    # Third step through the per-tensor entry point, still the full 291-tensor launch: the records of all 65
    # RMSNorm vectors and of one 4096 x 4096 projection against whole-tensor oracle sums, and the
    # records of all tensors against the global record of the same call.
    names = [name for name, _ in W.llama7b_shapes(32)]
    chosen = [i for i, name in enumerate(names) if name.endswith("norm")] + [names.index("l17.q")]
    assert len(chosen) == 66
    before = {i: ({k: W.bits(rows[i][j]) for j, k in enumerate(KEYS)}, W.bits(rows[i][5])) for i in chosen}
    per = torch.zeros(len(rows) * B.EDQ_RECORD_BYTES, dtype=torch.uint8, device=dev)
    cws = torch.empty(B.plan_workspace_bytes(plan), dtype=torch.uint8, device=dev)
    total = torch.zeros(64, dtype=torch.uint8, device=dev)
    B.adamw_step_multi_per_tensor(plan, B.make_hyper(**hyp, edq_out=total), 3, B.PLUS, per, len(rows), cws)
    torch.cuda.synchronize()
    recs = B.read_edq_array(per, len(rows))
    for i in chosen:
        st, g = before[i]
        want = oracle_step(st, g, 3, 2, hyp)
        edq_close(recs[i], want)
        assert recs[i]["n"] == rows[i][6]
        for j, k in enumerate(KEYS):
            assert_same_bits(W.bits(rows[i][j]), st[k], f"step 3 tensor {names[i]} {k}")
    whole = B.read_edq(total)
    summed = B.edq_combine(recs)
    assert whole["n"] == summed["n"] == n and whole["lost"] == summed["lost"]
    for k in ("dot", "sumsq", "edq"):
        assert abs(whole[k] - summed[k]) <= 1e-12 * abs(summed[k])
    # steps 1 and 2 went through the other entry point: its global record has the same shape
    assert abs(whole["edq"] / np.sqrt(whole["sumsq"]) - got["edq"] / np.sqrt(got["sumsq"])) < 0.05
    assert B.pipeline_fault() == 0
    B.plan_destroy(plan)
    del arrays, rows, per, cws
    torch.cuda.empty_cache()


def test_llama7b_layout_four_layers_whole_arrays_and_edq():
    # the same layout with four transformer layers (1.07 G parameters, 39 tensors): every element and the global EDQ
    dev = torch.device("cuda")
    arrays, rows, n = bench.build_llama7b_state(torch, W, dev, seed=3, layers=4)
    assert n == 262_148_096 + 4 * 202_383_360
    plan = B.plan_create(rows)
    e = EdqBuffers()
    st = {k: W.bits(arrays[k]) for k in KEYS}
    g = W.bits(arrays["grad"])
    B.adamw_step_multi(plan, e.hyper(W.HYPERS), 1, B.PLUS)
    torch.cuda.synchronize()
    want = oracle_step(st, g, 1, 2, W.HYPERS)
    for k in KEYS:
        assert_same_bits(W.bits(arrays[k]), st[k], k)
    got = e.read()
    edq_close(got, want)
    assert got["n"] == n
    B.plan_destroy(plan)
    del arrays, rows
    torch.cuda.empty_cache()


def test_gpt2_small_hundred_steps_collage_light_sampled():
    # config 1: 148 tensors, 124,439,808 parameters, multi-tensor Collage-light, 100 steps with fresh gradients
    dev = torch.device("cuda")
    shapes = W.gpt2_small_shapes()
    rng = np.random.default_rng(1)
    tensors, rows, samples = [], [], []
    for i, (_, n) in enumerate(shapes):
        x = W.flat_weights(n, 1000 + i, dev)
        d = dict(x_hi=x, x_lo=torch.zeros_like(x), m=torch.zeros_like(x), v_hi=torch.zeros_like(x),
                 grad=torch.zeros_like(x))
        tensors.append(d)
        rows.append((d["x_hi"], d["x_lo"], d["m"], d["v_hi"], None, d["grad"], n))
        wins = _windows(n, rng, 1024, 3)
        st = {k: (_gather(d[k], wins) if k in d else None) for k in KEYS}
        samples.append((wins, st))
    plan = B.plan_create(rows)
    e = EdqBuffers()
    hyp = W.HYPERS
    edq_hist = []
    for t in range(1, 101):
        for i, (_, n) in enumerate(shapes):
            tensors[i]["grad"].copy_(W.normal_bf16(n, 1e-3, 2000 * 1000 + t * 1000 + i, dev))
        B.adamw_step_multi(plan, e.hyper(hyp), t, B.LIGHT)
        for i, (wins, st) in enumerate(samples):
            oracle_step(st, _gather(tensors[i]["grad"], wins), t, 1, hyp, threads=1)
        edq_hist.append(e.read()["edq"])
        for i, (wins, st) in enumerate(samples):                      # every sampled window at every step
            for k in ("x_hi", "x_lo", "m", "v_hi"):
                assert_same_bits(_gather(tensors[i][k], wins), st[k], f"step {t} {shapes[i][0]} {k}")
    assert all(np.isfinite(edq_hist)) and min(edq_hist) > 0
    assert B.pipeline_fault() == 0
    B.plan_destroy(plan)


def test_stress_set_collage_plus_against_plain_bf16():
    # config 2: 64 Mi parameters, theta = +-U(0.5, 4), log-uniform gradients, lr 1e-5, 1000 steps: whole arrays
    # for the first 8 steps, then a fixed 2 Mi slice to the end; Collage-plus keeps what plain bfloat16 loses,
    # and stays close to AdamW in double precision on the same gradients
    dev = torch.device("cuda")
    n, hyp, steps = 1 << 26, W.HYPERS_STRESS, 1000
    lo, hi = 12_345_672, 12_345_672 + (1 << 21)
    theta = W.stress_weights(n, 2, dev)
    state, host, edq = {}, {}, {}
    for s in (2, 0):
        z = lambda: torch.zeros_like(theta)
        state[s] = dict(x_hi=theta.clone(), x_lo=z() if s else None, m=z(), v_hi=z(), v_lo=z() if s == 2 else None)
        host[s] = {k: (W.bits(v) if v is not None else None) for k, v in state[s].items()}
        edq[s] = []
    to_f64 = lambda b: (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    th64 = to_f64(host[0]["x_hi"][lo:hi])
    theta0 = th64.copy()
    m64, v64 = np.zeros_like(th64), np.zeros_like(th64)
    e = EdqBuffers()
    for t in range(1, steps + 1):
        g = W.stress_grads(n, 2, t, dev)
        whole = t <= 8
        gs = W.bits(W.stress_grads(hi - lo, 2, t, "cpu", offset=lo))
        gb = W.bits(g) if whole else gs
        if t == 9:                        # from here on the oracle follows the slice only
            host = {s: {k: (v[lo:hi].copy() if v is not None else None) for k, v in host[s].items()} for s in host}
        if t in (1, 9, 100, steps):
            assert np.array_equal(gs, W.bits(g[lo:hi]))              # the slice generator reproduces the full one
        oracle.adamw_fp64(th64, m64, v64, to_f64(gs), step=t, **hyp)
        for s in (2, 0):
            d = state[s]
            B.adamw_step(d["x_hi"], d["x_lo"], d["m"], d["v_hi"], d["v_lo"], g, n, e.hyper(hyp), t, s)
            torch.cuda.synchronize()
            edq[s].append(e.read())
            want = oracle_step(host[s], gb, t, s, hyp)
            if whole:
                edq_close(edq[s][-1], want)
            if whole or t in (9, 50, 150, 300, 600, steps):
                for k in KEYS:
                    if host[s][k] is not None:
                        got = W.bits(d[k]) if whole else W.bits(d[k][lo:hi])
                        assert_same_bits(got, host[s][k], f"strategy {s} step {t} {k}")
    # most updates fall below half an ulp of theta: plain bfloat16 drops them from the first step on; the
    # expansion carries them until its second component has grown to ~2^8 updates (a length-2 bfloat16
    # expansion resolves ~2^-17 of theta), after which part of them is lost there too
    assert edq[0][0]["lost"] > 0.5 * n and edq[0][-1]["lost"] > 0.5 * n
    assert edq[2][19]["lost"] < 0.05 * n
    assert edq[2][-1]["lost"] < edq[0][-1]["lost"]
    assert all(c["edq"] >= a["edq"] for c, a in zip(edq[2], edq[0]))
    # distance to the double-precision trajectory after 1000 steps, from the device's own arrays
    plus = to_f64(W.bits(state[2]["x_hi"][lo:hi])) + to_f64(W.bits(state[2]["x_lo"][lo:hi]))
    plain = to_f64(W.bits(state[0]["x_hi"][lo:hi]))
    moved = np.abs(th64 - theta0).sum()
    err_plus, err_plain = np.abs(plus - th64).sum(), np.abs(plain - th64).sum()
    assert moved > 0 and err_plain > 0.5 * moved          # plain bfloat16 has hardly followed
    assert err_plus < 0.5 * err_plain                     # observed 0.34: the second component saturates here
    assert B.pipeline_fault() == 0


@pytest.mark.parametrize("strategy", [1, 2])
def test_size_sweep_powers_of_four(strategy, step_kernel):
    # config 4: flat tensors of 4^6 ... 4^12 parameters, two steps each, every array and EDQ
    dev = torch.device("cuda")
    hyp = W.HYPERS
    for p in range(6, 13):
        n = 4 ** p
        theta = W.flat_weights(n, 4, dev)
        z = lambda: torch.zeros_like(theta)
        d = dict(x_hi=theta, x_lo=z(), m=z(), v_hi=z(), v_lo=z() if strategy == 2 else None)
        st = {k: (W.bits(v) if v is not None else None) for k, v in d.items()}
        e = EdqBuffers()
        for t in (1, 2):
            g = W.flat_grads(n, 4, t, dev)
            B.adamw_step(d["x_hi"], d["x_lo"], d["m"], d["v_hi"], d["v_lo"], g, n, e.hyper(hyp), t, strategy)
            torch.cuda.synchronize()
            want = oracle_step(st, W.bits(g), t, strategy, hyp)
            for k in KEYS:
                if st[k] is not None:
                    assert_same_bits(W.bits(d[k]), st[k], f"n=4^{p} step {t} {k}")
            edq_close(e.read(), want)


def test_effective_descent_quality_orders_the_precision_strategies():
    # Figure 3 (right) on synthetic data: share of the intended update that reaches the stored parameter,
    # EDQ / ||update||, with config-0 distributions (updates around half an ulp of the parameters).  Plain
    # bfloat16 loses part of every step, Kahan recovers it with a delay, the expansion-based options and
    # fp32 master weights apply it all.
    dev = torch.device("cuda")
    n, hyp, steps = 1 << 22, W.HYPERS, 40
    theta = W.flat_weights(n, 0, dev)
    e = EdqBuffers()
    quality = {}
    for name, strategy in (("A", B.BF16), ("Kahan", B.KAHAN), ("B", B.LIGHT), ("C", B.PLUS)):
        z = lambda: torch.zeros_like(theta)
        d = dict(x_hi=theta.clone(), x_lo=z() if strategy else None, m=z(), v_hi=z(), v_lo=z() if strategy == 2 else None)
        q = []
        for t in range(1, steps + 1):
            g = W.flat_grads(n, 0, t, dev)
            B.adamw_step(d["x_hi"], d["x_lo"], d["m"], d["v_hi"], d["v_lo"], g, n, e.hyper(hyp), t, strategy)
            torch.cuda.synchronize()
            r = e.read()
            q.append(r["edq"] / np.sqrt(r["sumsq"]))
        quality[name] = q
    master, m32, v32, th = theta.float(), torch.zeros(n, device=dev), torch.zeros(n, device=dev), theta.clone()
    q = []
    for t in range(1, steps + 1):
        g = W.flat_grads(n, 0, t, dev)
        B.adamw_step_fp32(th, master, m32, v32, g, n, e.hyper(hyp), t)
        torch.cuda.synchronize()
        r = e.read()
        q.append(r["edq"] / np.sqrt(r["sumsq"]))
    quality["D"] = q
    mean = {k: float(np.mean(v)) for k, v in quality.items()}
    print({k: (round(v[0], 4), round(v[-1], 4), round(mean[k], 4)) for k, v in quality.items()})
    for k in ("B", "C", "D"):
        assert min(quality[k]) > 0.995                               # the whole update arrives
    assert mean["A"] < 0.95 * mean["B"]                              # plain bfloat16 loses a visible share
    assert quality["Kahan"][0] == quality["A"][0]                    # first step: no compensation yet
    assert mean["A"] < mean["Kahan"] <= 1.05                         # later steps deliver what earlier ones lost


@pytest.mark.parametrize("api", ["flat", "multi"])
def test_one_tensor_longer_than_2_to_32_elements(api):
    # index arithmetic past 32 bits: a single Collage-plus tensor of 2^32 + 20,483 parameters (51.5 GB of
    # state), through the flat entry point and as a one-tensor plan; windows at the start, around 2^32 and
    # at the ragged end bit for bit, the element count and the sign of the sums from the EDQ record
    dev = torch.device("cuda")
    n = (1 << 32) + 20_483
    x = W.normal_bf16(n, 0.02, 9001, dev)
    g = W.normal_bf16(n, 1e-3, 9002, dev)
    xl, m, v, vl = (torch.zeros_like(x) for _ in range(4))
    arrs = (x, xl, m, v, vl)
    rng = np.random.default_rng(5)
    wins = _windows(n, rng, 4096, 8) + [((1 << 32) - 2048, (1 << 32) + 2048), (n - 20_483 - 64, n - 20_483 + 64)]
    st = {k: _gather(a, wins) for a, k in zip(arrs, KEYS)}
    gs = _gather(g, wins)
    e = EdqBuffers()
    plan = B.plan_create([(x, xl, m, v, vl, g, n)]) if api == "multi" else None
    for t in (1, 2):
        if api == "multi":      # the plan with the three-stage pipeline pinned, the flat call as chosen by size (large tiles)
            B.adamw_step_multi(plan, e.hyper(W.HYPERS, flags=B.FLAG_PIPELINE_KERNEL), t, B.PLUS)
        else:
            B.adamw_step(x, xl, m, v, vl, g, n, e.hyper(W.HYPERS), t, B.PLUS)
        torch.cuda.synchronize()
        oracle_step(st, gs, t, 2, W.HYPERS)
        for a, k in zip(arrs, KEYS):
            assert_same_bits(_gather(a, wins), st[k], f"{api} step {t} {k}")
        got = e.read()
        assert got["n"] == n and got["sumsq"] > 0 and got["edq"] > 0
    # every parameter moved: none of the 2^32 + 20,483 was skipped (theta changes in its pair with probability ~1)
    assert int((xl == 0).sum().item()) < n // 8
    assert B.pipeline_fault() == 0
    if plan is not None:
        B.plan_destroy(plan)
    del x, g, xl, m, v, vl, arrs
    torch.cuda.empty_cache()
