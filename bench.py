#!/usr/bin/env python
"""Benchmark of the Collage-plus multi-tensor AdamW step on the LLaMA-7B-shaped parameter set.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One "step" = one fused multi-tensor Collage-plus step (Algorithm 2 lines 8-13 with the EDQ
reduction of Eq. 3) over all 291 tensors / 6,738,415,616 parameters, state resident in HBM.
Prints ONE JSON line (rank 0).  With --impl reference the CPU oracle is timed instead, on a
bounded sample of the same workload, on this machine's host cores.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "collage_adamw_step_params_per_sec"
UNIT = "params/s"
BYTES_PER_PARAM = {0: 14, 1: 18, 2: 22}      # algorithmic HBM bytes per parameter per step (A, B, C)
STRATEGY = 2                                  # Collage-plus
WORKLOAD = "llama7b_shaped_291_tensors_collage_plus_with_edq"
# DRAM bytes per parameter of the step kernel from one ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum = 3.146 GB + 2.567 GB on the 262,148,096-parameter case, summary under
# profiles/); every byte is touched once, so traffic scales with the parameter count.
NCU_TRAFFIC_BYTES_PER_PARAM = (3.146235e9 + 2.567421e9) / 262_148_096


def host_threads():
    """Cores this process may run on: the oracle's thread count (a launcher's OMP_NUM_THREADS=1 does not apply)."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def measured_hbm_peak():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        return float(json.loads(f.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy)"
    return 6650.0, "fallback (earlier measurement on this pool)"


# ------------------------------------------------------------------ clocks ---

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.05)

    def __enter__(self):
        if self.nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


# ------------------------------------------------------------- GPU workload ---

def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def build_llama7b_state(torch, W, device, seed, layers=32):
    """Six flat bfloat16 arrays (theta, dtheta, m, v, dv, grad); tensors are consecutive views (16-byte aligned)."""
    shapes = W.llama7b_shapes(layers)
    n = sum(s for _, s in shapes)
    arrays = {k: torch.zeros(n, dtype=torch.bfloat16, device=device) for k in ("x_lo", "m", "v_hi", "v_lo")}
    arrays["x_hi"] = torch.empty(n, dtype=torch.bfloat16, device=device)
    arrays["grad"] = torch.empty(n, dtype=torch.bfloat16, device=device)
    rows, off = [], 0
    for i, (_, sz) in enumerate(shapes):
        arrays["x_hi"][off:off + sz] = W.normal_bf16(sz, 0.02, seed * 100_000 + i, device)
        arrays["grad"][off:off + sz] = W.normal_bf16(sz, 1e-3, seed * 100_000 + 50_000 + i, device)
        rows.append(tuple(arrays[k][off:off + sz] for k in ("x_hi", "x_lo", "m", "v_hi", "v_lo", "grad")) + (sz,))
        off += sz
    return arrays, rows, n


def run_collage(args):
    import torch
    import torch.distributed as dist
    from paper_2405_03637_b200 import binding as B
    from paper_2405_03637_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    # under torchrun (any world size, 1 included) the ranks talk over NCCL; a bare `python bench.py` does not
    use_dist = world > 1 or ("RANK" in os.environ and "MASTER_ADDR" in os.environ)
    if use_dist:
        dist.init_process_group("nccl", device_id=device)
    B.lib()                                             # fail loudly if the CUDA library is missing

    hyp = W.HYPERS
    arrays, rows, n = build_llama7b_state(torch, W, device, seed=3 + rank, layers=args.layers)
    plan = B.plan_create(rows, args.chunk_elems)
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    edq_sums = edq_dev[:16].view(torch.float64)         # {dot, sumsq}: what ranks exchange
    edq_lost = edq_dev[32:40].view(torch.int64)         # lost-update count
    stream = torch.cuda.current_stream()

    if args.replicas:                                   # variant: theta also written to R replicas by the step kernel
        rep_buffers = [torch.empty(n, dtype=torch.bfloat16, device=device) for _ in range(args.replicas)]
        offs, off = [], 0
        for r in rows:
            offs.append(off)
            off += r[6]
        B.plan_set_replicas(plan, [[buf[o:o + r[6]] for o, r in zip(offs, rows)] for buf in rep_buffers])
    if args.per_tensor:                                 # variant: EDQ kept per tensor (three launches per step)
        per = torch.zeros(len(rows) * 40, dtype=torch.uint8, device=device)
        cws = torch.empty(B.plan_workspace_bytes(plan), dtype=torch.uint8, device=device)

    def step(t):
        if args.per_tensor:
            B.adamw_step_multi_per_tensor(plan, B.make_hyper(**hyp, edq_out=edq_dev), t, STRATEGY, per, len(rows), cws, stream)
        else:
            B.adamw_step_multi(plan, B.make_hyper(**hyp, edq_out=edq_dev, workspace=ws), t, STRATEGY, stream)
        if use_dist:                                    # EDQ is global: sum the partial sums over ranks
            dist.all_reduce(edq_sums)
            dist.all_reduce(edq_lost)

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    t = 0
    for _ in range(args.warmup):
        t += 1
        step(t)
    barrier()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    with ClockSampler(physical_gpu_index(local_rank)) as clocks:
        ev[0].record(stream)
        for i in range(args.steps):
            t += 1
            step(t)
            ev[i + 1].record(stream)
        barrier()
    total_ms = ev[0].elapsed_time(ev[-1])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    if use_dist:
        tmax = torch.tensor([total_ms], dtype=torch.float64, device=device)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        total_ms = float(tmax.item())
    edq = B.read_edq(edq_dev)
    if use_dist:
        edq["edq"] = edq["dot"] / edq["sumsq"] ** 0.5 if edq["sumsq"] > 0 else 0.0

    ms_per_step = total_ms / args.steps
    value = world * n / (ms_per_step * 1e-3)
    peak, peak_src = measured_hbm_peak()
    kernel_ms = sorted(per_step)[len(per_step) // 2]    # median step on this rank: step kernel + 3-microsecond finalize
    achieved = n * BYTES_PER_PARAM[STRATEGY] / (kernel_ms * 1e-3) / 1e9

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD if args.layers == 32 else f"{WORKLOAD}_reduced_to_{args.layers}_layers",
                   "params_per_gpu": n, "tensors": len(rows), "strategy": "collage_plus",
                   "state_bytes_per_param": 12, "hbm_bytes_per_param_per_step": BYTES_PER_PARAM[STRATEGY],
                   "edq": True, "theta_replicas": args.replicas, "l2": "state (80.9 GB per GPU) far exceeds the 126 MB L2; no flush needed",
                   "parallelism": f"dp{world} (each rank owns a full 7B-shaped shard; EDQ sums all-reduced)"},
        "gpu_launches": (3 if args.per_tensor else 2) * args.steps,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": NCU_TRAFFIC_BYTES_PER_PARAM * n / 1e9, "traffic_unit": "GB per launch (ncu, scaled by parameters)",
                     "algorithmic": n * BYTES_PER_PARAM[STRATEGY] / 1e9, "peak_source": peak_src, "frac_of_nominal_8TBps": achieved / 8000.0,
                     "kernel": "adamw_step_pipeline_kernel<C, EDQ, multi-tensor>", "kernel_ms": kernel_ms},
        "clocks": clocks.summary(),
        "edq": edq["edq"],
    }
    if rank == 0 and world == 1 and not args.skip_extras:
        out["e2e"] = run_e2e(torch, B, W, device, args)
        out["cpu_baseline"] = run_cpu_baseline(W, seconds=args.cpu_seconds)
    elif rank == 0:
        out["e2e"] = None
    if use_dist:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


def run_e2e(torch, B, W, device, args):
    """Same step through collage_adamw_step_host: state in pinned HOST memory, H2D and D2H inside the timed region."""
    n = 1 << 30 if args.layers == 32 else 1 << 24
    host = {k: torch.zeros(n, dtype=torch.bfloat16).pin_memory() for k in ("x_lo", "m", "v_hi", "v_lo")}
    piece = 1 << 26
    x = torch.empty(n, dtype=torch.bfloat16).pin_memory()
    g = torch.empty(n, dtype=torch.bfloat16).pin_memory()
    for lo in range(0, n, piece):
        hi = min(n, lo + piece)
        x[lo:hi].copy_(W.normal_bf16(hi - lo, 0.02, 7000 + lo // piece, device))
        g[lo:hi].copy_(W.normal_bf16(hi - lo, 1e-3, 8000 + lo // piece, device))
    host["x_hi"], host["grad"] = x, g
    staging = torch.empty(768 << 20, dtype=torch.uint8, device=device)
    rec = (ctypes.c_uint8 * 64)()
    stream = torch.cuda.current_stream()

    def step(t):
        h = B.make_hyper(**W.HYPERS)
        h.edq_out = ctypes.addressof(rec)
        B.adamw_step_host(host["x_hi"], host["x_lo"], host["m"], host["v_hi"], host["v_lo"], host["grad"], n, h, t,
                          STRATEGY, staging, stream)

    steps = max(2, min(args.steps, 5))
    for t in (1, 2):
        step(t)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for t in range(3, 3 + steps):
        step(t)
    e1.record(stream)
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    ms = max(e0.elapsed_time(e1), wall * 1e3) / steps
    return {"value": n / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 12 * n, "d2h_bytes_per_step": 10 * n + 40,
            "ms_per_step": ms, "steps": steps,
            "sample": f"first {n} parameters of the flattened workload, state in pinned host memory, "
                      "collage_adamw_step_host (768 MiB device staging)"}


def run_size_sweep(args):
    """Flat tensors of 4^6 ... 4^15 parameters (Collage-light and -plus, EDQ on): one JSON line per size.

    Sizes whose state fits in L2 are rotated over enough independent buffer sets to exceed 512 MB, so
    that "HBM GB/s" is not an L2 number; the smallest sizes are launch-latency bound and say so.
    """
    import torch
    from paper_2405_03637_b200 import binding as B
    from paper_2405_03637_b200 import workloads as W
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    peak, _ = measured_hbm_peak()
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream()
    for p in range(6, 16):
        n = 4 ** p
        for strategy, name in ((1, "collage_light"), (2, "collage_plus")):
            state_bytes = (10 if strategy == 1 else 12) * n
            sets = max(1, min(64, -(-(512 << 20) // state_bytes)))
            bufs = []
            for k in range(sets):
                x = W.flat_weights(n, 4 + k, device)
                z = lambda: torch.zeros_like(x)
                bufs.append((x, z(), z(), z(), z() if strategy == 2 else None, W.flat_grads(n, 4 + k, 1, device)))
            h = B.make_hyper(**W.HYPERS, edq_out=edq_dev, workspace=ws)
            iters = max(20, min(400, int(2e10 // (n * BYTES_PER_PARAM[strategy])) * 4))
            for t in range(1, 4):
                B.adamw_step(*bufs[t % sets], n, h, t, strategy, stream)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(iters):
                B.adamw_step(*bufs[i % sets], n, h, 4 + i, strategy, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / iters
            gbs = n * BYTES_PER_PARAM[strategy] / (ms * 1e-3) / 1e9
            line = {"n": n, "strategy": name, "us_per_step": ms * 1e3, "params_per_sec": n / (ms * 1e-3),
                    "hbm_gbs": gbs, "frac_of_measured_peak": gbs / peak, "frac_of_nominal_8TBps": gbs / 8000.0,
                    "buffer_sets": sets, "launches_per_step": 2}
            if p <= 11:
                # the same steps recorded once into a CUDA graph and replayed: no per-launch host cost
                side = torch.cuda.Stream()
                side.wait_stream(stream)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(iters):
                        B.adamw_step(*bufs[i % sets], n, h, 4 + i, strategy, side)
                graph.replay()
                torch.cuda.synchronize()
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record(stream)
                for _ in range(3):
                    graph.replay()
                g1.record(stream)
                torch.cuda.synchronize()
                gms = g0.elapsed_time(g1) / (3 * iters)
                line["us_per_step_graph"] = gms * 1e3
                line["hbm_gbs_graph"] = n * BYTES_PER_PARAM[strategy] / (gms * 1e-3) / 1e9
                del graph
            print(json.dumps(line), flush=True)
            del bufs
            torch.cuda.empty_cache()


def run_strategy_sweep(args):
    """All precision options, the comparators and the step variants on one flat tensor (2^30 parameters by default)."""
    import torch
    from paper_2405_03637_b200 import binding as B
    from paper_2405_03637_b200 import workloads as W
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    peak, _ = measured_hbm_peak()
    n = 1 << args.sweep_log2n
    x = W.flat_weights(n, 0, device)
    z = lambda: torch.zeros_like(x)
    xl, m, v, vl, g = z(), z(), z(), z(), W.flat_grads(n, 0, 1, device)
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream()
    cases = [("A plain bf16", B.BF16, 0, 14), ("B collage-light", B.LIGHT, 0, 18), ("C collage-plus", B.PLUS, 0, 22),
             ("BF16-Kahan", B.KAHAN, 0, 18), ("B + TwoSum Grow", B.LIGHT, B.FLAG_TWOSUM_GROW, 18),
             ("C + TwoSum Grow", B.PLUS, B.FLAG_TWOSUM_GROW, 22), ("C + decay by Grow", B.PLUS, B.FLAG_DECAY_BY_GROW, 22),
             ("C storage, fp32 arithmetic in registers", B.PLUS_FP32_REGISTERS, 0, 22)]
    def timed(call, bytes_per_param, name):
        for t in range(1, 4):
            call(t)
        torch.cuda.synchronize()
        iters = args.sweep_iters
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
        ev[0].record(stream)
        for i in range(iters):
            call(4 + i)
            ev[i + 1].record(stream)
        torch.cuda.synchronize()
        ts = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(iters))
        ms = ts[len(ts) // 2]
        gbs = n * bytes_per_param / (ms * 1e-3) / 1e9
        print(json.dumps({"step": name, "n": n, "ms_per_step": ms, "params_per_sec": n / (ms * 1e-3),
                          "bytes_per_param": bytes_per_param, "hbm_gbs": gbs, "frac_of_measured_peak": gbs / peak}), flush=True)
    for name, strategy, flags, bpp in cases:
        h = B.make_hyper(**W.HYPERS, flags=flags, edq_out=edq_dev, workspace=ws)
        a = (x, xl if strategy >= 1 else None, m, v, vl if strategy in (2, 4) else None, g)
        timed(lambda t: B.adamw_step(*a, n, h, t, strategy, stream), bpp, name)
    del xl, vl, m, v
    torch.cuda.empty_cache()
    m32, v32 = torch.zeros(n, dtype=torch.float32, device=device), torch.zeros(n, dtype=torch.float32, device=device)
    master = x.float()
    h = B.make_hyper(**W.HYPERS, edq_out=edq_dev, workspace=ws)
    timed(lambda t: B.adamw_step_fp32(x, master, m32, v32, g, n, h, t, stream), 28, "D fp32 states + fp32 master")
    timed(lambda t: B.adamw_step_fp32(x, None, m32, v32, g, n, h, t, stream), 22, "D^-MW fp32 states, no master")


def run_cpu_baseline(W, seconds=15.0, threads=None):
    """The oracle as it stands on this machine's cores, on a bounded slice of the same workload."""
    import numpy as np
    import oracle
    threads = threads or host_threads()
    n = 1 << 24
    theta = W.bits(W.normal_bf16(n, 0.02, 300_000))
    g = W.bits(W.normal_bf16(n, 1e-3, 350_000))
    st = [theta, np.zeros_like(theta), np.zeros_like(theta), np.zeros_like(theta), np.zeros_like(theta)]
    done, t0, t = 0, time.perf_counter(), 0
    while True:
        t += 1
        oracle.adamw_step(st[0], st[1], st[2], st[3], st[4], g, step=t, strategy=STRATEGY, threads=threads, **W.HYPERS)
        done += n
        el = time.perf_counter() - t0
        if el >= seconds or t >= 200:
            break
    # one thread, on a 2^21-parameter piece of the same arrays (a few seconds)
    n1 = 1 << 21
    one = [a[:n1].copy() for a in st]
    t1, s0 = 0, time.perf_counter()
    while True:
        t1 += 1
        oracle.adamw_step(one[0], one[1], one[2], one[3], one[4], g[:n1].copy(), step=t + t1, strategy=STRATEGY, threads=1, **W.HYPERS)
        e1 = time.perf_counter() - s0
        if e1 >= 3.0 or t1 >= 50:
            break
    return {"value": done / el, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{t} Collage-plus steps over the first {n} parameters of the workload's embedding tensor "
                      f"({el:.1f} s)",
            "value_one_thread": n1 * t1 / e1, "sample_one_thread": f"{t1} steps over {n1} parameters ({e1:.1f} s)"}


def run_reference(args):
    """--impl reference: the oracle timed as the reference arm (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    import oracle
    from paper_2405_03637_b200 import workloads as W
    threads = host_threads()
    n = 1 << 23
    theta = W.bits(W.normal_bf16(n, 0.02, 300_000))
    g = W.bits(W.normal_bf16(n, 1e-3, 350_000))
    st = [theta, np.zeros_like(theta), np.zeros_like(theta), np.zeros_like(theta), np.zeros_like(theta)]
    t = 0
    for _ in range(args.warmup):
        t += 1
        oracle.adamw_step(st[0], st[1], st[2], st[3], st[4], g, step=t, strategy=STRATEGY, threads=threads, **W.HYPERS)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        t += 1
        oracle.adamw_step(st[0], st[1], st[2], st[3], st[4], g, step=t, strategy=STRATEGY, threads=threads, **W.HYPERS)
    el = time.perf_counter() - t0
    value = n * args.steps / el
    sample = f"each step = one Collage-plus oracle step over the first {n} parameters of the workload"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": el / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "strategy": "collage_plus", "edq": True},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="collage", choices=["collage", "reference"])
    ap.add_argument("--layers", type=int, default=32, help="transformer layers of the 7B-shaped set (32 = full)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--skip-extras", action="store_true", help="no e2e and no CPU baseline (profiling runs)")
    ap.add_argument("--chunk-elems", type=int, default=0, help="chunk size of the multi-tensor plan (0 = library default)")
    ap.add_argument("--replicas", type=int, default=0, help="also write theta to this many replica buffers (same GPU)")
    ap.add_argument("--per-tensor", action="store_true", help="time the per-tensor EDQ variant of the step")
    ap.add_argument("--strategy-sweep", action="store_true", help="time every option, comparator and variant on a flat tensor")
    ap.add_argument("--size-sweep", action="store_true", help="flat-tensor size sweep instead of the benchmark")
    ap.add_argument("--sweep-log2n", type=int, default=30, help="--strategy-sweep: log2 of the flat tensor's length")
    ap.add_argument("--sweep-iters", type=int, default=40, help="--strategy-sweep: timed steps per case")
    args = ap.parse_args()
    if args.size_sweep:
        run_size_sweep(args)
    elif args.strategy_sweep:
        run_strategy_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_collage(args)


if __name__ == "__main__":
    main()
