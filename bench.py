#!/usr/bin/env python
"""Benchmark of the Collage-plus multi-tensor AdamW step on the LLaMA-7B-shaped parameter set.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config 0..4]

One "step" = one fused multi-tensor Collage-plus step (Algorithm 2 lines 8-13 with the EDQ
reduction of Eq. 3) over all 291 tensors / 6,738,415,616 parameters, state resident in HBM: ONE
kernel launch.  Prints ONE JSON line (rank 0).  With --impl reference the CPU oracle is timed
instead, on a bounded sample of the same workload, on this machine's host cores.

--config selects one of the synthetic configurations (3, the default, is the headline above):
0 flat 2^20 parameters, options A/B/C; 1 GPT-2-small-shaped 148-tensor set, Collage-light;
2 the 64 Mi-parameter lost-arithmetic stress set, Collage-plus and plain bfloat16; 4 the flat
size sweep.  --primitive-sweep times the batched MCF primitives and the stand-alone EDQ.
With N > 1 ranks the headline is the weak-scaling step (every rank its own 7B-shaped set) and a
"sharded" record is added: ONE 7B-shaped set cut over the ranks, theta delivered to every rank's
full copy by the step kernel's own stores into peer memory.  --sharded-selfcheck runs that flow
with two emulated ranks on one GPU.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "collage_adamw_step_params_per_sec"
UNIT = "params/s"
BYTES_PER_PARAM = {0: 14, 1: 18, 2: 22}      # algorithmic HBM bytes per parameter per step (A, B, C)
STRATEGY_NAME = {0: "plain_bf16", 1: "collage_light", 2: "collage_plus"}
STRATEGY = 2                                  # Collage-plus
WORKLOAD = "llama7b_shaped_291_tensors_collage_plus_with_edq"
# DRAM bytes per parameter of the step kernel from one ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum = 3.146 GB + 2.565 GB on the 262,148,096-parameter case: the embedding, final norm
# and lm_head of the same layout); every byte is touched once, so traffic scales with the parameter count.
NCU_TRAFFIC_BYTES_PER_PARAM = (3.146280e9 + 2.564761e9) / 262_148_096


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


def load_binding(args):
    """The library's binding; --lib PATH selects another build of the same sources (a measurement build)."""
    from paper_2405_03637_b200 import binding as B
    if getattr(args, "lib", None):
        B.load(args.lib)
    B.lib()                                             # fail loudly if the CUDA library is missing
    return B


def run_collage(args):
    import torch
    import torch.distributed as dist
    from paper_2405_03637_b200 import workloads as W
    B = load_binding(args)

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

    hyp = W.HYPERS
    arrays, rows, n = build_llama7b_state(torch, W, device, seed=3 + rank, layers=args.layers)
    plan = B.plan_create(rows, args.chunk_elems)
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    B.workspace_init(ws)
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
        per = torch.zeros(len(rows) * B.EDQ_RECORD_BYTES, dtype=torch.uint8, device=device)
        cws = torch.empty(B.plan_workspace_bytes(plan), dtype=torch.uint8, device=device)

    pin = {"auto": 0, "pipeline": B.FLAG_PIPELINE_KERNEL, "large": B.FLAG_LARGE_TILES}[args.pin_kernel]

    def step(t):
        if args.per_tensor:
            B.adamw_step_multi_per_tensor(plan, B.make_hyper(**hyp, flags=pin, edq_out=edq_dev), t, STRATEGY, per, len(rows), cws, stream)
        else:
            B.adamw_step_multi(plan, B.make_hyper(**hyp, flags=pin, edq_out=edq_dev, workspace=ws), t, STRATEGY, stream)
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
    edq = B.edq_combine([B.read_edq(edq_dev)])          # Eq. 3 on the sums (summed over ranks when there are several)

    ms_per_step = total_ms / args.steps
    value = world * n / (ms_per_step * 1e-3)
    peak, peak_src = measured_hbm_peak()
    kernel_ms = sorted(per_step)[len(per_step) // 2]    # median step on this rank: one launch of the step kernel
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
        "gpu_launches": (3 if args.per_tensor else 1) * args.steps, "build_flavor": B.build_flavor(),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": NCU_TRAFFIC_BYTES_PER_PARAM * n / 1e9, "traffic_unit": "GB per launch (ncu, scaled by parameters)",
                     "algorithmic": n * BYTES_PER_PARAM[STRATEGY] / 1e9, "peak_source": peak_src, "frac_of_nominal_8TBps": achieved / 8000.0,
                     "kernel": "adamw_step_pipeline_kernel<C, EDQ, multi-tensor, " +
                               ("2 stages x 8192-element tiles>" if (args.pin_kernel == "large" or (args.pin_kernel == "auto" and n >= 1 << 27
                                                                     and (args.chunk_elems or 24576) % 8192 == 0))
                                else "3 stages x 4096-element tiles>"), "kernel_ms": kernel_ms},
        "clocks": clocks.summary(),
        "edq": edq["edq"], "edq_fault": edq["fault"],
    }
    if not args.skip_extras:
        # every rank takes part in the end-to-end leg; the oracle is timed on rank 0 of a one-GPU run only
        out["e2e"] = run_e2e(torch, B, W, device, args, dist if use_dist else None, world)
        if rank == 0 and world == 1:
            out["cpu_baseline"] = run_cpu_baseline(W, seconds=args.cpu_seconds)
    else:
        out["e2e"] = None
    # hand the GPUs back before the sharded leg (it runs as child processes of rank 0, so that nothing
    # it does can take the headline line with it)
    B.plan_destroy(plan)
    del arrays, rows, ws, edq_dev, edq_sums, edq_lost
    torch.cuda.empty_cache()
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        if world > 1 and not args.no_sharded:
            out["sharded"] = run_sharded_children(args, world)
        print(json.dumps(out))


# ------------------------------------------------------------ sharded step ---

def run_sharded_children(args, world):
    """Rank 0 of an N-rank run: time the sharded step in child processes (their own rendezvous, one per GPU)."""
    env = {k: v for k, v in os.environ.items()
           if not (k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "LOCAL_WORLD_SIZE", "GROUP_RANK", "ROLE_RANK", "ROLE_NAME",
                         "ROLE_WORLD_SIZE", "GROUP_WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT", "OMP_NUM_THREADS")
                   or k.startswith("TORCHELASTIC_") or k.startswith("TORCH_NCCL_"))}
    port = int(os.environ.get("MASTER_PORT", "29500")) + 7
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(ROOT / "bench.py"), "--gpus", str(world),
           "--sharded-only", "--steps", str(args.steps), "--warmup", str(args.warmup), "--layers", str(args.layers)]
    if args.lib:
        cmd += ["--lib", args.lib]
    if getattr(args, "sharded_backend", "nccl") != "nccl":
        cmd += ["--sharded-backend", args.sharded_backend]
    if getattr(args, "sharded_one_device", False):
        cmd += ["--sharded-one-device"]
    try:
        proc = subprocess.run(cmd, capture_output=True, text=True, timeout=420, env=env, cwd=str(ROOT))
    except subprocess.TimeoutExpired:
        return {"unavailable": "the sharded leg did not finish within 420 s"}
    for line in reversed(proc.stdout.splitlines()):
        if line.startswith("{") and '"sharded_step"' in line:
            return json.loads(line)["sharded_step"]
    tail = (proc.stderr or proc.stdout).strip().splitlines()[-1:] or ["no output"]
    return {"unavailable": f"child exit code {proc.returncode}: {tail[0][:300]}"}


def theta_views(flat, sizes):
    """Per-tensor views of one flat theta buffer (consecutive, so every tensor starts 16-byte aligned when n % 8 == 0)."""
    out, off = [], 0
    for n in sizes:
        out.append(flat[off:off + n])
        off += n
    return out


def fill_theta(flat, sizes, W, device, seed):
    off = 0
    for i, n in enumerate(sizes):
        flat[off:off + n] = W.normal_bf16(n, 0.02, seed * 100_000 + i, device)
        off += n


def run_sharded_only(args):
    """ONE 7B-shaped set cut over the ranks (optimizer-state ownership); every rank keeps a full copy of theta.

    A rank steps its slice with one launch; the same kernel stores the slice's new theta into every peer's
    copy (plain stores into peer memory mapped through CUDA IPC, no loads from peers, no waits on peers).
    {dot, sumsq, lost} are all-reduced over NCCL; that collective also orders the peers' stores before the
    next step.  Timed on the device, max over ranks.
    """
    import torch
    import torch.distributed as dist
    from torch.multiprocessing.reductions import rebuild_cuda_tensor, reduce_tensor
    from paper_2405_03637_b200 import sharding as S
    from paper_2405_03637_b200 import workloads as W
    B = load_binding(args)
    rank, local_rank, world = int(os.environ["RANK"]), int(os.environ["LOCAL_RANK"]), int(os.environ["WORLD_SIZE"])
    if args.sharded_one_device:
        # test mode for a box with one GPU: every rank is a process of its own on device 0, so the handle
        # exchange, the mapping of another process's memory and the stores into it are the real ones; only
        # the sums travel over gloo (NCCL does not take two ranks on one device).  The ranks' kernels never
        # wait on one another, so sharing a device is safe.
        local_rank = 0
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if args.sharded_backend == "gloo":
        dist.init_process_group("gloo")
    else:
        dist.init_process_group("nccl", device_id=device)
    result = None
    try:
        sizes = [n for _, n in W.llama7b_shapes(args.layers)]
        total = sum(sizes)
        mine_flat = torch.empty(total, dtype=torch.bfloat16, device=device)
        fill_theta(mine_flat, sizes, W, device, seed=3)              # the same theta on every rank
        torch.cuda.synchronize()
        # map every peer's copy into this process
        handles = [None] * world
        dist.all_gather_object(handles, (local_rank, reduce_tensor(mine_flat)[1]))
        flats = {}
        for r, (peer_device, ipc) in enumerate(handles):
            if r == rank:
                flats[r] = mine_flat
            else:
                if peer_device != local_rank:
                    B.enable_peer_access(peer_device)
                flats[r] = rebuild_cuda_tensor(*ipc)
        copies = [theta_views(flats[r], sizes) for r in range(world)]
        alloc = lambda n: torch.zeros(n, dtype=torch.bfloat16, device=device)
        shard = S.ShardedRank(sizes, rank, world, copies, alloc, STRATEGY)
        for k, row in enumerate(shard.rows):                         # gradients of the slice
            row[5].copy_(W.normal_bf16(row[6], 1e-3, 9_000_000 + rank * 10_000 + k, device))
        stepper = S.CudaStepper(shard, torch)
        stream = torch.cuda.current_stream()
        dist.barrier()
        torch.cuda.synchronize()
        t = 0
        for _ in range(args.warmup):
            t += 1
            stepper.step(W.HYPERS, t, stream)
            stepper.allreduce(dist)
        dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            t += 1
            stepper.step(W.HYPERS, t, stream)
            stepper.allreduce(dist)
        e1.record(stream)
        dist.barrier()
        torch.cuda.synchronize()
        ms = torch.tensor([e0.elapsed_time(e1) / args.steps], dtype=torch.float64, device=device)
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        ms = float(ms.item())
        edq = stepper.read()
        sums = [None] * world
        dist.all_gather_object(sums, S.theta_checksum(copies[rank], torch))
        sent = shard.gathered_bytes_per_step()
        hbm_ms = shard.elements * BYTES_PER_PARAM[STRATEGY] / (measured_hbm_peak()[0] * 1e9) * 1e3
        link_ms = sent / 770e9 * 1e3                                 # measured peer-copy bandwidth per direction
        result = {
            "ranks": world, "params_total": total, "params_per_rank": shard.elements, "ms_per_step": ms,
            "params_per_sec": total / (ms * 1e-3), "theta_bytes_sent_per_rank_per_step": sent,
            "nvlink_gbs_per_direction_per_rank": sent / (ms * 1e-3) / 1e9,
            "expected_ms": {"hbm": hbm_ms, "nvlink_at_770_gbs": link_ms, "bound": max(hbm_ms, link_ms)},
            "frac_of_bound": max(hbm_ms, link_ms) / ms, "copies_agree": len(set(sums)) == 1,
            "edq": edq["edq"], "edq_fault": edq["fault"], "exchange": "plain stores into CUDA-IPC mapped peer memory "
            "from inside the step kernel; {dot, sumsq, lost} all-reduced (" + args.sharded_backend + ")",
            "gpu_launches": args.steps,
        }
        stepper.close()
        del stepper, shard, copies, flats                            # peers' mappings are released before anyone exits
    except Exception as exc:                                         # noqa: BLE001 - reported, never fatal for the caller
        result = {"unavailable": f"{type(exc).__name__}: {str(exc)[:300]}"}
    finally:
        try:
            dist.barrier()
            dist.destroy_process_group()
        except Exception:                                            # noqa: BLE001
            pass
    if rank == 0:
        print(json.dumps({"sharded_step": result}))


def run_sharded_selfcheck(args):
    """The sharded flow on ONE GPU with two emulated ranks, through the same harness as run_sharded_only.

    The ranks' kernels never wait on one another, so running them one after the other is the same
    computation.  Checks: every rank's full theta copy equals the theta of an unsharded step over the
    same set bit for bit, and the summed EDQ records equal its record within 1e-5.
    """
    import torch
    from paper_2405_03637_b200 import sharding as S
    from paper_2405_03637_b200 import workloads as W
    B = load_binding(args)
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    world = 2
    sizes = [n for _, n in W.llama7b_shapes(args.layers)]
    total = sum(sizes)
    flats = [torch.empty(total, dtype=torch.bfloat16, device=device) for _ in range(world + 1)]   # last: unsharded run
    fill_theta(flats[0], sizes, W, device, seed=3)
    for f in flats[1:]:
        f.copy_(flats[0])
    copies = [theta_views(f, sizes) for f in flats]
    alloc = lambda n: torch.zeros(n, dtype=torch.bfloat16, device=device)
    shards = [S.ShardedRank(sizes, r, world, copies[:world], alloc, STRATEGY) for r in range(world)]
    whole = S.ShardedRank(sizes, 0, 1, [copies[world]], alloc, STRATEGY)
    # gradients: drawn per tensor for the unsharded set, each rank gets the matching slices
    grads = {}
    for (i, b, e), row in zip(whole.ranges, whole.rows):
        row[5].copy_(W.normal_bf16(e - b, 1e-3, 350_000 + i, device))
        grads[i] = row[5]
    for sh in shards:
        for (i, b, e), row in zip(sh.ranges, sh.rows):
            row[5].copy_(grads[i][b:e])
    steppers = [S.CudaStepper(sh, torch) for sh in shards]
    ref = S.CudaStepper(whole, torch)
    ok, worst = True, 0.0
    for t in range(1, args.steps + 1):
        for st in steppers:
            st.step(W.HYPERS, t)
        ref.step(W.HYPERS, t)
        torch.cuda.synchronize()
        recs = [B.read_edq(st.record) for st in steppers]
        got, want = B.edq_combine(recs), B.read_edq(ref.record)
        for k in ("dot", "sumsq", "edq"):
            worst = max(worst, abs(got[k] - want[k]) / abs(want[k]))
        ok = ok and got["lost"] == want["lost"] and got["n"] == want["n"] == total and got["fault"] == 0
        ok = ok and all(torch.equal(f.view(torch.int16), flats[world].view(torch.int16)) for f in flats[:world])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(args.steps + 1, args.steps + 4):                  # timing only: three more steps of both ranks
        for st in steppers:
            st.step(W.HYPERS, t)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / 3
    print(json.dumps({"sharded_selfcheck": {
        "ok": bool(ok and worst <= 1e-5), "emulated_ranks": world, "params_total": total, "steps": args.steps,
        "theta_copies_bitwise_equal_to_unsharded": bool(ok), "edq_max_relative_difference": worst,
        "ms_per_step_both_ranks_back_to_back": ms,
        "theta_bytes_sent_per_rank_per_step": shards[0].gathered_bytes_per_step()}}))
    for st in steppers + [ref]:
        st.close()


def run_e2e(torch, B, W, device, args, dist=None, world=1):
    """Same step through collage_adamw_step_host: state in pinned HOST memory, H2D and D2H inside the timed region.

    With several ranks every rank steps a sample of its own at the same time (they share the host's memory
    and PCIe root), the time is the maximum over ranks and the value the sum of the samples over it.
    """
    n = (1 << 30 if world == 1 else 1 << 28) if args.layers == 32 else 1 << 24
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
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for t in range(3, 3 + steps):
        step(t)
    e1.record(stream)
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    ms = max(e0.elapsed_time(e1), wall * 1e3) / steps
    if dist is not None:
        tmax = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        ms = float(tmax.item())
    return {"value": world * n / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": world * 12 * n,
            "d2h_bytes_per_step": world * (10 * n + 48), "ms_per_step": ms, "steps": steps,
            "sample": f"first {n} parameters of the flattened workload per GPU, state in pinned host memory, "
                      "collage_adamw_step_host (768 MiB device staging)"}


def run_size_sweep(args):
    """Flat tensors of 4^6 ... 4^15 parameters (Collage-light and -plus, EDQ on): one JSON line per size.

    Sizes whose state fits in L2 are rotated over enough independent buffer sets to exceed 512 MB, so
    that "HBM GB/s" is not an L2 number; the smallest sizes are launch-latency bound and say so.
    """
    import torch
    from paper_2405_03637_b200 import workloads as W
    B = load_binding(args)
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    peak, _ = measured_hbm_peak()
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    B.workspace_init(ws)
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
                    "buffer_sets": sets, "launches_per_step": 1}
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
    from paper_2405_03637_b200 import workloads as W
    B = load_binding(args)
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    peak, _ = measured_hbm_peak()
    n = 1 << args.sweep_log2n
    x = W.flat_weights(n, 0, device)
    z = lambda: torch.zeros_like(x)
    xl, m, v, vl, g = z(), z(), z(), z(), W.flat_grads(n, 0, 1, device)
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    B.workspace_init(ws)
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


def _time_steps(torch, call, iters, stream, warm=3):
    """Median and mean milliseconds of `call(i)` over `iters` launches, CUDA events on `stream`."""
    for i in range(warm):
        call(i)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    ev[0].record(stream)
    for i in range(iters):
        call(warm + i)
        ev[i + 1].record(stream)
    torch.cuda.synchronize()
    each = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(iters))
    return each[len(each) // 2], ev[0].elapsed_time(ev[-1]) / iters


def _line(args, B, workload, n, strategy, ms, extra):
    peak, peak_src = measured_hbm_peak()
    gbs = n * BYTES_PER_PARAM[strategy] / (ms * 1e-3) / 1e9
    out = {"metric": METRIC, "value": n / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "ms_per_step": ms,
           "higher_is_better": True, "dtype": "bf16", "data": "synthetic", "vs_baseline": None,
           "config": {"workload": workload, "params": n, "strategy": STRATEGY_NAME[strategy], "edq": True},
           "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                        "frac_of_nominal_8TBps": gbs / 8000.0, "algorithmic": n * BYTES_PER_PARAM[strategy] / 1e9,
                        "peak_source": peak_src},
           "gpu_launches_per_step": 1, "build_flavor": B.build_flavor()}
    out.update(extra)
    return out


def run_config0(args):
    """Config 0: one flat tensor of 2^20 parameters, options A, B and C with EDQ (the state is L2-resident:
    the steps rotate over buffer sets of more than 512 MB in total so that the figure is an HBM figure)."""
    import torch
    from paper_2405_03637_b200 import workloads as W
    B = load_binding(args)
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    stream = torch.cuda.current_stream()
    n = 1 << 20
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    B.workspace_init(ws)
    for strategy in (0, 1, 2):
        sets = -(-(512 << 20) // ((8, 10, 12)[strategy] * n))
        bufs = []
        for k in range(sets):
            x = W.flat_weights(n, k, device)
            z = lambda: torch.zeros_like(x)
            bufs.append((x, z() if strategy >= 1 else None, z(), z(), z() if strategy == 2 else None, W.flat_grads(n, k, 1, device)))
        h = B.make_hyper(**W.HYPERS, edq_out=edq_dev, workspace=ws)
        med, mean = _time_steps(torch, lambda i: B.adamw_step(*bufs[i % sets], n, h, 1 + i, strategy, stream), 2000, stream)
        # the same launches recorded into a CUDA graph and replayed: no per-launch host cost
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(400):
                B.adamw_step(*bufs[i % sets], n, h, 1 + i, strategy, side)
        graph.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for _ in range(5):
            graph.replay()
        g1.record(stream)
        torch.cuda.synchronize()
        gms = g0.elapsed_time(g1) / (5 * 400)
        print(json.dumps(_line(args, B, "config0_flat_2p20", n, strategy, mean, {
            "us_per_step": mean * 1e3, "us_per_step_median": med * 1e3, "us_per_step_graph_replay": gms * 1e3,
            "hbm_gbs_graph_replay": n * BYTES_PER_PARAM[strategy] / (gms * 1e-3) / 1e9, "buffer_sets": sets,
            "timing": "2000 launches back to back on one stream; the state (12 MB) fits L2, so the launches rotate over "
                      f"{sets} buffer sets"})), flush=True)
        del bufs, graph
        torch.cuda.empty_cache()


def run_config1(args):
    """Config 1: GPT-2-small-shaped set (148 tensors, 124,439,808 parameters), one multi-tensor Collage-light
    launch per step, 100 timed steps."""
    import torch
    from paper_2405_03637_b200 import workloads as W
    B = load_binding(args)
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    stream = torch.cuda.current_stream()
    shapes = W.gpt2_small_shapes()
    rows = []
    for i, (_, n) in enumerate(shapes):
        x = W.flat_weights(n, 1000 + i, device)
        rows.append((x, torch.zeros_like(x), torch.zeros_like(x), torch.zeros_like(x), None, W.normal_bf16(n, 1e-3, 2_001_000 + i, device), n))
    total = sum(r[6] for r in rows)
    plan = B.plan_create(rows, args.chunk_elems)
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    B.workspace_init(ws)
    h = B.make_hyper(**W.HYPERS, edq_out=edq_dev, workspace=ws)
    med, mean = _time_steps(torch, lambda i: B.adamw_step_multi(plan, h, 1 + i, B.LIGHT, stream), 100, stream, warm=5)
    print(json.dumps(_line(args, B, "config1_gpt2_small_shaped_148_tensors", total, 1, med, {
        "ms_per_step_mean": mean, "steps": 100, "tensors": len(rows), "chunks": B.plan_num_chunks(plan),
        "l2": "state (1.24 GB) exceeds the 126 MB L2"})), flush=True)
    B.plan_destroy(plan)


def run_config2(args):
    """Config 2: 64 Mi parameters of the lost-arithmetic stress distributions, Collage-plus and plain bfloat16."""
    import torch
    from paper_2405_03637_b200 import workloads as W
    B = load_binding(args)
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    stream = torch.cuda.current_stream()
    n = 1 << 26
    theta = W.stress_weights(n, 2, device)
    g = W.stress_grads(n, 2, 1, device)
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    B.workspace_init(ws)
    h = B.make_hyper(**W.HYPERS_STRESS, edq_out=edq_dev, workspace=ws)
    for strategy in (2, 0):
        z = lambda: torch.zeros_like(theta)
        a = (theta.clone(), z() if strategy else None, z(), z(), z() if strategy == 2 else None, g)
        med, mean = _time_steps(torch, lambda i: B.adamw_step(*a, n, h, 1 + i, strategy, stream), 200, stream, warm=5)
        rec = B.read_edq(edq_dev)
        print(json.dumps(_line(args, B, "config2_stress_64Mi", n, strategy, med, {
            "ms_per_step_mean": mean, "steps": 200, "lost_fraction_last_step": rec["lost"] / n,
            "edq_over_update_norm_last_step": rec["edq"] / rec["sumsq"] ** 0.5 if rec["sumsq"] > 0 else 0.0,
            "l2": "state (0.5 - 0.8 GB) exceeds the 126 MB L2"})), flush=True)
        del a
        torch.cuda.empty_cache()


def run_primitive_sweep(args):
    """The batched MCF primitives, single rounded operations and the stand-alone EDQ on 2^28 elements:
    GB/s = 2 B x arrays moved / time, against the measured copy peak."""
    import torch
    from paper_2405_03637_b200 import workloads as W
    B = load_binding(args)
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    stream = torch.cuda.current_stream()
    peak, _ = measured_hbm_peak()
    n = 1 << args.sweep_log2n if args.sweep_log2n != 30 else 1 << 28
    a, b, c, d = (W.normal_bf16(n, s, 40 + k, device) for k, s in enumerate((0.02, 1e-3, 1e-4, 1.0)))
    o0, o1 = torch.empty_like(a), torch.empty_like(a)
    edq_dev = torch.zeros(64, dtype=torch.uint8, device=device)
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
    B.workspace_init(ws)
    cases = [
        ("fast_two_sum", 4, lambda: B.fast_two_sum(a, b, o0, o1, n, stream)),
        ("two_sum", 4, lambda: B.two_sum(a, b, o0, o1, n, stream)),
        ("two_prod", 4, lambda: B.two_prod(a, b, o0, o1, n, stream)),
        ("renormalize", 4, lambda: B.renormalize(a, b, o0, o1, n, stream)),
        ("grow", 5, lambda: B.grow(a, b, c, o0, o1, n, stream)),
        ("scaling", 5, lambda: B.scaling(a, b, c, o0, o1, n, stream)),
        ("mul", 6, lambda: B.mul(a, b, c, d, o0, o1, n, stream)),
        ("rounded add", 3, lambda: B.rounded_op(B.OP_ADD, a, b, None, o0, n, stream)),
        ("rounded div", 3, lambda: B.rounded_op(B.OP_DIV, a, d, None, o0, n, stream)),
        ("rounded sqrt", 2, lambda: B.rounded_op(B.OP_SQRT, d, None, None, o0, n, stream)),
        ("rounded fma", 4, lambda: B.rounded_op(B.OP_FMA, a, b, c, o0, n, stream)),
        ("edq (pair)", 5, lambda: B.edq(a, b, o0, o1, c, n, edq_dev, ws, stream)),
        ("edq (single)", 3, lambda: B.edq(a, None, o0, None, c, n, edq_dev, ws, stream)),
        ("edq_static (pair)", 5, lambda: B.edq_static(a, b, o0, o1, c, n, edq_dev, stream)),
    ]
    for name, arrays, call in cases:
        med, mean = _time_steps(torch, lambda i: call(), args.sweep_iters, stream)
        gbs = 2 * arrays * n / (med * 1e-3) / 1e9
        print(json.dumps({"primitive": name, "n": n, "arrays_moved": arrays, "ms": med, "hbm_gbs": gbs,
                          "frac_of_measured_peak": gbs / peak, "elements_per_sec": n / (med * 1e-3)}), flush=True)


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
    # config 0 whole: 2^20 parameters, 10 steps each of options A, B, C
    n0 = 1 << 20
    th0 = W.bits(W.flat_weights(n0, 0))
    c0 = time.perf_counter()
    for strategy in (0, 1, 2):
        z = lambda: np.zeros_like(th0)
        st0 = [th0.copy(), z() if strategy >= 1 else None, z(), z(), z() if strategy == 2 else None]
        for t0_ in range(1, 11):
            oracle.adamw_step(st0[0], st0[1], st0[2], st0[3], st0[4], W.bits(W.flat_grads(n0, 0, t0_)), step=t0_,
                              strategy=strategy, threads=threads, **W.HYPERS)
    c0 = time.perf_counter() - c0
    return {"value": done / el, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{t} Collage-plus steps over the first {n} parameters of the workload's embedding tensor "
                      f"({el:.1f} s)",
            "value_one_thread": n1 * t1 / e1, "sample_one_thread": f"{t1} steps over {n1} parameters ({e1:.1f} s)",
            "config0_whole": {"value": 30 * n0 / c0, "unit": UNIT, "seconds": c0,
                              "sample": "config 0 whole: 10 steps each of options A, B, C over 2^20 parameters "
                                        "(gradient generation included)"}}


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
    ap.add_argument("--sweep-iters", type=int, default=40, help="--strategy-sweep / --primitive-sweep: timed launches per case")
    ap.add_argument("--config", type=int, default=3, choices=[0, 1, 2, 3, 4],
                    help="synthetic configuration to time (3 = the LLaMA-7B-shaped headline; 4 = the size sweep)")
    ap.add_argument("--primitive-sweep", action="store_true", help="time the batched primitives and the stand-alone EDQ")
    ap.add_argument("--lib", default=None, help="another build of the library (build.py --out), e.g. the data-movement-only build")
    ap.add_argument("--pin-kernel", default="auto", choices=["auto", "pipeline", "large"],
                    help="headline step: kernel as chosen by size, or pin the three-stage / the large-tile pipeline (A/B runs)")
    ap.add_argument("--no-sharded", action="store_true", help="N > 1: skip the sharded-step record")
    ap.add_argument("--sharded-only", action="store_true", help="(internal) run only the sharded step, under torchrun")
    ap.add_argument("--sharded-selfcheck", action="store_true", help="the sharded flow with two emulated ranks on one GPU")
    ap.add_argument("--sharded-backend", default="nccl", choices=["nccl", "gloo"], help="--sharded-only: how the EDQ sums travel")
    ap.add_argument("--sharded-one-device", action="store_true",
                    help="--sharded-only test mode: all ranks are separate processes on device 0 (use with --sharded-backend gloo)")
    args = ap.parse_args()
    if args.sharded_only:
        run_sharded_only(args)
    elif args.sharded_selfcheck:
        run_sharded_selfcheck(args)
    elif args.primitive_sweep:
        run_primitive_sweep(args)
    elif args.size_sweep or (args.config == 4 and args.impl == "collage"):
        run_size_sweep(args)
    elif args.strategy_sweep:
        run_strategy_sweep(args)
    elif args.impl == "collage" and args.config == 0:
        run_config0(args)
    elif args.impl == "collage" and args.config == 1:
        run_config1(args)
    elif args.impl == "collage" and args.config == 2:
        run_config2(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_collage(args)


if __name__ == "__main__":
    main()
