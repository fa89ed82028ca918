"""World-size-2 run on CPU (gloo): rank partition of the parameter space and the EDQ all-reduce.

The CUDA kernels cannot run here; each rank steps its slice with the oracle, which is what the
GPU path is proven bit-identical to.  What this test covers is the host logic: the partition is a
disjoint cover that keeps alignment, and summing the per-rank EDQ sums reproduces the global EDQ.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2405_03637_b200 import sharding
from paper_2405_03637_b200 import workloads as W


def test_partition_is_an_aligned_disjoint_cover():
    sizes = [s for _, s in W.ragged_shapes()] + [s for _, s in W.gpt2_small_shapes()[:20]]
    total = sum(sizes)
    for world in (1, 2, 3, 4, 8):
        parts = sharding.partition(sizes, world)
        assert len(parts) == world
        seen = [np.zeros(s, dtype=np.int8) for s in sizes]
        loads = []
        for ranges in parts:
            loads.append(sum(e - b for _, b, e in ranges))
            for i, b, e in ranges:
                assert 0 <= b < e <= sizes[i]
                assert b % 8 == 0                       # a slice starts on a 16-byte boundary of its tensor
                seen[i][b:e] += 1
        assert all((s == 1).all() for s in seen)        # every element owned exactly once
        assert sum(loads) == total
        assert max(loads) - min(loads) <= 8 * world + max(8, total // 10 ** 6)
    assert sharding.partition([], 2) == [[], []]
    with pytest.raises(ValueError):
        sharding.partition([8], 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, sizes, out_q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        hyp, strategy = W.HYPERS, 2
        mine = sharding.partition(sizes, world)[rank]
        sums = torch.zeros(3, dtype=torch.float64)
        state = {}
        for t in (1, 2):
            step_sums = torch.zeros(3, dtype=torch.float64)
            for i, b, e in mine:
                if (i, b) not in state:
                    theta = W.bits(W.flat_weights(sizes[i], 700 + i))[b:e].copy()
                    z = lambda: np.zeros_like(theta)
                    state[(i, b)] = [theta, z(), z(), z(), z()]
                g = W.bits(W.flat_grads(sizes[i], 700 + i, t))[b:e]
                st = state[(i, b)]
                s, _ = oracle.adamw_step(st[0], st[1], st[2], st[3], st[4], g, step=t, strategy=strategy, **hyp)
                step_sums += torch.tensor([s["dot"], s["sumsq"], float(s["lost"])], dtype=torch.float64)
            sums = step_sums
            got = sharding.allreduce_edq(sums, dist)
        checksum = sum(int(st[0].astype(np.uint64).sum() + st[1].astype(np.uint64).sum()) for st in state.values())
        out_q.put((rank, got, checksum))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_global_edq():
    sizes = [50_001, 4096, 9, 120_000]
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, sizes, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # single-process reference over the whole parameter set
    tot = dict(dot=0.0, sumsq=0.0, lost=0)
    checksum = 0
    for i, n in enumerate(sizes):
        theta = W.bits(W.flat_weights(n, 700 + i))
        st = [theta, np.zeros_like(theta), np.zeros_like(theta), np.zeros_like(theta), np.zeros_like(theta)]
        for t in (1, 2):
            s, _ = oracle.adamw_step(st[0], st[1], st[2], st[3], st[4], W.bits(W.flat_grads(n, 700 + i, t)), step=t,
                                     strategy=2, **W.HYPERS)
        tot["dot"] += s["dot"]; tot["sumsq"] += s["sumsq"]; tot["lost"] += s["lost"]
        checksum += int(st[0].astype(np.uint64).sum() + st[1].astype(np.uint64).sum())
    want_edq = tot["dot"] / np.sqrt(tot["sumsq"])
    for rank, got, _ in results:
        assert got["edq"] == pytest.approx(want_edq, rel=1e-12)      # both ranks hold the same global value
        assert got["lost"] == tot["lost"]
    assert sum(c for _, _, c in results) == checksum                  # the slices together are the whole state


def _as_u16(t):
    """numpy uint16 view of a CPU bfloat16 tensor (shares its memory)."""
    return t.view(torch.int16).numpy().view(np.uint16)


def _harness_rank(rank, world, port, sizes, copies, out_q):
    # the benchmark's sharded flow on CPU: the same ShardedRank (partition, plan rows, replica table) and the
    # same all-reduce helper; the oracle steps the rows, and a plain copy into the peers' shared-memory theta
    # stands in for the step kernel's replica stores
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        hyp, strategy = W.HYPERS, 2
        alloc = lambda n: torch.zeros(n, dtype=torch.bfloat16)
        shard = sharding.ShardedRank(sizes, rank, world, copies, alloc, strategy)
        assert len(shard.replicas) == world - 1 and all(len(rep) == len(shard.rows) for rep in shard.replicas)
        assert shard.gathered_bytes_per_step() == 2 * shard.elements * (world - 1)
        for t in (1, 2):
            sums = torch.zeros(3, dtype=torch.float64)
            for k, ((i, b, e), row) in enumerate(zip(shard.ranges, shard.rows)):
                g = W.bits(W.flat_grads(sizes[i], 700 + i, t))[b:e]
                x_hi, x_lo, m, v_hi, v_lo = (_as_u16(a) for a in row[:5])
                s, _ = oracle.adamw_step(x_hi, x_lo, m, v_hi, v_lo, g, step=t, strategy=strategy, **hyp)
                sums += torch.tensor([s["dot"], s["sumsq"], float(s["lost"])], dtype=torch.float64)
                for rep in shard.replicas:                       # theta of the slice goes to every peer's copy
                    rep[k].copy_(row[0])
            got = sharding.allreduce_edq(sums, dist)             # also the point after which every copy is complete
            dist.barrier()
        out_q.put((rank, got, sharding.theta_checksum(copies[rank], torch)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_drive_the_sharded_harness_with_the_oracle_as_stepper():
    sizes = [50_001, 4096, 9, 120_000, 8]
    world = 2
    theta = [W.flat_weights(n, 700 + i) for i, n in enumerate(sizes)]
    copies = [[t.clone().share_memory_() for t in theta] for _ in range(world)]     # each rank's full copy of theta
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_harness_rank, args=(r, world, port, sizes, copies, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=180) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the unsharded step over the whole set
    tot, full = dict(dot=0.0, sumsq=0.0, lost=0), []
    for i, n in enumerate(sizes):
        st = [W.bits(theta[i]), *(np.zeros(n, np.uint16) for _ in range(4))]
        for t in (1, 2):
            s, _ = oracle.adamw_step(st[0], st[1], st[2], st[3], st[4], W.bits(W.flat_grads(n, 700 + i, t)), step=t,
                                     strategy=2, **W.HYPERS)
        tot["dot"] += s["dot"]; tot["sumsq"] += s["sumsq"]; tot["lost"] += s["lost"]
        full.append(st[0])
    for r in range(world):                                            # every rank's copy holds the whole new theta
        for i in range(len(sizes)):
            assert np.array_equal(_as_u16(copies[r][i]), full[i]), (r, i)
    want = sharding.theta_checksum([W.from_bits(f) for f in full], torch)
    for rank, got, checksum in results:
        assert checksum == want
        assert got["edq"] == pytest.approx(tot["dot"] / np.sqrt(tot["sumsq"]), rel=1e-12) and got["lost"] == tot["lost"]


def test_slices_of_all_ranks_tile_every_tensor_and_keep_alignment():
    sizes = [4096, 9, 100_003, 0, 65_536]
    rows = []
    for n in sizes:
        ts = [torch.arange(n, dtype=torch.int32).to(torch.bfloat16) for _ in range(6)]
        rows.append(tuple(ts) + (n,))
    world = 3
    parts = sharding.partition(sizes, world)
    covered = [torch.zeros(n, dtype=torch.int32) for n in sizes]
    for rank in range(world):
        mine = sharding.slice_rows(rows, parts[rank])
        reps = sharding.replica_rows([[r[0] for r in rows]], parts[rank])
        assert len(mine) == len(parts[rank]) == len(reps[0])
        for (i, b, e), row, rep in zip(parts[rank], mine, reps[0]):
            assert row[6] == e - b and all(t.numel() == e - b for t in row[:6])
            assert row[0].data_ptr() == rows[i][0].data_ptr() + 2 * b          # a view, not a copy
            assert (row[0].data_ptr() - rows[i][0].data_ptr()) % 16 == 0        # alignment carried over
            assert rep.data_ptr() == row[0].data_ptr()
            covered[i][b:e] += 1
    assert all(bool((c == 1).all()) for c in covered)
