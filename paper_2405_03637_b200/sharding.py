"""Host-side logic for running the step on several GPUs: who owns which parameters, and how EDQ is combined.

Every parameter is independent, so ranks own disjoint contiguous slices of the concatenated
parameter space (optimizer-state ownership, no data-path exchange).  The only cross-parameter
quantity is EDQ (Eq. 3), whose two sums -- and the lost-update count -- are added over ranks.
"""
from __future__ import annotations


def partition(sizes: list[int], world: int, align: int = 8) -> list[list[tuple[int, int, int]]]:
    """Split tensors of the given sizes over `world` ranks.

    Returns, per rank, a list of (tensor index, begin, end) element ranges.  Ranges of one rank are
    contiguous in the concatenated order; cut points inside a tensor are multiples of `align`
    elements from the tensor's start, so that 16-byte aligned tensors stay 16-byte aligned.
    Loads differ by less than `align` elements plus the rounding at tensor ends.
    """
    if world < 1 or align < 1:
        raise ValueError("world and align must be positive")
    total = sum(sizes)
    starts, acc = [], 0
    for s in sizes:
        starts.append(acc)
        acc += s
    cuts = [0]
    for r in range(1, world):
        target = total * r // world
        # locate the tensor holding `target` and round the cut down to the alignment inside it
        i = 0
        while i < len(sizes) and starts[i] + sizes[i] <= target:
            i += 1
        if i == len(sizes):
            cut = total
        else:
            inside = (target - starts[i]) // align * align
            cut = starts[i] + inside
        cuts.append(max(cut, cuts[-1]))
    cuts.append(total)
    out = []
    for r in range(world):
        lo, hi = cuts[r], cuts[r + 1]
        ranges = []
        for i, s in enumerate(sizes):
            b, e = max(lo, starts[i]), min(hi, starts[i] + s)
            if b < e:
                ranges.append((i, b - starts[i], e - starts[i]))
        out.append(ranges)
    return out


def slice_rows(rows, ranges):
    """Rows of a rank's own plan: the (x_hi, x_lo, m, v_hi, v_lo, grad, n) tuples of `rows` cut to `ranges`.

    `rows` are the full tensors (torch tensors or None); `ranges` is one rank's entry of `partition`.
    The result feeds `binding.plan_create`; element `begin` of a tensor stays 16-byte aligned whenever
    the tensor is, because `partition` cuts at multiples of 8 elements.
    """
    out = []
    for i, b, e in ranges:
        cut = tuple(None if t is None else t[b:e] for t in rows[i][:6])
        out.append(cut + (e - b,))
    return out


def replica_rows(peer_x_hi, ranges):
    """For `binding.plan_set_replicas`: this rank's slices inside each peer's full copy of theta.

    `peer_x_hi[r][i]` is tensor i of peer r's parameter copy, mapped into this process (its own memory for
    a single-GPU test; a peer-access or symmetric-memory mapping on several GPUs).  Returns one list per
    peer, aligned with `slice_rows(rows, ranges)`.
    """
    return [[peer[i][b:e] for i, b, e in ranges] for peer in peer_x_hi]


def allreduce_edq(sums, dist=None, group=None) -> dict:
    """Add {dot, sumsq, lost} over ranks in place (a 3-element float64 tensor); the library forms EDQ.

    `dist` is torch.distributed (NCCL on GPUs, gloo on CPU); None means a single process.  The
    quotient of Eq. 3 is taken by the library's `collage_edq_combine` on the summed record, not here.
    """
    from . import binding
    if dist is not None and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(sums, group=group)
    dot, sumsq, lost = (float(x) for x in sums.tolist())
    return binding.edq_combine([dict(dot=dot, sumsq=sumsq, lost=int(round(lost)))])


# --------------------------------------------------------------- harness ---
# One rank of the sharded step, independent of where the memory lives: the benchmark builds it on
# CUDA tensors (peer copies mapped through CUDA IPC), the CPU test on shared-memory CPU tensors with
# the oracle as the stepper.  The exchange pattern is the library's: a rank steps its slice and the
# new theta of that slice is stored into every rank's full copy; {dot, sumsq, lost} are all-reduced.

class ShardedRank:
    """State, plan rows and replica table of rank `rank` out of `world`.

    theta_copies[r][i] : tensor i of rank r's full copy of theta, as mapped into this process
                         (theta_copies[rank] is this rank's own copy; the others are peer memory)
    alloc(n)           : a zeroed bfloat16 tensor of n elements where this rank keeps optimizer state
    """

    def __init__(self, sizes, rank, world, theta_copies, alloc, strategy):
        self.sizes, self.rank, self.world, self.strategy = list(sizes), rank, world, strategy
        self.ranges = partition(self.sizes, world)[rank]
        full = [(theta_copies[rank][i], None, None, None, None, None) for i in range(len(self.sizes))]
        self.rows = []
        for (i, b, e), cut in zip(self.ranges, slice_rows(full, self.ranges)):
            n = e - b
            self.rows.append((cut[0], alloc(n) if strategy >= 1 else None, alloc(n), alloc(n),
                              alloc(n) if strategy in (2, 4) else None, alloc(n), n))
        peers = [theta_copies[r] for r in range(world) if r != rank]
        self.replicas = replica_rows(peers, self.ranges)
        self.elements = sum(r[6] for r in self.rows)

    def gathered_bytes_per_step(self) -> int:
        """Bytes this rank sends to peers per step: 2 B per owned parameter and peer."""
        return 2 * self.elements * (self.world - 1)


class CudaStepper:
    """Steps a ShardedRank with the library: one multi-tensor launch that also stores theta to the peers."""

    def __init__(self, shard: ShardedRank, torch):
        from . import binding
        self.B, self.shard, self.torch = binding, shard, torch
        device = shard.rows[0][0].device if shard.rows else torch.device("cuda")
        self.plan = binding.plan_create(shard.rows)
        if shard.replicas:
            binding.plan_set_replicas(self.plan, shard.replicas)
        self.record = torch.zeros(64, dtype=torch.uint8, device=device)
        self.workspace = torch.empty(binding.workspace_bytes(), dtype=torch.uint8, device=device)
        binding.workspace_init(self.workspace)
        # what ranks exchange: {dot, sumsq} as doubles and the lost count, views of the device record
        self.sums = self.record[:16].view(torch.float64)
        self.lost = self.record[32:40].view(torch.int64)

    def step(self, hyp: dict, t: int, stream=None):
        B = self.B
        B.adamw_step_multi(self.plan, B.make_hyper(**hyp, edq_out=self.record, workspace=self.workspace), t,
                           self.shard.strategy, stream)

    def allreduce(self, dist):
        """Sum the EDQ partial sums over ranks: on the device over NCCL (no host synchronisation), through
        host copies when the process group is gloo (CPU tests of the flow)."""
        if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
            if dist.get_backend() == "gloo":
                for t in (self.sums, self.lost):
                    h = t.cpu()
                    dist.all_reduce(h)
                    t.copy_(h)
            else:
                dist.all_reduce(self.sums)
                dist.all_reduce(self.lost)

    def read(self) -> dict:
        """The record after `allreduce`: Eq. 3 on the summed sums, formed by the library."""
        rec = self.B.read_edq(self.record)
        return self.B.edq_combine([dict(dot=rec["dot"], sumsq=rec["sumsq"], lost=rec["lost"], fault=rec["fault"])])

    def close(self):
        self.B.plan_destroy(self.plan)


def theta_checksum(copy, torch) -> int:
    """Order-independent digest of a full theta copy (sum of the bit patterns), to compare copies across ranks."""
    total = 0
    for t in copy:
        total += int(t.view(torch.int16).to(torch.int64).sum().item())
    return total
