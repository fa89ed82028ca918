"""Host-side logic for running the step on several GPUs: who owns which parameters, and how EDQ is combined.

Every parameter is independent, so ranks own disjoint contiguous slices of the concatenated
parameter space (optimizer-state ownership, no data-path exchange).  The only cross-parameter
quantity is EDQ (Eq. 3), whose two sums -- and the lost-update count -- are added over ranks.
"""
from __future__ import annotations

import math


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
    """Add {dot, sumsq, lost} over ranks in place (a 3-element float64 tensor) and form EDQ.

    `dist` is torch.distributed (NCCL on GPUs, gloo on CPU); None means a single process.
    """
    if dist is not None and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(sums, group=group)
    dot, sumsq, lost = (float(x) for x in sums.tolist())
    return dict(dot=dot, sumsq=sumsq, edq=dot / math.sqrt(sumsq) if sumsq > 0 else 0.0, lost=int(round(lost)))
