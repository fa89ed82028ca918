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


def allreduce_edq(sums, dist=None, group=None) -> dict:
    """Add {dot, sumsq, lost} over ranks in place (a 3-element float64 tensor) and form EDQ.

    `dist` is torch.distributed (NCCL on GPUs, gloo on CPU); None means a single process.
    """
    if dist is not None and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(sums, group=group)
    dot, sumsq, lost = (float(x) for x in sums.tolist())
    return dict(dot=dot, sumsq=sumsq, edq=dot / math.sqrt(sumsq) if sumsq > 0 else 0.0, lost=int(round(lost)))
