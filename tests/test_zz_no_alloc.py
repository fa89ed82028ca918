"""GPU test of collage_edq_static, the EDQ entry point for callers that cannot allocate.

Some users of the library run where device allocation is off limits: all GPU memory already
belongs to a pool, or they are a plugin without access to the host framework's allocator.  The
entry point keeps its scratch in a fixed array inside the library instead of taking a workspace.
This file is collected last on purpose, so that a run stopping at the first failure has already
run every other test; the test itself does not depend on what ran before it.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from conftest import bf16_window
from paper_2405_03637_b200 import binding as B

pytestmark = pytest.mark.gpu


def _inputs(n, seed):
    rng = np.random.default_rng(seed)
    old_hi = rng.choice(bf16_window(-8, 0), n)
    old_lo = rng.choice(bf16_window(-20, -10, with_zero=True), n)
    delta = rng.choice(bf16_window(-16, -9, with_zero=True), n)
    new_hi, new_lo = oracle.grow(old_hi, old_lo, delta)
    new_hi[::5] = old_hi[::5]
    new_lo[::5] = old_lo[::5]                                   # some updates lost entirely
    to_dev = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).cuda()
    host = (old_hi, old_lo, new_hi, new_lo, delta)
    return [to_dev(a) for a in host], host


def _close(got, want):
    for k in ("dot", "sumsq", "edq"):
        assert abs(got[k] - want[k]) <= 1e-5 * abs(want[k]) + 1e-300, (k, got[k], want[k])
    assert got["lost"] == want["lost"] and got["n"] == want["n"]


def test_static_scratch_matches_workspace_version_on_two_calls_in_a_row():
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device="cuda")
    ref_out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    # two different problems back to back through the one shared array: the second call must not see
    # anything of the first (a larger problem first, so stale partial sums would be left behind)
    for n, seed, with_lo in [(5_000_003, 1, True), (2_097_153, 2, False)]:
        (old_hi, old_lo, new_hi, new_lo, delta), host = _inputs(n, seed)
        lo_args = (old_lo, new_lo) if with_lo else (None, None)
        B.edq(old_hi, lo_args[0], new_hi, lo_args[1], delta, n, ref_out, ws)
        B.edq_static(old_hi, lo_args[0], new_hi, lo_args[1], delta, n, out)
        torch.cuda.synchronize()
        _close(B.read_edq(out), B.read_edq(ref_out))
        # and against the CPU oracle directly (Eq. 2-3 in double, index order)
        want = oracle.edq(host[0], host[1] if with_lo else None, host[2], host[3] if with_lo else None, host[4])
        _close(B.read_edq(out), dict(want, n=n))
    # same inputs again: identical result (deterministic, nothing carried over)
    first = B.read_edq(out)
    B.edq_static(old_hi, None, new_hi, None, delta, n, out)
    torch.cuda.synchronize()
    assert B.read_edq(out) == first
    # misaligned views and an empty input
    B.edq(old_hi[1:], None, new_hi[1:], None, delta[1:], n - 1, ref_out, ws)
    B.edq_static(old_hi[1:], None, new_hi[1:], None, delta[1:], n - 1, out)
    torch.cuda.synchronize()
    _close(B.read_edq(out), B.read_edq(ref_out))
    B.edq_static(old_hi, None, new_hi, None, delta, 0, out)
    torch.cuda.synchronize()
    assert B.read_edq(out)["edq"] == 0.0 and B.read_edq(out)["n"] == 0


def test_calls_leave_the_amount_of_free_device_memory_unchanged():
    # what the entry point exists for: it takes no device memory.  The first call on a device looks the
    # scratch array's address up (and the CUDA runtime may load the library's code then); from the second
    # call on, free memory as the driver reports it is the same before and after any number of calls,
    # small and large, with and without second components.
    (old_hi, old_lo, new_hi, new_lo, delta), host = _inputs(3_000_001, 3)
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    B.edq_static(old_hi, old_lo, new_hi, new_lo, delta, 1000, out)
    B.edq_static(old_hi, None, new_hi, None, delta, 1000, out)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for n in (1, 2049, 300_000, 3_000_001):
        B.edq_static(old_hi, old_lo, new_hi, new_lo, delta, n, out)
        B.edq_static(old_hi, None, new_hi, None, delta, n, out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    want = oracle.edq(host[0], None, host[2], None, host[4])
    _close(B.read_edq(out), dict(want, n=3_000_001))


def test_sizes_beyond_the_capacity_are_rejected():
    z = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.CollageError) as err:
        B.edq_static(z, None, z, None, z, (1 << 32) + 1, out)        # rejected before anything is touched
    assert err.value.status == B.ERR_LIMIT
    assert "capacity" in B.status_string(B.ERR_LIMIT)
    with pytest.raises(B.CollageError) as err:
        B.edq_static(z, None, z, z, z, 64, out)                       # only one of the two low parts given
    assert err.value.status == B.ERR_NULL
