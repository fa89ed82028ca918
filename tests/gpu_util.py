"""Helpers of the GPU parity tests: guarded device buffers, bit comparison, oracle-side state."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2405_03637_b200 import binding as B

GUARD = 2048            # elements (4 KiB) of sentinel on each side of every test buffer
SENTINEL = 0x5A5A


class Guarded:
    """A bfloat16 device buffer of n elements with sentinel bands around it.

    `misalign` shifts the payload by that many elements (2 bytes each) off its 16-byte boundary.
    """

    def __init__(self, bits: np.ndarray, misalign: int = 0, device="cuda"):
        bits = np.ascontiguousarray(bits, dtype=np.uint16)
        self.n = bits.size
        self.lo = GUARD + misalign
        raw = np.full(self.n + 2 * GUARD + 8, SENTINEL, dtype=np.uint16)
        raw[self.lo:self.lo + self.n] = bits
        self.raw = torch.from_numpy(raw.view(np.int16)).to(device)
        self.t = self.raw[self.lo:self.lo + self.n].view(torch.bfloat16)

    def bits(self) -> np.ndarray:
        return self.t.view(torch.int16).cpu().numpy().view(np.uint16).copy()

    def guards_intact(self) -> bool:
        r = self.raw.cpu().numpy().view(np.uint16)
        return bool(np.all(r[:self.lo] == SENTINEL) and np.all(r[self.lo + self.n:] == SENTINEL))


def same_bits(got: np.ndarray, want: np.ndarray) -> np.ndarray:
    """Elementwise: identical bit patterns, NaNs compared as a class."""
    got = np.asarray(got, dtype=np.uint16)
    want = np.asarray(want, dtype=np.uint16)
    nan_g = ((got & 0x7F80) == 0x7F80) & ((got & 0x7F) != 0)
    nan_w = ((want & 0x7F80) == 0x7F80) & ((want & 0x7F) != 0)
    return (got == want) | (nan_g & nan_w)


def assert_same_bits(got, want, what=""):
    ok = same_bits(got, want)
    if not ok.all():
        bad = np.flatnonzero(~ok)
        i = int(bad[0])
        raise AssertionError(f"{what}: {bad.size} of {ok.size} elements differ; first at {i}: "
                             f"gpu {int(got[i]):04X} oracle {int(want[i]):04X}")


class EdqBuffers:
    """Device record + workspace for the fused EDQ reduction."""

    def __init__(self, device="cuda"):
        self.out = torch.zeros(64, dtype=torch.uint8, device=device)
        self.ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device=device)
        B.workspace_init(self.ws)                 # once; every step leaves it ready for the next

    def hyper(self, hyp: dict, flags=0) -> B.Hyper:
        return B.make_hyper(hyp["lr"], hyp["beta1"], hyp["beta2"], hyp["eps"], hyp["weight_decay"], flags,
                            edq_out=self.out, workspace=self.ws)

    def read(self) -> dict:
        return B.read_edq(self.out)


def oracle_state(theta_bits: np.ndarray, strategy: int) -> dict:
    z = lambda: np.zeros_like(theta_bits)
    return dict(x_hi=theta_bits.copy(), x_lo=z() if strategy >= 1 else None, m=z(), v_hi=z(),
                v_lo=z() if strategy == 2 else None)


def oracle_step(st: dict, g: np.ndarray, t: int, strategy: int, hyp: dict, flags=0, threads=None):
    threads = threads or oracle.max_threads()
    sums, _ = oracle.adamw_step(st["x_hi"], st["x_lo"], st["m"], st["v_hi"], st["v_lo"], g, step=t,
                                strategy=strategy, flags=flags, threads=threads, **hyp)
    return sums


def edq_close(got: dict, want: dict, rel=1e-5):
    for k in ("dot", "sumsq", "edq"):
        a, b = got[k], want[k]
        assert abs(a - b) <= rel * abs(b) + 1e-300, (k, a, b)
    assert got["lost"] == want["lost"], ("lost", got["lost"], want["lost"])


def resplit_pairs(update_bits: int):
    """Normalised pairs (x, y) on which Grow((x, y), update) returns the same value x + y split over other
    components: the parameter has not moved although both stored patterns changed.  Input selection only
    (expected results always come from the oracle's step); found by scanning windows with the oracle's Grow."""
    hi = np.concatenate([np.arange(0x3E80, 0x4080), np.arange(0xBE80, 0xC080)]).astype(np.uint16)
    lo = np.concatenate([np.arange(0x3900, 0x3C01), np.arange(0xB900, 0xBC01)]).astype(np.uint16)
    x, y = np.repeat(hi, lo.size), np.tile(lo, hi.size)
    f = lambda b: (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    ulp = np.ldexp(1.0, (((x >> 7) & 0xFF).astype(np.int32) - 127 - 7))
    ok = np.abs(f(y)) <= ulp / 2
    x, y = x[ok], y[ok]
    u, v = oracle.grow(x, y, np.full(x.size, update_bits, np.uint16))
    same_value = f(u) + f(v) == f(x) + f(y)            # exact in double: all terms within a few binades
    moved_bits = (f(u) != f(x)) | (f(v) != f(y))
    pick = same_value & moved_bits
    return x[pick], y[pick]
