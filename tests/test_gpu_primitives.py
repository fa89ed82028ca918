"""GPU parity of the single rounded operations and the batched MCF primitives against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from conftest import bf16_window
from gpu_util import Guarded, assert_same_bits
from paper_2405_03637_b200 import binding as B

pytestmark = pytest.mark.gpu


def _all_patterns():
    return np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)


def _edge_values():
    """Zeros, subnormals, smallest/largest normals, infinities, NaNs, and a dense middle window."""
    sub = np.arange(0x0000, 0x0100, dtype=np.uint16)
    top = np.arange(0x7F00, 0x7FC2, dtype=np.uint16)
    mid = bf16_window(-4, 4, signs=(0,))
    pos = np.unique(np.concatenate([sub, top, mid, bf16_window(-126, -124, signs=(0,)), bf16_window(61, 64, signs=(0,)),
                                    bf16_window(-64, -61, signs=(0,))]))
    return np.concatenate([pos, pos | np.uint16(0x8000)])


def _run_op(op, a, b=None, c=None):
    A = Guarded(a)
    Bv = Guarded(b) if b is not None else None
    C = Guarded(c) if c is not None else None
    out = Guarded(np.zeros_like(a))
    B.rounded_op(op, A.t, Bv.t if Bv else None, C.t if C else None, out.t, a.size)
    torch.cuda.synchronize()
    assert out.guards_intact() and A.guards_intact()
    return out.bits()


@pytest.mark.parametrize("op", [B.OP_ADD, B.OP_SUB, B.OP_MUL, B.OP_DIV])
def test_binary_ops_on_edge_grid(op):
    w = _edge_values()
    a, b = np.repeat(w, w.size), np.tile(w, w.size)
    assert_same_bits(_run_op(op, a, b), oracle.binary_op(op, a, b), f"op {op}")


@pytest.mark.parametrize("op", [B.OP_ADD, B.OP_SUB, B.OP_MUL, B.OP_DIV])
def test_binary_ops_random_over_all_patterns(op):
    rng = np.random.default_rng(100 + op)
    a = rng.integers(0, 65536, 1 << 24, dtype=np.uint32).astype(np.uint16)
    b = rng.integers(0, 65536, 1 << 24, dtype=np.uint32).astype(np.uint16)
    assert_same_bits(_run_op(op, a, b), oracle.binary_op(op, a, b), f"op {op}")


def test_division_all_significand_pairs_many_exponents():
    # every 128 x 128 significand pair, both signs, numerator and denominator exponents swept so that quotients
    # cover normal results, gradual underflow and overflow
    sig = np.arange(128, dtype=np.uint16)
    for ea, eb in [(0, 0), (1, 0), (0, 1), (-60, 60), (-63, 64), (-64, 64), (-100, 30), (60, -60), (64, -64),
                   (-126, 0), (-126, 7), (0, 126), (-126, 127), (127, -126), (-20, 3)]:
        a = np.repeat(((ea + 127) << 7) | sig, 128).astype(np.uint16)
        b = np.tile(((eb + 127) << 7) | sig, 128).astype(np.uint16)
        a = np.concatenate([a, a | np.uint16(0x8000)])
        b = np.concatenate([b, b])
        assert_same_bits(_run_op(B.OP_DIV, a, b), oracle.binary_op(oracle.OP_DIV, a, b), f"div e=({ea},{eb})")
    # subnormal numerators and denominators
    sub = np.arange(1, 128, dtype=np.uint16)
    norm = bf16_window(-126, -110, signs=(0,))
    for x, y in [(sub, sub), (sub, norm), (norm, sub), (sub, bf16_window(-3, 3, signs=(0,)))]:
        a, b = np.repeat(x, y.size), np.tile(y, x.size)
        assert_same_bits(_run_op(B.OP_DIV, a, b), oracle.binary_op(oracle.OP_DIV, a, b), "div subnormal")


def test_sqrt_every_pattern():
    a = _all_patterns()
    assert_same_bits(_run_op(B.OP_SQRT, a), oracle.binary_op(oracle.OP_SQRT, a), "sqrt")


def test_fma_random_and_two_prod_shape():
    rng = np.random.default_rng(7)
    w = _edge_values()
    a, b, c = (rng.choice(w, 1 << 23) for _ in range(3))
    assert_same_bits(_run_op(B.OP_FMA, a, b, c), oracle.binary_op(oracle.OP_FMA, a, b, c), "fma edge")
    a, b, c = (rng.integers(0, 65536, 1 << 23, dtype=np.uint32).astype(np.uint16) for _ in range(3))
    assert_same_bits(_run_op(B.OP_FMA, a, b, c), oracle.binary_op(oracle.OP_FMA, a, b, c), "fma random")
    # the form TwoProdFMA uses: c = -(a (*) b), all significand pairs
    w = np.concatenate([bf16_window(e, e) for e in (-40, -1, 0, 2, 40)])
    a, b = np.repeat(w, w.size), np.tile(w, w.size)
    c = oracle.binary_op(oracle.OP_MUL, a, b) ^ np.uint16(0x8000)
    assert_same_bits(_run_op(B.OP_FMA, a, b, c), oracle.binary_op(oracle.OP_FMA, a, b, c), "fma residual")


def _prim_inputs(k, n, seed):
    rng = np.random.default_rng(seed)
    w = np.concatenate([bf16_window(-14, 6, with_zero=True), np.arange(0, 64, dtype=np.uint16),
                        bf16_window(-126, -122), bf16_window(120, 127)])
    return [rng.choice(w, n) for _ in range(k)]


PRIMS = [
    ("fast_two_sum", 2, B.fast_two_sum, oracle.fast_two_sum),
    ("two_sum", 2, B.two_sum, oracle.two_sum),
    ("two_prod", 2, B.two_prod, oracle.two_prod),
    ("renormalize", 2, B.renormalize, oracle.renormalize),
    ("grow", 3, B.grow, oracle.grow),
    ("scaling", 3, B.scaling, oracle.scaling),
    ("mul", 4, B.mul, oracle.mul),
]


@pytest.mark.parametrize("name,k,gpu_fn,cpu_fn", PRIMS, ids=[p[0] for p in PRIMS])
@pytest.mark.parametrize("n,misalign", [(1 << 22, 0), (100_003, 0), (4097, 3), (7, 1), (1, 0)])
def test_primitives_match_oracle(name, k, gpu_fn, cpu_fn, n, misalign):
    ins = _prim_inputs(k, n, seed=hash(name) % 1000 + n)
    dev = [Guarded(a, misalign) for a in ins]
    o1, o2 = Guarded(np.zeros(n, np.uint16), misalign), Guarded(np.zeros(n, np.uint16), misalign)
    gpu_fn(*[d.t for d in dev], o1.t, o2.t, n)
    torch.cuda.synchronize()
    w1, w2 = cpu_fn(*ins)
    assert_same_bits(o1.bits(), w1, f"{name} first")
    assert_same_bits(o2.bits(), w2, f"{name} second")
    assert all(d.guards_intact() for d in dev + [o1, o2])
    assert all(np.array_equal(d.bits(), a) for d, a in zip(dev, ins))      # inputs untouched


def test_primitives_exhaustive_window_pairs():
    # every ordered pair of a 13-binade window with zeros: Fast2Sum, TwoSum, TwoProd
    w = bf16_window(-6, 6, with_zero=True)
    a, b = np.repeat(w, w.size), np.tile(w, w.size)
    for name, _, gpu_fn, cpu_fn in PRIMS[:3]:
        A, Bv = Guarded(a), Guarded(b)
        o1, o2 = Guarded(np.zeros_like(a)), Guarded(np.zeros_like(a))
        gpu_fn(A.t, Bv.t, o1.t, o2.t, a.size)
        torch.cuda.synchronize()
        w1, w2 = cpu_fn(a, b)
        assert_same_bits(o1.bits(), w1, name)
        assert_same_bits(o2.bits(), w2, name)


def test_outputs_may_be_the_inputs():
    n = 50_001
    x, y, a = _prim_inputs(3, n, 5)
    X, Y, A = Guarded(x), Guarded(y), Guarded(a)
    B.grow(X.t, Y.t, A.t, X.t, Y.t, n)
    torch.cuda.synchronize()
    u, v = oracle.grow(x, y, a)
    assert_same_bits(X.bits(), u, "grow in place u")
    assert_same_bits(Y.bits(), v, "grow in place v")
    assert X.guards_intact() and Y.guards_intact()


def test_empty_input_is_a_no_op():
    z = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    B.grow(z, z, z, z, z.clone(), 0)
    B.rounded_op(B.OP_ADD, z, z, None, z.clone(), 0)
    torch.cuda.synchronize()


def test_standalone_edq_matches_oracle():
    n = 1_000_003
    rng = np.random.default_rng(3)
    w = bf16_window(-8, 0)
    old_hi = rng.choice(w, n)
    old_lo = rng.choice(bf16_window(-20, -10, with_zero=True), n)
    delta = rng.choice(bf16_window(-16, -9, with_zero=True), n)
    new_hi, new_lo = oracle.grow(old_hi, old_lo, delta)
    new_hi[::7] = old_hi[::7]; new_lo[::7] = old_lo[::7]            # some lost updates
    # and some where Grow re-splits the same value over other components: not updated either (value reading)
    from gpu_util import resplit_pairs
    xs, ys = resplit_pairs(0x35AB)
    kp = np.arange(3, n, 13)
    old_hi[kp], old_lo[kp], delta[kp] = xs[kp % xs.size], ys[kp % xs.size], 0x35AB
    new_hi[kp], new_lo[kp] = oracle.grow(old_hi[kp], old_lo[kp], delta[kp])
    assert np.all((new_hi[kp] != old_hi[kp]) | (new_lo[kp] != old_lo[kp]))
    dev = [Guarded(a, 1) for a in (old_hi, old_lo, new_hi, new_lo, delta)]
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device="cuda")
    for has_lo in (True, False):
        args = [d.t for d in dev]
        if not has_lo:
            args[1] = args[3] = None
        B.edq(*args, n, out, ws)
        torch.cuda.synchronize()
        got = B.read_edq(out)
        want = oracle.edq(old_hi, old_lo if has_lo else None, new_hi, new_lo if has_lo else None, delta)
        for k in ("dot", "sumsq", "edq"):
            assert abs(got[k] - want[k]) <= 1e-5 * abs(want[k])
        assert got["lost"] == want["lost"] and got["n"] == n
        if has_lo:
            assert got["lost"] >= kp.size                      # every planted pair is counted


def test_standalone_edq_past_2_to_32_elements_is_the_sum_of_its_pieces():
    # index arithmetic past 32 bits: the sums over 2^32 + 4,099 parameters equal those of two pieces taken by
    # the same entry point (each piece below 2^32; small n is compared with the oracle above)
    from paper_2405_03637_b200 import workloads as W
    n = (1 << 32) + 4_099
    old = W.normal_bf16(n, 0.02, 811, "cuda")
    delta = W.normal_bf16(n, 1e-4, 812, "cuda")
    new = old + delta
    new[5::11] = old[5::11]                                          # lost updates on both sides of 2^32
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    ws = torch.empty(B.workspace_bytes(), dtype=torch.uint8, device="cuda")

    def run(lo, hi):
        B.edq(old[lo:hi], None, new[lo:hi], None, delta[lo:hi], hi - lo, out, ws)
        torch.cuda.synchronize()
        return B.read_edq(out)

    whole, cut = run(0, n), (1 << 31) + 8
    a, b = run(0, cut), run(cut, n)
    assert whole["n"] == n and a["n"] + b["n"] == n
    assert whole["lost"] == a["lost"] + b["lost"] and whole["lost"] >= n // 11
    for k in ("dot", "sumsq"):
        assert abs(whole[k] - (a[k] + b[k])) <= 1e-9 * abs(whole[k])
    del old, new, delta
    torch.cuda.empty_cache()


def test_selftest_every_operand_pair():
    # all 2^32 operand pairs on the device: native packed ops and the reciprocal/root shortcuts vs IEEE references
    assert B.selftest() == dict(add=0, sub=0, mul=0, div=0, sqrt=0, scalar_div=0)
