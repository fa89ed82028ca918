"""CPU checks of the C-ABI boundary: the library loads, exports what the header declares, derives the
step's scalars exactly as the oracle does, and rejects bad arguments before touching CUDA."""
import ctypes
import re
from pathlib import Path

import pytest

import oracle
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import build as builder

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def L():
    builder.build()
    return B.lib()


def test_library_exports_every_declared_symbol(L):
    header = (ROOT / "include" / "collage.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(collage_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations parsed"
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(B.Hyper) == 5 * 8 + 8 + 3 * 8        # flags padded to 8
    assert ctypes.sizeof(B.Edq) == 48 == B.EDQ_RECORD_BYTES
    assert ctypes.sizeof(B.Tensor) == 56
    assert B.workspace_bytes(0) == B.workspace_bytes(1 << 40) > 0


@pytest.mark.parametrize("hyp", [
    dict(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1),
    dict(lr=1.2e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1),
    dict(lr=3e-3, beta1=0.8, beta2=0.98, eps=1e-6, weight_decay=0.0),
    dict(lr=2e-5, beta1=0.0, beta2=0.99, eps=1e-12, weight_decay=1e-2),
])
def test_scalars_equal_the_oracles_bit_for_bit(L, hyp):
    h = B.make_hyper(**hyp)
    steps = list(range(1, 3000)) + list(range(3000, 100_001, 97)) + [10 ** 6, 10 ** 9]
    for t in steps:
        got = B.derive_scalars(h, t)
        want = oracle.derive_scalars(hyp["lr"], hyp["beta1"], hyp["beta2"], hyp["eps"], hyp["weight_decay"], t)
        assert got == want, (t, got, want)


def test_host_rounder_equals_oracle_on_awkward_doubles(L):
    # drive the library's double->bfloat16 rounding through the lr slot (any finite value >= 0 is legal)
    import numpy as np
    rng = np.random.default_rng(1)
    vals = np.concatenate([
        np.ldexp(rng.uniform(1.0, 2.0, 20000), rng.integers(-140, 128, 20000)),
        np.ldexp(1.0 + (np.arange(0, 512) + 0.5) / 256.0, -3),             # exact midpoints
        np.ldexp(np.arange(0, 300) / 2.0, -133),                           # subnormal grid and its midpoints
        [0.0, 2.0 ** -134, 2.0 ** -135, 3.3895313892515355e38, 3.4e38, 1e39],
    ])
    for v in vals:
        h = B.make_hyper(float(v), 0.9, 0.999, 1e-8, 0.1)
        assert B.derive_scalars(h, 1)["a"] == oracle.round_to_bf16(float(v)), v


def test_argument_errors_are_reported_before_any_cuda_call(L):
    ok = B.make_hyper(1e-4, 0.9, 0.999, 1e-8, 0.1)
    dummy = 0x10000  # never dereferenced: every call below must fail validation first
    call = lambda **kw: L.collage_adamw_step(kw.get("x_hi", dummy), kw.get("x_lo", None), kw.get("m", dummy * 2),
                                             kw.get("v_hi", dummy * 3), kw.get("v_lo", None), kw.get("grad", dummy * 4),
                                             kw.get("n", 16), ctypes.byref(kw.get("hyper", ok)), kw.get("step", 1),
                                             kw.get("strategy", B.BF16), None)
    assert L.collage_adamw_step(dummy, None, dummy, dummy, None, dummy, 16, None, 1, 0, None) == B.ERR_NULL
    assert call(step=0) == B.ERR_ARG
    assert call(strategy=5) == B.ERR_ARG
    assert call(strategy=B.KAHAN) == B.ERR_NULL                      # the compensation array is missing
    assert call(strategy=-1) == B.ERR_ARG
    for bad in (dict(lr=-1.0), dict(beta1=1.0), dict(beta2=1.5), dict(eps=float("nan")), dict(weight_decay=float("inf"))):
        kw = dict(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
        kw.update(bad)
        assert call(hyper=B.make_hyper(**kw)) == B.ERR_ARG
    assert call(hyper=B.make_hyper(1e-4, 0.9, 0.999, 1e-8, 0.1, flags=64)) == B.ERR_ARG
    both = B.FLAG_PIPELINE_KERNEL | B.FLAG_DIRECT_KERNEL                      # contradictory kernel choice
    assert call(hyper=B.make_hyper(1e-4, 0.9, 0.999, 1e-8, 0.1, flags=both)) == B.ERR_ARG
    assert call(hyper=B.make_hyper(1e-4, 0.9, 0.999, 1e-8, 0.1, flags=B.FLAG_LARGE_TILES | B.FLAG_PIPELINE_KERNEL)) == B.ERR_ARG
    # variant flags only where they mean something
    assert call(hyper=B.make_hyper(1e-4, 0.9, 0.999, 1e-8, 0.1, flags=B.FLAG_TWOSUM_GROW)) == B.ERR_ARG      # option A
    kahan_bad = B.make_hyper(1e-4, 0.9, 0.999, 1e-8, 0.1, flags=B.FLAG_DECAY_BY_GROW)
    assert call(strategy=B.KAHAN, x_lo=dummy * 5, hyper=kahan_bad) == B.ERR_ARG
    assert call(x_hi=None) == B.ERR_NULL
    assert call(grad=None) == B.ERR_NULL
    assert call(strategy=B.LIGHT) == B.ERR_NULL                      # x_lo missing
    assert call(strategy=B.PLUS, x_lo=dummy * 5) == B.ERR_NULL       # v_lo missing
    assert call(strategy=B.BF16, x_lo=dummy * 5) == B.ERR_ARG        # component the strategy does not use
    assert call(m=dummy + 8) == B.ERR_ALIAS                          # m overlaps x_hi
    assert call(grad=dummy * 3 + 30) == B.ERR_ALIAS                  # grad overlaps the tail of v_hi
    # EDQ requested without workspace
    h = B.make_hyper(1e-4, 0.9, 0.999, 1e-8, 0.1)
    h.edq_out = dummy * 7
    assert call(hyper=h) == B.ERR_WORKSPACE
    h.workspace, h.workspace_bytes = dummy * 8, 16
    assert call(hyper=h) == B.ERR_WORKSPACE
    # the record and the workspace may overlap neither a tensor nor each other
    big = B.workspace_bytes()
    h.workspace, h.workspace_bytes = dummy * 8, big
    h.edq_out = dummy + 8                                              # inside x_hi
    assert call(hyper=h) == B.ERR_ALIAS
    h.edq_out, h.workspace = dummy * 7, dummy * 3 - 64                 # workspace runs into v_hi
    assert call(hyper=h) == B.ERR_ALIAS
    h.edq_out, h.workspace = dummy * 8 + 4096, dummy * 8               # record inside the workspace
    assert call(hyper=h) == B.ERR_ALIAS
    h.edq_out, h.workspace = dummy * 7 + 4, dummy * 8                  # a record of doubles must be 8-byte aligned
    assert call(hyper=h) == B.ERR_ARG
    assert L.collage_workspace_init(None, big, None) == B.ERR_NULL
    assert L.collage_workspace_init(dummy, 16, None) == B.ERR_WORKSPACE
    assert L.collage_workspace_init(dummy + 4, big, None) == B.ERR_WORKSPACE
    # derive_scalars
    out = (ctypes.c_uint16 * 11)()
    assert L.collage_derive_scalars(None, 1, out) == B.ERR_NULL
    assert L.collage_derive_scalars(ctypes.byref(ok), 0, out) == B.ERR_ARG
    # primitives: NULL, unknown op, partial overlap
    assert L.collage_grow(dummy, dummy * 2, None, dummy * 3, dummy * 4, 8, None) == B.ERR_NULL
    assert L.collage_rounded_op(9, dummy, dummy * 2, None, dummy * 3, 8, None) == B.ERR_ARG
    assert L.collage_fast_two_sum(dummy, dummy * 2, dummy + 2, dummy * 3, 8, None) == B.ERR_ALIAS
    assert L.collage_fast_two_sum(dummy, dummy * 2, dummy * 3, dummy * 3, 8, None) == B.ERR_ALIAS
    # plan: bad chunk size, NULL member, overlap between two tensors
    plan = ctypes.c_void_p()
    t = (B.Tensor * 2)(B.Tensor(dummy, None, dummy * 2, dummy * 3, None, dummy * 4, 64),
                       B.Tensor(dummy * 5, None, dummy * 6, dummy * 7, None, dummy * 8, 64))
    assert L.collage_plan_create(t, 2, 1000, ctypes.byref(plan)) == B.ERR_ARG
    assert L.collage_plan_create(t, -1, 0, ctypes.byref(plan)) == B.ERR_ARG
    assert L.collage_plan_create(t, 2, 0, None) == B.ERR_NULL
    t[1].m = None
    assert L.collage_plan_create(t, 2, 0, ctypes.byref(plan)) == B.ERR_NULL
    t[1].m = dummy + 64
    assert L.collage_plan_create(t, 2, 0, ctypes.byref(plan)) == B.ERR_ALIAS
    assert L.collage_adamw_step_multi(None, ctypes.byref(ok), 1, 0, None) == B.ERR_NULL
    assert L.collage_plan_destroy(None) == B.OK
    for s in range(8):
        assert B.status_string(s)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_lib_path", tmp_path / "absent.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.lib()


def test_no_environment_variable_selects_the_library(monkeypatch, tmp_path):
    # the library that runs is the in-tree build unless load(path) is called; load() after first use is refused
    monkeypatch.setenv("COLLAGE_B200_LIB", str(tmp_path / "elsewhere.so"))
    assert B.lib()._name == str(ROOT / "paper_2405_03637_b200" / "libcollage_b200.so")
    assert B.build_flavor() == "product"
    with pytest.raises(RuntimeError, match="already loaded"):
        B.load(tmp_path / "elsewhere.so")


def test_edq_combine_is_equation_3_on_the_summed_partial_sums(L):
    # records of disjoint slices of one step, as ranks or tensors would hold them, against the oracle's sums
    # over the whole array; the quotient is taken by the library, on the host, with no CUDA call
    import numpy as np
    from paper_2405_03637_b200 import workloads as W
    n = 50_000
    th = W.bits(W.flat_weights(n, 40)); g = W.bits(W.flat_grads(n, 40, 1))
    hyp = dict(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
    z = lambda: np.zeros(n, np.uint16)
    whole_state = [th.copy(), z(), z(), z()]
    whole, _ = oracle.adamw_step(whole_state[0], None, whole_state[1], whole_state[2], None, g, step=1, strategy=0, **hyp)
    cuts, parts = [0, 7, 12_345, 12_345, 40_000, n], []
    for lo, hi in zip(cuts, cuts[1:]):
        st = [th[lo:hi].copy(), np.zeros(hi - lo, np.uint16), np.zeros(hi - lo, np.uint16)]
        s, _ = oracle.adamw_step(st[0], None, st[1], st[2], None, g[lo:hi].copy(), step=1, strategy=0, **hyp)
        parts.append(dict(s, n=hi - lo))
    got = B.edq_combine(parts)
    assert got["n"] == n and got["lost"] == whole["lost"] and got["fault"] == 0
    assert got["dot"] == pytest.approx(whole["dot"], rel=1e-12) and got["sumsq"] == pytest.approx(whole["sumsq"], rel=1e-12)
    assert got["edq"] == pytest.approx(whole["edq"], rel=1e-12)
    assert got["edq"] == got["dot"] / np.sqrt(got["sumsq"])
    # fixed order: the sums are those of a left-to-right addition
    d = 0.0
    for p in parts:
        d += p["dot"]
    assert got["dot"] == d
    assert B.edq_combine([]) == dict(dot=0.0, sumsq=0.0, edq=0.0, n=0, lost=0, fault=0)
    assert B.edq_combine([dict(dot=1.0, sumsq=0.0, lost=0)])["edq"] == 0.0                     # zero norm: EDQ is 0
    assert B.edq_combine([dict(dot=0.0, sumsq=1.0, lost=0, fault=0), dict(dot=0.0, sumsq=1.0, lost=0, fault=41)])["fault"] == 41
    assert L.collage_edq_combine(None, 1, ctypes.byref(B.Edq())) == B.ERR_NULL
    assert L.collage_edq_combine(None, 0, None) == B.ERR_NULL
    assert L.collage_edq_combine(None, -1, ctypes.byref(B.Edq())) == B.ERR_ARG
