"""ctypes front end of the CPU oracle (``collage_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU
baseline leg load this; the CUDA library and its Python binding never do, and
nothing here imports them.  All arrays are numpy ``uint16`` holding bfloat16
bit patterns; the functions cite the passage of the paper they follow in the
C++ source.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "collage_oracle.cpp"
_LIB = _HERE / "liboracle_collage.so"

STRATEGY_BF16 = 0   # option A
STRATEGY_LIGHT = 1  # option B
STRATEGY_PLUS = 2   # option C
STRATEGY_KAHAN = 3  # BF16-Kahan comparator (Appendix B): x_lo holds the compensation c
FLAG_EPS_INSIDE_SQRT = 1
FLAG_TWOSUM_GROW = 2     # parameter Grow built on TwoSum (Appendix C)
FLAG_DECAY_BY_GROW = 4   # weight decay applied by an addition of its own (Appendix D)

OP_ADD, OP_SUB, OP_MUL, OP_DIV, OP_SQRT, OP_FMA = range(6)

SCALAR_NAMES = ("b1", "c1", "b2", "c2", "b2h", "b2l", "bc1", "bc2", "a", "lam", "eps")


def build(force: bool = False) -> Path:
    """Compile the oracle with g++ (OpenMP) if the library is missing or stale."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
             "-o", str(tmp), str(_SRC)])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.oracle_round_to_bf16.restype = ctypes.c_uint16
        _lib.oracle_round_to_bf16.argtypes = [ctypes.c_double]
        _lib.oracle_bf16_to_double.restype = ctypes.c_double
        _lib.oracle_bf16_to_double.argtypes = [ctypes.c_uint16]
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.uint16)
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def max_threads() -> int:
    return int(lib().oracle_max_threads())


# ----------------------------------------------------------------- format ---

def round_to_bf16(x) -> np.ndarray | int:
    """Round double(s) to bfloat16 bit pattern(s), nearest-even."""
    if np.isscalar(x):
        return int(lib().oracle_round_to_bf16(float(x)))
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().oracle_round_array(_p(x), _p(out), ctypes.c_uint64(x.size))
    return out


def widen(h) -> np.ndarray | float:
    """bfloat16 bit pattern(s) to double (exact)."""
    if np.isscalar(h):
        return float(lib().oracle_bf16_to_double(int(h)))
    h = _u16(h)
    out = np.empty(h.shape, dtype=np.float64)
    lib().oracle_widen_array(_p(h), _p(out), ctypes.c_uint64(h.size))
    return out


def binary_op(op: int, a, b=None, c=None) -> np.ndarray:
    """One rounded bfloat16 operation elementwise (Section 3.1)."""
    a = _u16(a)
    b = _u16(b) if b is not None else a
    c = _u16(c) if c is not None else a
    out = np.empty(a.shape, dtype=np.uint16)
    lib().oracle_binary_op(int(op), _p(a), _p(b), _p(c), _p(out), ctypes.c_uint64(a.size))
    return out


# ------------------------------------------------------------- primitives ---

def _two_in_two_out(name, a, b):
    a, b = _u16(a), _u16(b)
    hi = np.empty(a.shape, dtype=np.uint16)
    lo = np.empty(a.shape, dtype=np.uint16)
    getattr(lib(), name)(_p(a), _p(b), _p(hi), _p(lo), ctypes.c_uint64(a.size))
    return hi, lo


def fast_two_sum(a, b):
    return _two_in_two_out("oracle_fast_two_sum", a, b)


def two_sum(a, b):
    return _two_in_two_out("oracle_two_sum", a, b)


def two_prod(a, b):
    return _two_in_two_out("oracle_two_prod", a, b)


def two_prod_dekker(a, b):
    return _two_in_two_out("oracle_two_prod_dekker", a, b)


def renormalize(hi, lo):
    return _two_in_two_out("oracle_renormalize", hi, lo)


def split(a):
    a = _u16(a)
    hi = np.empty(a.shape, dtype=np.uint16)
    lo = np.empty(a.shape, dtype=np.uint16)
    lib().oracle_split(_p(a), _p(hi), _p(lo), ctypes.c_uint64(a.size))
    return hi, lo


def grow(x, y, a):
    x, y, a = _u16(x), _u16(y), _u16(a)
    u = np.empty(x.shape, dtype=np.uint16)
    v = np.empty(x.shape, dtype=np.uint16)
    lib().oracle_grow(_p(x), _p(y), _p(a), _p(u), _p(v), ctypes.c_uint64(x.size))
    return u, v


def scaling(v, a1, a2):
    v, a1, a2 = _u16(v), _u16(a1), _u16(a2)
    x = np.empty(v.shape, dtype=np.uint16)
    e = np.empty(v.shape, dtype=np.uint16)
    lib().oracle_scaling(_p(v), _p(a1), _p(a2), _p(x), _p(e), ctypes.c_uint64(v.size))
    return x, e


def mul(a1, a2, b1, b2):
    a1, a2, b1, b2 = _u16(a1), _u16(a2), _u16(b1), _u16(b2)
    x = np.empty(a1.shape, dtype=np.uint16)
    e = np.empty(a1.shape, dtype=np.uint16)
    lib().oracle_mul(_p(a1), _p(a2), _p(b1), _p(b2), _p(x), _p(e), ctypes.c_uint64(a1.size))
    return x, e


# ---------------------------------------------------------------- scalars ---

def derive_scalars(lr, beta1, beta2, eps, wd, step) -> dict:
    out = np.zeros(11, dtype=np.uint16)
    lib().oracle_derive_scalars(ctypes.c_double(lr), ctypes.c_double(beta1), ctypes.c_double(beta2),
                                ctypes.c_double(eps), ctypes.c_double(wd), ctypes.c_uint64(step), _p(out))
    return dict(zip(SCALAR_NAMES, (int(v) for v in out)))


# ------------------------------------------------------------------- step ---

def adamw_step(x_hi, x_lo, m, v_hi, v_lo, grad, *, lr, beta1, beta2, eps, weight_decay,
               step, strategy, flags=0, want_delta=False, threads=1):
    """One step of Algorithm 2 in place on uint16 numpy arrays.

    Returns ``(sums, delta)`` with ``sums = dict(dot, sumsq, edq, lost)`` (Eq. 2-3)
    and ``delta`` the bfloat16 update of line 12 (or None).
    """
    for arr in (x_hi, x_lo, m, v_hi, v_lo):
        if arr is not None:
            assert arr.dtype == np.uint16 and arr.flags.c_contiguous and arr.flags.writeable
    grad = _u16(grad)
    n = x_hi.size
    delta = np.empty(n, dtype=np.uint16) if want_delta else None
    sums = np.zeros(4, dtype=np.float64)
    lib().oracle_adamw_step(_p(x_hi), _p(x_lo), _p(m), _p(v_hi), _p(v_lo), _p(grad), ctypes.c_uint64(n),
                            ctypes.c_double(lr), ctypes.c_double(beta1), ctypes.c_double(beta2),
                            ctypes.c_double(eps), ctypes.c_double(weight_decay), ctypes.c_uint32(flags),
                            ctypes.c_uint64(step), ctypes.c_int(strategy), _p(delta), _p(sums),
                            ctypes.c_int(threads))
    return dict(dot=float(sums[0]), sumsq=float(sums[1]), edq=float(sums[2]), lost=int(sums[3])), delta


def edq(old_hi, old_lo, new_hi, new_lo, delta) -> dict:
    """Eq. 2-3 on stored arrays."""
    old_hi, new_hi, delta = _u16(old_hi), _u16(new_hi), _u16(delta)
    old_lo = _u16(old_lo) if old_lo is not None else None
    new_lo = _u16(new_lo) if new_lo is not None else None
    sums = np.zeros(4, dtype=np.float64)
    lib().oracle_edq(_p(old_hi), _p(old_lo), _p(new_hi), _p(new_lo), _p(delta),
                     ctypes.c_uint64(old_hi.size), _p(sums))
    return dict(dot=float(sums[0]), sumsq=float(sums[1]), edq=float(sums[2]), lost=int(sums[3]))


def adamw_fp64(theta, m, v, grad, *, lr, beta1, beta2, eps, weight_decay, step, flags=0,
               want_delta=False):
    """AdamW in double with the formulas of Algorithm 2 and no bfloat16 rounding, in place."""
    for arr in (theta, m, v):
        assert arr.dtype == np.float64 and arr.flags.c_contiguous
    grad = np.ascontiguousarray(grad, dtype=np.float64)
    delta = np.empty(theta.size, dtype=np.float64) if want_delta else None
    lib().oracle_adamw_fp64(_p(theta), _p(m), _p(v), _p(grad), ctypes.c_uint64(theta.size),
                            ctypes.c_double(lr), ctypes.c_double(beta1), ctypes.c_double(beta2),
                            ctypes.c_double(eps), ctypes.c_double(weight_decay), ctypes.c_uint32(flags),
                            ctypes.c_uint64(step), _p(delta))
    return delta


def adamw_fp32_step(theta, master, m, v, grad, *, lr, beta1, beta2, eps, weight_decay, step, flags=0):
    """Comparator option D (master = float32 array) / D^-MW (master = None), in place.

    theta, grad: uint16 bfloat16 bit patterns; m, v, master: float32.  Returns the EDQ sums dict.
    """
    assert theta.dtype == np.uint16 and m.dtype == np.float32 and v.dtype == np.float32
    assert master is None or master.dtype == np.float32
    grad = _u16(grad)
    sums = np.zeros(4, dtype=np.float64)
    lib().oracle_adamw_fp32_step(_p(theta), _p(master), _p(m), _p(v), _p(grad), ctypes.c_uint64(theta.size),
                                 ctypes.c_double(lr), ctypes.c_double(beta1), ctypes.c_double(beta2),
                                 ctypes.c_double(eps), ctypes.c_double(weight_decay), ctypes.c_uint32(flags),
                                 ctypes.c_uint64(step), _p(sums))
    return dict(dot=float(sums[0]), sumsq=float(sums[1]), edq=float(sums[2]), lost=int(sums[3]))


def adamw_fp32_register_step(x_hi, x_lo, m, v_hi, v_lo, grad, *, lr, beta1, beta2, eps, weight_decay, step, flags=0):
    """Variant: Collage-plus storage, float arithmetic in registers, re-split on store.  In place; EDQ sums dict."""
    for arr in (x_hi, x_lo, m, v_hi, v_lo):
        assert arr.dtype == np.uint16 and arr.flags.c_contiguous
    grad = _u16(grad)
    sums = np.zeros(4, dtype=np.float64)
    lib().oracle_adamw_fp32_register_step(_p(x_hi), _p(x_lo), _p(m), _p(v_hi), _p(v_lo), _p(grad),
                                          ctypes.c_uint64(x_hi.size), ctypes.c_double(lr), ctypes.c_double(beta1),
                                          ctypes.c_double(beta2), ctypes.c_double(eps), ctypes.c_double(weight_decay),
                                          ctypes.c_uint32(flags), ctypes.c_uint64(step), _p(sums))
    return dict(dot=float(sums[0]), sumsq=float(sums[1]), edq=float(sums[2]), lost=int(sums[3]))
