"""Thin ctypes binding of the CUDA library: same names as ``include/collage.h``, argument marshalling only.

Tensors are ``torch.bfloat16`` CUDA tensors (or anything with ``data_ptr()``); torch supplies
device memory and streams, every step of the computation runs in the library's kernels.
There is no fallback: if the shared library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

_LIB_PATH = Path(__file__).resolve().parent / "libcollage_b200.so"      # the in-tree build

OK, ERR_NULL, ERR_ARG, ERR_ALIAS, ERR_ARCH, ERR_CUDA, ERR_WORKSPACE, ERR_LIMIT = range(8)
BF16, LIGHT, PLUS, KAHAN, PLUS_FP32_REGISTERS = 0, 1, 2, 3, 4
FLAG_EPS_INSIDE_SQRT, FLAG_TWOSUM_GROW, FLAG_DECAY_BY_GROW = 1, 2, 4
FLAG_PIPELINE_KERNEL, FLAG_DIRECT_KERNEL, FLAG_LARGE_TILES = 8, 16, 32
OP_ADD, OP_SUB, OP_MUL, OP_DIV, OP_SQRT, OP_FMA = range(6)
SCALAR_NAMES = ("b1", "c1", "b2", "c2", "b2h", "b2l", "bc1", "bc2", "a", "lam", "eps")

EXPORTS = (
    "collage_status_string", "collage_derive_scalars", "collage_workspace_bytes", "collage_adamw_step",
    "collage_adamw_step_host", "collage_adamw_step_fp32",
    "collage_plan_create", "collage_adamw_step_multi", "collage_plan_destroy", "collage_plan_num_elements",
    "collage_plan_num_chunks", "collage_plan_set_replicas", "collage_plan_workspace_bytes", "collage_adamw_step_multi_per_tensor",
    "collage_fast_two_sum", "collage_two_sum", "collage_two_prod", "collage_grow",
    "collage_scaling", "collage_mul", "collage_renormalize", "collage_rounded_op", "collage_edq",
    "collage_selftest", "collage_pipeline_fault", "collage_edq_static", "collage_wait_timeout_selftest",
    "collage_workspace_init", "collage_edq_combine", "collage_build_flavor", "collage_enable_peer_access",
)


class Hyper(ctypes.Structure):
    """collage_hyper_t"""
    _fields_ = [("lr", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
                ("eps", ctypes.c_double), ("weight_decay", ctypes.c_double), ("flags", ctypes.c_uint32),
                ("edq_out", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


class Edq(ctypes.Structure):
    """collage_edq_t"""
    _fields_ = [("dot", ctypes.c_double), ("sumsq", ctypes.c_double), ("edq", ctypes.c_double),
                ("n", ctypes.c_uint64), ("lost", ctypes.c_uint64), ("fault", ctypes.c_uint64)]


EDQ_RECORD_BYTES = ctypes.sizeof(Edq)


class Tensor(ctypes.Structure):
    """collage_tensor_t"""
    _fields_ = [("x_hi", ctypes.c_void_p), ("x_lo", ctypes.c_void_p), ("m", ctypes.c_void_p),
                ("v_hi", ctypes.c_void_p), ("v_lo", ctypes.c_void_p), ("grad", ctypes.c_void_p),
                ("n", ctypes.c_uint64)]


class CollageError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


_lib = None
_lib_path = _LIB_PATH


def load(path) -> ctypes.CDLL:
    """Use another build of the same sources (``build.py --out``) instead of the in-tree library.

    Only an explicit call selects it (the benchmark's ``--lib``); nothing in the environment can swap
    the library under a caller.  Must come before the first use of the library in this process.
    """
    global _lib_path
    if _lib is not None:
        raise RuntimeError("the library is already loaded; call load() before any other function")
    _lib_path = Path(path).resolve()
    return lib()


def lib() -> ctypes.CDLL:
    """The loaded CUDA library; raises if it has not been built (there is no other path)."""
    global _lib
    if _lib is None:
        if not _lib_path.exists():
            raise RuntimeError(f"{_lib_path} is missing: build it with `python -m paper_2405_03637_b200.build` "
                               "(this package has no CPU or PyTorch fallback)")
        L = ctypes.CDLL(str(_lib_path))
        vp, u64, i32 = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int
        L.collage_status_string.restype = ctypes.c_char_p
        L.collage_status_string.argtypes = [i32]
        L.collage_derive_scalars.argtypes = [ctypes.POINTER(Hyper), u64, ctypes.POINTER(ctypes.c_uint16)]
        L.collage_workspace_bytes.restype = ctypes.c_size_t
        L.collage_workspace_bytes.argtypes = [u64]
        L.collage_adamw_step.argtypes = [vp, vp, vp, vp, vp, vp, u64, ctypes.POINTER(Hyper), u64, i32, vp]
        L.collage_adamw_step_host.argtypes = [vp, vp, vp, vp, vp, vp, u64, ctypes.POINTER(Hyper), u64, i32, vp,
                                              ctypes.c_size_t, vp]
        L.collage_adamw_step_fp32.argtypes = [vp, vp, vp, vp, vp, u64, ctypes.POINTER(Hyper), u64, vp]
        L.collage_plan_create.argtypes = [ctypes.POINTER(Tensor), i32, ctypes.c_uint32, ctypes.POINTER(vp)]
        L.collage_adamw_step_multi.argtypes = [vp, ctypes.POINTER(Hyper), u64, i32, vp]
        L.collage_plan_destroy.argtypes = [vp]
        L.collage_plan_num_elements.restype = u64
        L.collage_plan_num_elements.argtypes = [vp]
        L.collage_plan_num_chunks.restype = u64
        L.collage_plan_num_chunks.argtypes = [vp]
        L.collage_plan_set_replicas.argtypes = [vp, ctypes.POINTER(vp), i32]
        L.collage_plan_workspace_bytes.restype = ctypes.c_size_t
        L.collage_plan_workspace_bytes.argtypes = [vp]
        L.collage_adamw_step_multi_per_tensor.argtypes = [vp, ctypes.POINTER(Hyper), u64, i32, vp, i32, vp,
                                                          ctypes.c_size_t, vp]
        for name in ("collage_fast_two_sum", "collage_two_sum", "collage_two_prod", "collage_renormalize"):
            getattr(L, name).argtypes = [vp, vp, vp, vp, u64, vp]
        L.collage_grow.argtypes = [vp, vp, vp, vp, vp, u64, vp]
        L.collage_scaling.argtypes = [vp, vp, vp, vp, vp, u64, vp]
        L.collage_mul.argtypes = [vp, vp, vp, vp, vp, vp, u64, vp]
        L.collage_rounded_op.argtypes = [i32, vp, vp, vp, vp, u64, vp]
        L.collage_edq.argtypes = [vp, vp, vp, vp, vp, u64, vp, vp, ctypes.c_size_t, vp]
        L.collage_edq_static.argtypes = [vp, vp, vp, vp, vp, u64, vp, vp]
        L.collage_selftest.argtypes = [ctypes.POINTER(ctypes.c_uint64), vp]
        L.collage_pipeline_fault.argtypes = [ctypes.POINTER(ctypes.c_uint32)]
        L.collage_wait_timeout_selftest.argtypes = [ctypes.c_uint32, ctypes.c_void_p]
        L.collage_workspace_init.argtypes = [vp, ctypes.c_size_t, vp]
        L.collage_edq_combine.argtypes = [ctypes.POINTER(Edq), i32, ctypes.POINTER(Edq)]
        L.collage_build_flavor.restype = ctypes.c_char_p
        L.collage_build_flavor.argtypes = []
        L.collage_enable_peer_access.argtypes = [i32]
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "cuda_stream"):      # torch.cuda.Stream
        return t.cuda_stream
    return t.data_ptr()


def _check(status: int, where: str):
    if status != OK:
        raise CollageError(status, where)


def status_string(status: int) -> str:
    return lib().collage_status_string(int(status)).decode()


def make_hyper(lr, beta1, beta2, eps, weight_decay, flags=0, edq_out=None, workspace=None) -> Hyper:
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return Hyper(lr, beta1, beta2, eps, weight_decay, flags, _ptr(edq_out), _ptr(workspace), ws_bytes)


def derive_scalars(hyper: Hyper, step: int) -> dict:
    out = (ctypes.c_uint16 * 11)()
    _check(lib().collage_derive_scalars(ctypes.byref(hyper), step, out), "collage_derive_scalars")
    return dict(zip(SCALAR_NAMES, (int(v) for v in out)))


def workspace_bytes(n_total: int = 0) -> int:
    return int(lib().collage_workspace_bytes(n_total))


def workspace_init(workspace, stream=None):
    """Clear an EDQ workspace (a CUDA uint8 tensor): needed once, before its first use."""
    _check(lib().collage_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(stream)),
           "collage_workspace_init")


def _record(rec: Edq) -> dict:
    return dict(dot=rec.dot, sumsq=rec.sumsq, edq=rec.edq, n=int(rec.n), lost=int(rec.lost), fault=int(rec.fault))


def edq_combine(parts) -> dict:
    """EDQ record of the union of disjoint parameter sets from their records (dicts with dot, sumsq, n, lost)."""
    arr = (Edq * max(len(parts), 1))()
    for i, p in enumerate(parts):
        arr[i] = Edq(p["dot"], p["sumsq"], p.get("edq", 0.0), p.get("n", 0), p["lost"], p.get("fault", 0))
    out = Edq()
    _check(lib().collage_edq_combine(arr, len(parts), ctypes.byref(out)), "collage_edq_combine")
    return _record(out)


def build_flavor() -> str:
    return lib().collage_build_flavor().decode()


def adamw_step(x_hi, x_lo, m, v_hi, v_lo, grad, n, hyper: Hyper, step: int, strategy: int, stream=None):
    _check(lib().collage_adamw_step(_ptr(x_hi), _ptr(x_lo), _ptr(m), _ptr(v_hi), _ptr(v_lo), _ptr(grad), n,
                                    ctypes.byref(hyper), step, strategy, _ptr(stream)), "collage_adamw_step")


def adamw_step_host(x_hi, x_lo, m, v_hi, v_lo, grad, n, hyper: Hyper, step: int, strategy: int, staging, stream=None):
    """Host-resident state (pinned CPU tensors); `staging` is a CUDA uint8 tensor; hyper.edq_out is a host address."""
    _check(lib().collage_adamw_step_host(_ptr(x_hi), _ptr(x_lo), _ptr(m), _ptr(v_hi), _ptr(v_lo), _ptr(grad), n,
                                         ctypes.byref(hyper), step, strategy, _ptr(staging),
                                         staging.numel() * staging.element_size(), _ptr(stream)),
           "collage_adamw_step_host")


def adamw_step_fp32(theta, master, m, v, grad, n, hyper: Hyper, step: int, stream=None):
    """Comparator option D (master: float32 CUDA tensor) / D^-MW (master None); m, v float32, theta, grad bfloat16."""
    _check(lib().collage_adamw_step_fp32(_ptr(theta), _ptr(master), _ptr(m), _ptr(v), _ptr(grad), n, ctypes.byref(hyper),
                                         step, _ptr(stream)), "collage_adamw_step_fp32")


def plan_create(tensors, chunk_elems: int = 0) -> int:
    """tensors: list of (x_hi, x_lo, m, v_hi, v_lo, grad, n); returns the opaque plan handle."""
    arr = (Tensor * max(len(tensors), 1))()
    for i, (x_hi, x_lo, m, v_hi, v_lo, grad, n) in enumerate(tensors):
        arr[i] = Tensor(_ptr(x_hi), _ptr(x_lo), _ptr(m), _ptr(v_hi), _ptr(v_lo), _ptr(grad), n)
    plan = ctypes.c_void_p()
    _check(lib().collage_plan_create(arr, len(tensors), chunk_elems, ctypes.byref(plan)), "collage_plan_create")
    return plan.value


def adamw_step_multi(plan: int, hyper: Hyper, step: int, strategy: int, stream=None):
    _check(lib().collage_adamw_step_multi(plan, ctypes.byref(hyper), step, strategy, _ptr(stream)),
           "collage_adamw_step_multi")


def plan_set_replicas(plan: int, replicas):
    """replicas: list (one per replica) of lists (one per tensor of the plan, None for empty tensors) of tensors/addresses."""
    flat = [(_ptr(t) or 0) for rep in replicas for t in rep]
    arr = (ctypes.c_void_p * max(len(flat), 1))(*flat)
    _check(lib().collage_plan_set_replicas(plan, arr, len(replicas)), "collage_plan_set_replicas")


def enable_peer_access(peer_device: int):
    """Let kernels of the current device store into `peer_device`'s memory (set-up for replicas on other GPUs)."""
    _check(lib().collage_enable_peer_access(peer_device), "collage_enable_peer_access")


def plan_workspace_bytes(plan: int) -> int:
    return int(lib().collage_plan_workspace_bytes(plan))


def adamw_step_multi_per_tensor(plan: int, hyper: Hyper, step: int, strategy: int, per_tensor_out, num: int,
                                chunk_workspace, stream=None):
    """per_tensor_out: CUDA uint8 tensor of num * EDQ_RECORD_BYTES bytes; chunk_workspace: CUDA uint8 tensor."""
    _check(lib().collage_adamw_step_multi_per_tensor(plan, ctypes.byref(hyper), step, strategy, _ptr(per_tensor_out), num,
                                                     _ptr(chunk_workspace),
                                                     chunk_workspace.numel() * chunk_workspace.element_size(),
                                                     _ptr(stream)), "collage_adamw_step_multi_per_tensor")


def read_edq_array(dev_bytes, num: int) -> list:
    """Decode num consecutive device collage_edq_t records."""
    raw = dev_bytes.detach().cpu().numpy().tobytes()
    out = []
    for i in range(num):
        out.append(_record(Edq.from_buffer_copy(raw[i * ctypes.sizeof(Edq):(i + 1) * ctypes.sizeof(Edq)])))
    return out


def plan_destroy(plan: int):
    _check(lib().collage_plan_destroy(plan), "collage_plan_destroy")


def plan_num_elements(plan: int) -> int:
    return int(lib().collage_plan_num_elements(plan))


def plan_num_chunks(plan: int) -> int:
    return int(lib().collage_plan_num_chunks(plan))


def fast_two_sum(a, b, hi, lo, n, stream=None):
    _check(lib().collage_fast_two_sum(_ptr(a), _ptr(b), _ptr(hi), _ptr(lo), n, _ptr(stream)), "collage_fast_two_sum")


def two_sum(a, b, hi, lo, n, stream=None):
    _check(lib().collage_two_sum(_ptr(a), _ptr(b), _ptr(hi), _ptr(lo), n, _ptr(stream)), "collage_two_sum")


def two_prod(a, b, hi, lo, n, stream=None):
    _check(lib().collage_two_prod(_ptr(a), _ptr(b), _ptr(hi), _ptr(lo), n, _ptr(stream)), "collage_two_prod")


def renormalize(hi_in, lo_in, hi, lo, n, stream=None):
    _check(lib().collage_renormalize(_ptr(hi_in), _ptr(lo_in), _ptr(hi), _ptr(lo), n, _ptr(stream)),
           "collage_renormalize")


def grow(x, y, a, u, v, n, stream=None):
    _check(lib().collage_grow(_ptr(x), _ptr(y), _ptr(a), _ptr(u), _ptr(v), n, _ptr(stream)), "collage_grow")


def scaling(v, a1, a2, x, e, n, stream=None):
    _check(lib().collage_scaling(_ptr(v), _ptr(a1), _ptr(a2), _ptr(x), _ptr(e), n, _ptr(stream)), "collage_scaling")


def mul(a1, a2, b1, b2, x, e, n, stream=None):
    _check(lib().collage_mul(_ptr(a1), _ptr(a2), _ptr(b1), _ptr(b2), _ptr(x), _ptr(e), n, _ptr(stream)), "collage_mul")


def rounded_op(op, a, b, c, out, n, stream=None):
    _check(lib().collage_rounded_op(op, _ptr(a), _ptr(b), _ptr(c), _ptr(out), n, _ptr(stream)), "collage_rounded_op")


def edq(old_hi, old_lo, new_hi, new_lo, delta, n, out_dev, workspace, stream=None):
    ws_bytes = workspace.numel() * workspace.element_size()
    _check(lib().collage_edq(_ptr(old_hi), _ptr(old_lo), _ptr(new_hi), _ptr(new_lo), _ptr(delta), n, _ptr(out_dev),
                             _ptr(workspace), ws_bytes, _ptr(stream)), "collage_edq")


def edq_static(old_hi, old_lo, new_hi, new_lo, delta, n, out_dev, stream=None):
    """EDQ with the library's built-in scratch: for callers that cannot allocate a workspace (n <= 2^32)."""
    _check(lib().collage_edq_static(_ptr(old_hi), _ptr(old_lo), _ptr(new_hi), _ptr(new_lo), _ptr(delta), n,
                                    _ptr(out_dev), _ptr(stream)), "collage_edq_static")


def selftest(stream=None) -> dict:
    out = (ctypes.c_uint64 * 6)()
    _check(lib().collage_selftest(out, _ptr(stream)), "collage_selftest")
    return dict(zip(("add", "sub", "mul", "div", "sqrt", "scalar_div"), (int(v) for v in out)))


def pipeline_fault() -> int:
    out = ctypes.c_uint32(0)
    _check(lib().collage_pipeline_fault(ctypes.byref(out)), "collage_pipeline_fault")
    return int(out.value)


def wait_timeout_selftest(limit_ms: int, stream=None):
    _check(lib().collage_wait_timeout_selftest(limit_ms, _ptr(stream)), "collage_wait_timeout_selftest")


def read_edq(edq_dev) -> dict:
    """Copy a device collage_edq_t (a >= EDQ_RECORD_BYTES torch.uint8 CUDA tensor) to the host and decode it."""
    raw = edq_dev.detach().cpu().numpy().tobytes()
    return _record(Edq.from_buffer_copy(raw[:ctypes.sizeof(Edq)]))
