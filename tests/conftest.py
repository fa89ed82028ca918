"""Shared pytest configuration: markers, import path, and the bf16 helpers the CPU tests use."""
import sys
from pathlib import Path

import numpy as np
import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a); run with -m gpu on a B200")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device in this process")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def library_under_test_is_the_product_build():
    """Every test runs against the ordinary in-tree build, never a measurement build of the same sources."""
    from paper_2405_03637_b200 import binding, build
    build.build()
    assert binding.build_flavor() == "product"
    assert Path(binding.lib()._name) == ROOT / "paper_2405_03637_b200" / "libcollage_b200.so"


@pytest.fixture(params=["kernel chosen by size", "pipeline kernel", "large-tile pipeline"])
def step_kernel(request, monkeypatch):
    """Runs a test three times: as a caller would (small flat tensors take the kernel without staging), with
    the three-stage bulk-copy pipeline pinned, and with the two-stage large-tile pipeline pinned (it applies to
    Collage-plus; other options then run as chosen by size), so that the kernels that stream the large sets
    see every edge case too."""
    from paper_2405_03637_b200 import binding
    pin = {"pipeline kernel": binding.FLAG_PIPELINE_KERNEL, "large-tile pipeline": binding.FLAG_LARGE_TILES}.get(request.param)
    if pin:
        make = binding.make_hyper

        def pinned(*args, **kwargs):
            h = make(*args, **kwargs)
            h.flags |= pin
            return h
        monkeypatch.setattr(binding, "make_hyper", pinned)
    return request.param


def bf16_window(e_lo: int, e_hi: int, signs=(0, 1), with_zero=False) -> np.ndarray:
    """All bfloat16 bit patterns whose unbiased exponent is in [e_lo, e_hi] (normal numbers)."""
    out = []
    for s in signs:
        for e in range(e_lo, e_hi + 1):
            field = e + 127
            assert 1 <= field <= 254
            base = (s << 15) | (field << 7)
            out.append(np.arange(base, base + 128, dtype=np.uint32))
    if with_zero:
        out.append(np.array([0x0000, 0x8000], dtype=np.uint32))
    return np.concatenate(out).astype(np.uint16)


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Independent decode of bfloat16 bit patterns (numpy view as float32, then double)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def ulp_f64(bits: np.ndarray) -> np.ndarray:
    """ulp of a bfloat16 value (Def. 3.1 with 7 stored mantissa bits, e clamped at -126)."""
    field = (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.int64) >> 7) & 0xFF
    e = np.maximum(field - 127, -126)
    return np.ldexp(1.0, (e - 7).astype(np.int32))


def neighbours(bits: np.ndarray):
    """The next bfloat16 away from and toward zero for finite non-zero inputs (same sign)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.int64)
    mag = b & 0x7FFF
    sign = b & 0x8000
    up = sign | np.minimum(mag + 1, 0x7F80)
    down = sign | np.maximum(mag - 1, 0)
    return up.astype(np.uint16), down.astype(np.uint16)
