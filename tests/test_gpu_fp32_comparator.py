"""GPU parity of the option-D / D^-MW comparator step against the oracle: bfloat16 parameter and float
states bit for bit, EDQ within 1e-5."""
import numpy as np
import pytest
import torch

import oracle
from conftest import bits_to_f64
from gpu_util import EdqBuffers, edq_close
from paper_2405_03637_b200 import binding as B
from paper_2405_03637_b200 import workloads as W

pytestmark = pytest.mark.gpu
GUARD = 1024


def _guarded_f32(a, misalign=0):
    raw = np.full(a.size + 2 * GUARD + 4, np.float32(-777.25), dtype=np.float32)
    lo = GUARD + misalign
    raw[lo:lo + a.size] = a
    t = torch.from_numpy(raw).cuda()
    return t, t[lo:lo + a.size], lo


def _guards_ok(t, lo, n):
    r = t.cpu().numpy()
    return bool(np.all(r[:lo] == np.float32(-777.25)) and np.all(r[lo + n:] == np.float32(-777.25)))


@pytest.mark.parametrize("with_master", [True, False])
@pytest.mark.parametrize("n,misalign,flags", [(1 << 20, 0, 0), (100_003, 0, 1), (4097, 1, 0), (4096, 0, 0), (5, 0, 0),
                                              (3 * 4096 + 17, 0, 0)])
def test_fp32_comparator_bitwise(with_master, n, misalign, flags):
    hyp = dict(W.HYPERS, beta2=0.98)
    theta = W.bits(W.flat_weights(n, 80))
    master = bits_to_f64(theta).astype(np.float32) if with_master else None
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    d_theta = W.from_bits(np.concatenate([np.zeros(8 + misalign, np.uint16), theta]), "cuda")[8 + misalign:]
    raw_m, d_m, lo_m = _guarded_f32(m, misalign)
    raw_v, d_v, lo_v = _guarded_f32(v, misalign)
    raw_w, d_w, lo_w = _guarded_f32(master, misalign) if with_master else (None, None, 0)
    e = EdqBuffers()
    for t in (1, 2, 3, 4):
        g = W.bits(W.flat_grads(n, 81, t))
        d_g = W.from_bits(g, "cuda")
        B.adamw_step_fp32(d_theta, d_w, d_m, d_v, d_g, n, e.hyper(hyp, flags), t)
        torch.cuda.synchronize()
        want = oracle.adamw_fp32_step(theta, master, m, v, g, step=t, flags=flags, **hyp)
        assert np.array_equal(W.bits(d_theta), theta), f"theta step {t}"
        assert np.array_equal(d_m.cpu().numpy().view(np.uint32), m.view(np.uint32)), f"m step {t}"
        assert np.array_equal(d_v.cpu().numpy().view(np.uint32), v.view(np.uint32)), f"v step {t}"
        if with_master:
            assert np.array_equal(d_w.cpu().numpy().view(np.uint32), master.view(np.uint32)), f"master step {t}"
        got = e.read()
        edq_close(got, want)
        assert got["n"] == n
    assert _guards_ok(raw_m, lo_m, n) and _guards_ok(raw_v, lo_v, n)
    if with_master:
        assert _guards_ok(raw_w, lo_w, n)
    assert B.pipeline_fault() == 0


def test_fp32_comparator_argument_checks():
    n = 64
    th = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    g = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(n, dtype=torch.float32, device="cuda")
    v = torch.zeros(n, dtype=torch.float32, device="cuda")
    h = B.make_hyper(**W.HYPERS)
    with pytest.raises(B.CollageError) as err:
        B.adamw_step_fp32(th, None, m, m, g, n, h, 1)
    assert err.value.status == B.ERR_ALIAS
    with pytest.raises(B.CollageError) as err:
        B.adamw_step_fp32(th, None, m, v, g, n, h, 0)
    assert err.value.status == B.ERR_ARG
    with pytest.raises(B.CollageError) as err:
        B.adamw_step_fp32(th, None, m, v, g, n, B.make_hyper(**W.HYPERS, flags=B.FLAG_TWOSUM_GROW), 1)
    assert err.value.status == B.ERR_ARG
    B.adamw_step_fp32(th, None, m, v, g, 0, h, 1)
    torch.cuda.synchronize()


@pytest.mark.parametrize("with_master", [True, False])
def test_fp32_comparator_over_a_sweep_of_hyper_parameters(with_master):
    n = 30_011
    sweep = [(1e-4, 0.9, 0.999, 1e-8, 0.1, 1_000_000), (0.0, 0.9, 0.999, 1e-8, 0.1, 3), (1.0, 0.0, 0.5, 1e-8, 0.0, 2),
             (3e-3, 0.5, 0.95, 1e-6, 0.5, 7), (1e-2, 0.999, 0.9999, 1e-3, 1.0, 12345)]
    for lr, b1, b2, eps, wd, t0 in sweep:
        hyp = dict(lr=lr, beta1=b1, beta2=b2, eps=eps, weight_decay=wd)
        theta = W.bits(W.flat_weights(n, 82))
        master = bits_to_f64(theta).astype(np.float32) if with_master else None
        m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
        d_theta = W.from_bits(theta, "cuda")
        d_m, d_v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        d_w = torch.from_numpy(master).cuda() if with_master else None
        e = EdqBuffers()
        for t in (t0, t0 + 1, t0 + 2):
            g = W.bits(W.flat_grads(n, 83, t % 1000))
            B.adamw_step_fp32(d_theta, d_w, d_m, d_v, W.from_bits(g, "cuda"), n, e.hyper(hyp), t)
            torch.cuda.synchronize()
            want = oracle.adamw_fp32_step(theta, master, m, v, g, step=t, **hyp)
            assert np.array_equal(W.bits(d_theta), theta), f"{hyp} theta step {t}"
            assert np.array_equal(d_m.cpu().numpy().view(np.uint32), m.view(np.uint32)), f"{hyp} m step {t}"
            assert np.array_equal(d_v.cpu().numpy().view(np.uint32), v.view(np.uint32)), f"{hyp} v step {t}"
            if with_master:
                assert np.array_equal(d_w.cpu().numpy().view(np.uint32), master.view(np.uint32)), f"{hyp} master step {t}"
            edq_close(e.read(), want)
