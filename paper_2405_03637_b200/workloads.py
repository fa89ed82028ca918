"""Seeded synthetic inputs shaped like the paper's workloads.

This module only *generates data* (shapes, distributions, seeds).  It holds
none of the optimizer's arithmetic and is the one module that both the CUDA
path's tests/benchmark and the CPU oracle's tests are fed from.  Tensors are
``torch.bfloat16``; ``bits()`` gives the uint16 bit patterns as numpy, which is
the form the oracle consumes.

Stand-ins: the paper trains GPT-125M ... OpenLLaMA-7B (Appendix E, model
configuration table) on a text corpus; only the parameter *shapes* and the
magnitude scales (weights ~ N(0, 0.02^2), gradients ~ N(0, (1e-3)^2), parameter
norm far above update norm, Figure 2) are reproduced here.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

# AdamW hyper-parameters of the small configurations
HYPERS = dict(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
HYPERS_STRESS = dict(lr=1e-5, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)


def bits(t: torch.Tensor) -> np.ndarray:
    """uint16 bit patterns of a bfloat16 tensor, on the host."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16).copy()


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    """bfloat16 tensor from uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.uint16)
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)


def normal_bf16(n: int, std: float, seed: int, device="cpu") -> torch.Tensor:
    """n values ~ N(0, std^2) drawn in float32 and rounded to bfloat16 (generator of `device`)."""
    g = torch.Generator(device=device).manual_seed(seed)
    piece = 1 << 26
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for lo in range(0, n, piece):
        hi = min(n, lo + piece)
        out[lo:hi] = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32).mul_(std).to(torch.bfloat16)
    return out


# ---------------------------------------------------------------- shapes ---

def gpt2_small_shapes() -> list[tuple[str, int]]:
    """GPT-2-small-shaped parameter set: 148 tensors, 124,439,808 parameters."""
    d, ff, vocab, ctx, layers = 768, 3072, 50257, 1024, 12
    out = [("wte", vocab * d), ("wpe", ctx * d)]
    for i in range(layers):
        p = f"h{i}."
        out += [(p + "ln1.w", d), (p + "ln1.b", d), (p + "attn.qkv.w", d * 3 * d), (p + "attn.qkv.b", 3 * d),
                (p + "attn.proj.w", d * d), (p + "attn.proj.b", d), (p + "ln2.w", d), (p + "ln2.b", d),
                (p + "mlp.fc.w", d * ff), (p + "mlp.fc.b", ff), (p + "mlp.proj.w", ff * d), (p + "mlp.proj.b", d)]
    out += [("ln_f.w", d), ("ln_f.b", d)]
    return out


def llama7b_shapes(layers: int = 32) -> list[tuple[str, int]]:
    """LLaMA-7B-shaped parameter set (hidden 4096, FFN 11008, vocab 32000, untied embeddings).

    layers=32 gives 291 tensors and 6,738,415,616 parameters; smaller values give the reduced
    versions of the same layout used for whole-array parity checks.
    """
    d, ff, vocab = 4096, 11008, 32000
    out = [("embed", vocab * d)]
    for i in range(layers):
        p = f"l{i}."
        out += [(p + "attn_norm", d), (p + "q", d * d), (p + "k", d * d), (p + "v", d * d), (p + "o", d * d),
                (p + "ffn_norm", d), (p + "gate", d * ff), (p + "up", d * ff), (p + "down", ff * d)]
    out += [("norm", d), ("lm_head", vocab * d)]
    return out


def ragged_shapes() -> list[tuple[str, int]]:
    """A small set with lengths that are not multiples of 8, single elements, and an empty tensor."""
    sizes = [1, 7, 8, 9, 0, 4095, 4097, 65536, 65537, 3, 100_003, 2048, 31, 262_144 + 5]
    return [(f"t{i}", s) for i, s in enumerate(sizes)]


# ---------------------------------------------------------------- states ---

@dataclass
class State:
    """Optimizer state of one tensor (or one flat set) as bfloat16 tensors; unused parts are None."""
    x_hi: torch.Tensor
    x_lo: torch.Tensor | None
    m: torch.Tensor
    v_hi: torch.Tensor
    v_lo: torch.Tensor | None

    def arrays(self):
        return [t for t in (self.x_hi, self.x_lo, self.m, self.v_hi, self.v_lo) if t is not None]


def fresh_state(x_hi: torch.Tensor, strategy: int) -> State:
    """theta as given; delta-theta, m, v, delta-v start at +0 (Algorithm 2 lines 2-4)."""
    z = lambda: torch.zeros_like(x_hi)
    return State(x_hi, z() if strategy >= 1 else None, z(), z(), z() if strategy == 2 else None)


def flat_weights(n: int, seed: int, device="cpu") -> torch.Tensor:
    return normal_bf16(n, 0.02, seed, device)


def flat_grads(n: int, seed: int, step: int, device="cpu") -> torch.Tensor:
    """Fresh gradient for step t: seed 1000*(seed+1)+t."""
    return normal_bf16(n, 1e-3, 1000 * (seed + 1) + step, device)


# ---------------------------------------------- lost-arithmetic stress set ---

def _mix(x: torch.Tensor) -> torch.Tensor:
    """64-bit integer mixer (splitmix-style) on int64 tensors; identical bits on CPU and GPU."""
    def mulc(t, c):
        return t * c  # int64 multiplication wraps modulo 2^64

    def shr(t, k):
        return (t >> k) & ((1 << (64 - k)) - 1)   # logical shift on a signed type

    x = x + (-7046029254386353131)                # 0x9E3779B97F4A7C15
    x = mulc(x ^ shr(x, 30), -4658895280553007687)  # 0xBF58476D1CE4E5B9
    x = mulc(x ^ shr(x, 27), -7723592293110705685)  # 0x94D049BB133111EB
    return x ^ shr(x, 31)


def stress_weights(n: int, seed: int, device="cpu") -> torch.Tensor:
    """theta = +-U(0.5, 4) rounded to bfloat16, sign uniform."""
    g = torch.Generator(device=device).manual_seed(seed)
    mag = torch.rand(n, generator=g, device=device, dtype=torch.float32) * 3.5 + 0.5
    sign = torch.randint(0, 2, (n,), generator=g, device=device, dtype=torch.int32) * 2 - 1
    return (mag * sign).to(torch.bfloat16)


def stress_grads(n: int, seed: int, step: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """Gradient magnitudes log-uniform over [1e-8, 1e-2], integer-only.

    The bfloat16 bit pattern is drawn uniformly from [bits(1e-8), bits(1e-2)] = [0x322C, 0x3C24]
    (uniform over patterns = uniform over binades, log-uniform overall); the sign is a hash of
    (seed, index) only, fixed over steps, so that sub-ulp updates accumulate in one direction.
    `offset` is the global index of element 0, so that a slice reproduces the same values.
    """
    lo, hi = 0x322C, 0x3C24
    idx = torch.arange(offset, offset + n, dtype=torch.int64, device=device)
    h = _mix(idx * 0x100000001B3 + (seed * 1_000_003 + step))
    mag = lo + ((h >> 1) & 0x3FFFFFFFFFFFFFFF) % (hi - lo + 1)
    sgn = (_mix(idx + (seed << 40)) & 1) << 15
    return (mag | sgn).to(torch.int16).view(torch.bfloat16)
