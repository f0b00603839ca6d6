"""Seeded synthetic inputs shaped like the MoE layers the Rectify-Router paper
trains (LLaMA2-7B-derived layers, micro-batches of 8 x 2048 tokens, 8 or 32
experts, top-1 / top-2, capacity factors 0.5-3.0; Section 5.1, Tables 3-6).

This module holds no arithmetic of the method: it only draws numbers.  Every
tensor is generated once on the host with NumPy's ``default_rng(seed)`` so that
the very same bytes can be handed to the CUDA library and to a CPU checker.
bf16 tensors are returned as ``uint16`` bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20240212


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class Workload:
    """One synthetic workload.  ``bias`` describes the per-expert logit bias:
    ("normal", sigma), ("zipf", s) or ("none", 0)."""
    name: str
    T: int
    E: int
    k: int
    G: int
    capacity_factors: tuple
    bias: tuple
    d: int = 0
    d_ff: int = 0
    dtype: str = "bf16"          # element type of hidden / weights / dout
    backward: bool = False
    mode: int = 3                # bit 0 = IR, bit 1 = FR
    index: int = 0

    def capacity(self, cf: float) -> int:
        c = cf * self.T / self.E
        return int(-(-c // 1))   # ceil; every listed workload divides exactly

    def seed(self, cf_index: int = 0, mode: int | None = None, extra: int = 0) -> int:
        m = self.mode if mode is None else mode
        return BASE_SEED + 1000 * self.index + 10 * cf_index + m + 100000 * extra


WORKLOADS = {
    "c1": Workload("c1", 2048, 8, 1, 2, (1.0,), ("normal", 0.7), 256, 512, "f32", False, 3, 1),
    "c2": Workload("c2", 65536, 64, 2, 8, (1.0, 1.25), ("zipf", 1.1), 0, 0, "bf16", False, 3, 2),
    "c3": Workload("c3", 16384, 8, 2, 4, (1.0,), ("normal", 0.5), 4096, 14336, "bf16", False, 3, 3),
    "c4": Workload("c4", 32768, 32, 1, 8, (1.0, 1.5), ("none", 0.0), 2048, 5632, "bf16", True, 3, 4),
    "c5": Workload("c5", 65536, 64, 2, 8, (1.0,), ("normal", 1.5), 1024, 2816, "bf16", True, 3, 5),
}


def scaled(w: Workload, t_div: int = 8, d_div: int = 4) -> Workload:
    """A reduced copy with the same E, k, G and capacity factors (T/t_div, d/d_div, d_ff/d_div)."""
    return Workload(w.name + "_small", w.T // t_div, w.E, w.k, w.G, w.capacity_factors, w.bias,
                    w.d // d_div, w.d_ff // d_div, w.dtype, w.backward, w.mode, w.index)


def expert_bias(E: int, bias: tuple, rng: np.random.Generator) -> np.ndarray:
    kind, p = bias
    if kind == "none":
        return np.zeros(E, np.float32)
    if kind == "normal":
        return rng.normal(0.0, p, E).astype(np.float32)
    if kind == "zipf":
        # log-probabilities of a Zipf(s) law over ranks 1..E, centred, handed to
        # the experts in a seeded random order so popular experts fall in all groups
        r = np.arange(1, E + 1, dtype=np.float64)
        logp = -p * np.log(r)
        logp -= np.log(np.exp(logp).sum())
        logp -= logp.mean()
        return logp[rng.permutation(E)].astype(np.float32)
    raise ValueError(kind)


def make_logits(T: int, E: int, bias: tuple, seed: int) -> np.ndarray:
    """fp32 N(0,1) logits plus a per-expert bias drawn once."""
    rng = np.random.default_rng(seed)
    b = expert_bias(E, bias, rng)
    a = rng.standard_normal((T, E), dtype=np.float32)
    a += b[None, :]
    return a


def _normal(shape, std, rng, dtype):
    n = int(np.prod(shape))
    out = np.empty(n, np.float32 if dtype == "f32" else np.uint16)
    step = 1 << 24
    for s in range(0, n, step):
        blk = rng.standard_normal(min(step, n - s), dtype=np.float32)
        if std != 1.0:
            blk *= np.float32(std)
        out[s:s + len(blk)] = blk if dtype == "f32" else to_bf16_bits(blk)
    return out.reshape(shape)


@dataclass
class LayerInputs:
    logits: np.ndarray
    hidden: np.ndarray
    W1: np.ndarray
    W3: np.ndarray
    W2: np.ndarray
    dout: np.ndarray | None
    dtype: str
    meta: dict = field(default_factory=dict)


def make_layer(T, E, d, d_ff, bias, seed, dtype="bf16", backward=False, w_std=0.02) -> LayerInputs:
    """Logits, hidden N(0,1), expert weights N(0, w_std) and (optionally) dout N(0,1)."""
    logits = make_logits(T, E, bias, seed)
    rng = np.random.default_rng(seed + 7919)
    hidden = _normal((T, d), 1.0, rng, dtype)
    W1 = _normal((E, d_ff, d), w_std, rng, dtype)
    W3 = _normal((E, d_ff, d), w_std, rng, dtype)
    W2 = _normal((E, d, d_ff), w_std, rng, dtype)
    dout = _normal((T, d), 1.0, rng, dtype) if backward else None
    return LayerInputs(logits, hidden, W1, W3, W2, dout, dtype)


def make_workload(w: Workload, cf_index: int = 0, extra_seed: int = 0) -> LayerInputs:
    return make_layer(w.T, w.E, w.d, w.d_ff, w.bias, w.seed(cf_index, extra=extra_seed), w.dtype,
                      w.backward)
