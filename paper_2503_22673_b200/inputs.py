"""Seeded synthetic inputs for the LoRA projection layer (Section 3.2.2, LoRA fine-tuning).

This module only *draws* inputs; it contains none of the layer's arithmetic.  Both the
CPU oracle's tests and the CUDA path's tests/benchmarks call it, so that the two sides
see byte-identical tensors.

Conventions
-----------
* All tensors are row-major: X[T, d_in], W[d_out, d_in], A[r, d_in], B[d_out, r],
  dY[T, d_out].  They are returned as ``numpy.uint16`` arrays holding bf16 bit patterns
  (numpy has no bf16 type).  ``bf16_to_f64`` widens them exactly.
* "N(0, v)" in a workload description is read as a normal with *variance* v.
* Random numbers come from numpy's counter-based Philox generator keyed by
  (seed, workload id, projection id, tensor id), so every tensor is reproducible on its
  own and independent of generation order.
* The workloads stand in for packed multi-turn agent trajectories (Section 4.1: training
  sequences of 4k-32k tokens): a projection layer sees only a T x d matrix of activations,
  so packing boundaries never reach it.  ``cu_seqlens`` is produced for the record only.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np

# tensor ids used to key the generator
_TID = {"X": 0, "W": 1, "A": 2, "B": 3, "dY": 4, "g": 5, "u": 6, "len": 7}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 (exact)."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float64 (exact)."""
    return bf16_bits_to_f32(b).astype(np.float64)


def _rng(seed: int, workload: int, proj: int, tensor: str) -> np.random.Generator:
    key = (int(seed) & 0xFFFFFFFF) | ((workload & 0xFFFF) << 32) | ((proj & 0xFF) << 48) | (
        (_TID[tensor] & 0xFF) << 56)
    return np.random.Generator(np.random.Philox(key=key))


def _normal(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    out = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        out *= np.float32(std)
    return out


@dataclasses.dataclass(frozen=True)
class Projection:
    """One LoRA linear problem: shapes, scale and how its tensors are drawn."""
    name: str
    T: int
    d_in: int
    d_out: int
    r: int
    scale: float
    x_kind: str = "normal"        # "normal" | "rmsnorm" | "swiglu"
    dy_var: float = 1.0           # variance of dY entries
    b_var: float = 0.02           # variance of B entries
    x_group: int = 0              # projections with equal x_group share X (workload 4)

    @property
    def flops(self) -> int:
        """Algorithmic FLOPs of forward + backward (dense dW is not part of LoRA)."""
        return 4 * self.T * self.d_in * self.d_out + 6 * self.T * self.r * (self.d_in + self.d_out)


def workload(idx: int, T: Optional[int] = None) -> List[Projection]:
    """The five benchmark workloads, plus (5) the paper's own q/k/v/o, r = 32 setting; ``T`` overrides the token count."""
    if idx == 0:
        return [Projection("tiny", T or 256, 512, 512, 8, 2.0)]
    if idx == 1:
        return [Projection("q_proj", T or 8192, 4096, 4096, 16, 2.0)]
    if idx == 2:
        return [Projection("gate_up_proj", T or 16384, 4096, 14336, 16, 2.0, x_kind="rmsnorm", dy_var=1e-2)]
    if idx == 3:
        return [Projection("down_proj", T or 16384, 14336, 4096, 64, 0.5, x_kind="swiglu", dy_var=1e-2)]
    if idx == 4:
        t = T or 32768
        return [
            Projection("q_proj", t, 4096, 4096, 16, 2.0, x_group=0),
            Projection("k_proj", t, 4096, 1024, 16, 2.0, x_group=0),
            Projection("v_proj", t, 4096, 1024, 16, 2.0, x_group=0),
            Projection("o_proj", t, 4096, 4096, 16, 2.0, x_group=1),
            Projection("gate_proj", t, 4096, 14336, 16, 2.0, x_group=2),
            Projection("up_proj", t, 4096, 14336, 16, 2.0, x_group=2),
            Projection("down_proj", t, 14336, 4096, 16, 2.0, x_group=3),
        ]
    if idx == 5:
        # the paper's own adapter setting (Section 4.5: q, k, v, o adapted, lora_r = 32, alpha = 64, i.e. scale 2) on its
        # Llama-3.1-8B batch shape (throughput table: 6 sequences of 8k tokens per GPU = 49152 packed tokens)
        t = T or 49152
        return [
            Projection("q_proj", t, 4096, 4096, 32, 2.0, x_group=0),
            Projection("k_proj", t, 4096, 1024, 32, 2.0, x_group=0),
            Projection("v_proj", t, 4096, 1024, 32, 2.0, x_group=0),
            Projection("o_proj", t, 4096, 4096, 32, 2.0, x_group=1),
        ]
    raise ValueError(f"unknown workload {idx}")


def packed_lengths(total: int, seed: int = 0, lo: int = 256, hi: int = 4096) -> np.ndarray:
    """Trajectory lengths, log-uniform in [lo, hi], packed until ``total`` tokens (last one cut)."""
    rng = _rng(seed, 4, 0, "len")
    lens: List[int] = []
    acc = 0
    while acc < total:
        L = int(round(lo * math.exp(rng.random() * math.log(hi / lo))))
        L = min(max(L, lo), hi)
        L = min(L, total - acc)
        lens.append(L)
        acc += L
    return np.asarray(lens, dtype=np.int64)


def cu_seqlens(idx: int, T: int, seed: int = 0) -> np.ndarray:
    """Cumulative sequence boundaries of the packed batch (never passed to the layer)."""
    if idx == 4:
        lens = packed_lengths(T, seed)
    elif idx == 1:
        lens = np.full(4, T // 4, dtype=np.int64)
        lens[-1] += T - int(lens.sum())
    elif idx == 5:
        lens = np.full(6, T // 6, dtype=np.int64)
        lens[-1] += T - int(lens.sum())
    else:
        lens = np.asarray([T], dtype=np.int64)
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)


def _draw_x(p: Projection, seed: int, wl: int, group: int) -> np.ndarray:
    if p.x_kind == "normal":
        return f32_to_bf16_bits(_normal(_rng(seed, wl, group, "X"), (p.T, p.d_in), 1.0))
    if p.x_kind == "rmsnorm":
        # post-RMSNorm activations: N(0,1) rows rescaled to unit RMS (no gain, no eps)
        x = _normal(_rng(seed, wl, group, "X"), (p.T, p.d_in), 1.0)
        rms = np.sqrt(np.mean(x.astype(np.float64) ** 2, axis=1, keepdims=True)).astype(np.float32)
        return f32_to_bf16_bits(x / rms)
    if p.x_kind == "swiglu":
        # X = SiLU(g) * u with g, u ~ N(0,1) already rounded to bf16; product in fp32
        g = bf16_bits_to_f32(f32_to_bf16_bits(_normal(_rng(seed, wl, group, "g"), (p.T, p.d_in), 1.0)))
        u = bf16_bits_to_f32(f32_to_bf16_bits(_normal(_rng(seed, wl, group, "u"), (p.T, p.d_in), 1.0)))
        silu = g / (np.float32(1.0) + np.exp(-g))
        return f32_to_bf16_bits(silu * u)
    raise ValueError(p.x_kind)


def draw(p: Projection, seed: int = 0, wl: int = 0, proj: int = 0,
         x_cache: Optional[Dict[int, np.ndarray]] = None) -> Dict[str, np.ndarray]:
    """Draw X, W, A, B, dY (bf16 bit patterns) for one projection."""
    if x_cache is not None and p.x_group in x_cache:
        X = x_cache[p.x_group]
    else:
        X = _draw_x(p, seed, wl, p.x_group)
        if x_cache is not None:
            x_cache[p.x_group] = X
    w_std = 1.0 / math.sqrt(p.d_in)
    out = {
        "X": X,
        "W": f32_to_bf16_bits(_normal(_rng(seed, wl, proj, "W"), (p.d_out, p.d_in), w_std)),
        "A": f32_to_bf16_bits(_normal(_rng(seed, wl, proj, "A"), (p.r, p.d_in), w_std)),
        "B": f32_to_bf16_bits(_normal(_rng(seed, wl, proj, "B"), (p.d_out, p.r), math.sqrt(p.b_var))),
        "dY": f32_to_bf16_bits(_normal(_rng(seed, wl, proj, "dY"), (p.T, p.d_out), math.sqrt(p.dy_var))),
    }
    return out


def draw_workload(idx: int, seed: int = 0, T: Optional[int] = None):
    """Yield (Projection, tensors) for every projection of workload ``idx``."""
    cache: Dict[int, np.ndarray] = {}
    for j, p in enumerate(workload(idx, T)):
        yield p, draw(p, seed, idx, j, cache)


def draw_custom(T: int, d_in: int, d_out: int, r: int, scale: float, seed: int = 0,
                tag: int = 99) -> "tuple[Projection, Dict[str, np.ndarray]]":
    """A free-form problem (ragged / odd shapes for edge-case tests)."""
    p = Projection(f"custom_{T}x{d_in}x{d_out}r{r}", T, d_in, d_out, r, scale)
    return p, draw(p, seed, tag, (T * 131 + d_in * 17 + d_out * 7 + r) & 0xFF)
