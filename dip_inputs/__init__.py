"""Seeded synthetic inputs for the DIP / DIP-CA decode-MLP workloads.

This module only draws numbers and encodes them into storage formats; it holds
none of the method's arithmetic (no masks, no scores, no MLP).  It is the one
module that both the CPU oracle's tests and the CUDA path's tests and benchmark
use, so that both sides see identical bytes.  numpy only.

Every array is a pure function of (seed, workload, layer, role): draws come from
numpy's counter-based Philox generator keyed by those integers, so any layer can
be produced on demand without generating the ones before it.

Workloads (shapes of the paper's models, Sec. 6: Phi-3-mini, Phi-3-Medium,
Llama-3-8B; the paper's own evaluation data and checkpoints are replaced by
heavy-tailed synthetic activations and N(0, 0.02) weights):

  block_f32      1 block   d_model 1024  d_ff  2816  fp32   64 tokens  Student-t(3), unit RMS
  phi3_mini      32 layers d_model 3072  d_ff  8192  bf16  256 tokens  Student-t(3), unit RMS
  phi3_medium    40 layers d_model 5120  d_ff 17920  bf16  512 tokens  Laplace(0, 1)
  llama3_8b_int4 32 layers d_model 4096  d_ff 14336  int4  512 tokens  Student-t(3), unit RMS
  phi3_medium_batched      phi3_medium shapes, 256 steps, Student-t(3), batch 1..16
"""
from dataclasses import dataclass, replace
from typing import Optional, Tuple

import numpy as np

W_F32, W_BF16, W_INT4_G128 = 0, 1, 2
GROUP = 128
WEIGHT_STD = 0.02

_ROLE = {"gate": 1, "up": 2, "down": 3, "x": 4}


@dataclass(frozen=True)
class Workload:
    name: str
    wid: int            # enters the generator key
    seed: int
    n_layers: int
    d_model: int
    d_ff: int
    wtype: int
    n_tokens: int
    dist: str           # "student_t3" (scaled to unit RMS) or "laplace"
    keep_ratio: float
    gamma: float
    cache_budget: Optional[float]   # fraction of each layer's columns; None = cache-aware masking off
    batch: int = 1

    @property
    def k_x(self) -> int:
        return keep_count(self.keep_ratio, self.d_model)

    @property
    def k_h(self) -> int:
        return keep_count(self.keep_ratio, self.d_ff)

    @property
    def cap_gu(self) -> Optional[int]:
        return None if self.cache_budget is None else cache_capacity(self.cache_budget, self.d_model)

    @property
    def cap_d(self) -> Optional[int]:
        return None if self.cache_budget is None else cache_capacity(self.cache_budget, self.d_ff)

    def scaled(self, **kw) -> "Workload":
        """Same recipe with some fields replaced (smaller shapes for tests, other keep ratios)."""
        return replace(self, **kw)


def keep_count(ratio: float, d: int) -> int:
    """Number of kept columns for a keep ratio: round half up, clamped to [1, d]."""
    return max(1, min(d, int(np.floor(ratio * d + 0.5))))


def cache_capacity(budget: float, d: int) -> int:
    """Cache size in columns for a budget given as a fraction of d: floor (never above the budget)."""
    return max(0, min(d, int(np.floor(budget * d + 1e-9))))


WORKLOADS = {
    w.name: w for w in [
        Workload("block_f32", 0, 0, 1, 1024, 2816, W_F32, 64, "student_t3", 0.5, 1.0, None),
        Workload("phi3_mini", 1, 1, 32, 3072, 8192, W_BF16, 256, "student_t3", 0.25, 0.2, 0.5),
        Workload("phi3_medium", 2, 2, 40, 5120, 17920, W_BF16, 512, "laplace", 0.25, 0.2, 0.5),
        Workload("llama3_8b_int4", 3, 3, 32, 4096, 14336, W_INT4_G128, 512, "student_t3", 0.25, 0.2, 0.4),
        Workload("phi3_medium_batched", 4, 4, 40, 5120, 17920, W_BF16, 256, "student_t3", 0.25, 1.0, None, 16),
    ]
}
PHI3_MEDIUM_KEEP_RATIOS = (0.1, 0.25, 0.5, 1.0)
PHI3_MEDIUM_CACHE_BUDGETS = (0.25, 0.5)
BATCH_SIZES = (1, 2, 4, 8, 16)


def _rng(w: Workload, layer: int, role: str, extra: int = 0) -> np.random.Generator:
    key = (np.uint64(w.seed) << np.uint64(32)) | np.uint64(w.wid)
    ctr_hi = (np.uint64(layer) << np.uint64(32)) | (np.uint64(_ROLE[role]) << np.uint64(24)) | np.uint64(extra)
    return np.random.Generator(np.random.Philox(key=[key, ctr_hi]))


# ----------------------------------------------------------------------------
# storage encodings
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round binary32 to bfloat16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def quantize_int4_g128(w: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Symmetric 4-bit quantisation with one binary16 scale per 128 input indices.

    w: float32 [d_out, d_in].  Returns (q_packed uint8 [d_out, d_in // 2] with the
    even column in the low nibble, codes in 1..15 meaning -7..7 after subtracting 8;
    scales uint16 binary16 bit patterns [d_in // 128, d_out]).
    """
    d_out, d_in = w.shape
    assert d_in % GROUP == 0
    g = w.reshape(d_out, d_in // GROUP, GROUP).astype(np.float64)
    s = np.abs(g).max(axis=2) / 7.0
    s16 = s.astype(np.float16)
    s16 = np.where(s16 == 0, np.float16(6e-8), s16)           # keep the division defined
    q = np.rint(g / s16.astype(np.float64)[:, :, None])
    q = np.clip(q, -7, 7).astype(np.int8) + 8
    q = q.reshape(d_out, d_in).astype(np.uint8)
    packed = (q[:, 0::2] | (q[:, 1::2] << 4)).astype(np.uint8)
    scales = np.ascontiguousarray(s16.T).view(np.uint16)       # [d_in/128, d_out]
    return np.ascontiguousarray(packed), scales


def dequantize_int4_g128(packed: np.ndarray, scales: np.ndarray, d_out: int, d_in: int) -> np.ndarray:
    """Decode the storage format back to float32 (format definition; used to build comparison matrices)."""
    q = np.empty((d_out, d_in), dtype=np.int32)
    q[:, 0::2] = packed & 0xF
    q[:, 1::2] = packed >> 4
    s = scales.view(np.float16).astype(np.float32)             # [d_in/128, d_out]
    return ((q - 8).astype(np.float32) * np.repeat(s.T, GROUP, axis=1)).astype(np.float32)


# ----------------------------------------------------------------------------
# weights
# ----------------------------------------------------------------------------
@dataclass
class LayerWeights:
    """One MLP block in canonical orientation: gate, up [d_ff, d_model]; down [d_model, d_ff].

    F32: float32 arrays.  BF16: uint16 bit patterns.  INT4_G128: packed uint8
    [d_out, d_in // 2] plus binary16 scale bit patterns [d_in // 128, d_out].
    """
    wtype: int
    d_model: int
    d_ff: int
    gate: np.ndarray
    up: np.ndarray
    down: np.ndarray
    gate_scales: Optional[np.ndarray] = None
    up_scales: Optional[np.ndarray] = None
    down_scales: Optional[np.ndarray] = None


def _matrix(w: Workload, layer: int, role: str, d_out: int, d_in: int):
    z = _rng(w, layer, role).standard_normal((d_out, d_in), dtype=np.float32)
    z *= np.float32(WEIGHT_STD)
    if w.wtype == W_F32:
        return z, None
    if w.wtype == W_BF16:
        return f32_to_bf16_bits(z), None
    return quantize_int4_g128(z)


def layer_weights(w: Workload, layer: int) -> LayerWeights:
    g, gs = _matrix(w, layer, "gate", w.d_ff, w.d_model)
    u, us = _matrix(w, layer, "up", w.d_ff, w.d_model)
    d, ds = _matrix(w, layer, "down", w.d_model, w.d_ff)
    return LayerWeights(w.wtype, w.d_model, w.d_ff, g, u, d, gs, us, ds)


# ----------------------------------------------------------------------------
# activations
# ----------------------------------------------------------------------------
def token_inputs(w: Workload, n_tokens: Optional[int] = None, batch: Optional[int] = None,
                 d: Optional[int] = None, correlation: float = 0.0) -> np.ndarray:
    """First-layer inputs x_0 for every decode step: float32 [n_tokens, batch, d].

    student_t3: Student-t with 3 degrees of freedom, each vector scaled to unit RMS
    in fp64 and rounded to binary32.  laplace: Laplace(0, 1), rounded to binary32.
    correlation c > 0: consecutive tokens of a sequence are mixed, x_t = c x_{t-1} +
    sqrt(1 - c^2) draw_t (real activations are correlated over time; independent draws are not).
    """
    n = w.n_tokens if n_tokens is None else n_tokens
    b = w.batch if batch is None else batch
    dd = w.d_model if d is None else d
    rng = _rng(w, 0, "x")
    if w.dist == "student_t3":
        v = rng.standard_t(3.0, size=(n, b, dd))
    elif w.dist == "laplace":
        v = rng.laplace(0.0, 1.0, size=(n, b, dd))
    else:
        raise ValueError(w.dist)
    if correlation > 0.0:
        fresh = float(np.sqrt(1.0 - correlation * correlation))
        for t in range(1, n):
            v[t] = correlation * v[t - 1] + fresh * v[t]
    if w.dist == "student_t3":
        v /= np.sqrt((v * v).mean(axis=2, keepdims=True))
    return v.astype(np.float32)


def heavy_tail_vector(seed: int, d: int, dist: str = "student_t3") -> np.ndarray:
    """A single activation-like vector (float32 [d]) for kernel-level tests."""
    rng = np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(d)]))
    v = rng.standard_t(3.0, size=d) if dist == "student_t3" else rng.laplace(0.0, 1.0, size=d)
    if dist == "student_t3":
        v /= np.sqrt((v * v).mean())
    return v.astype(np.float32)
