"""Python binding of the CPU oracle (oracle/dip_oracle.c).

TEST INFRASTRUCTURE: imported only by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  It imports nothing from the CUDA package and the
CUDA package imports nothing from here.  Arrays are numpy; weights are in the
paper's canonical orientation [d_out, d_in] (W^u, W^g: [d_ff, d_model];
W^d: [d_model, d_ff]).
"""
import ctypes as C
from dataclasses import dataclass
from typing import Optional

import numpy as np

from . import build as _build

W_F32, W_BF16, W_INT4_G128 = 0, 1, 2
GROUP = 128

import os as _os

# DIP_ORACLE_LIB: load another build of the oracle (the mutation tests plant mistakes in a copy)
_lib = C.CDLL(_os.environ.get("DIP_ORACLE_LIB") or _build.build())

_vp, _i32, _f32, _f64 = C.c_void_p, C.c_int, C.c_float, C.c_double

_lib.orc_num_threads.restype = _i32
_lib.orc_set_num_threads.restype = None
_lib.orc_set_num_threads.argtypes = [_i32]
_lib.orc_silu.restype = _f64
_lib.orc_silu.argtypes = [_f64]
_lib.orc_glu.restype = None
_lib.orc_glu.argtypes = [_vp, _vp, _i32, _vp]
_lib.orc_weight.restype = _f64
_lib.orc_weight.argtypes = [_i32, _vp, _vp, _i32, _i32, _i32, _i32]
_lib.orc_rank_key.restype = C.c_uint32
_lib.orc_rank_key.argtypes = [_f32, _i32, _f32]
_lib.orc_ca_score.restype = None
_lib.orc_ca_score.argtypes = [_vp, _vp, _f64, _i32, _vp]
_lib.orc_topk_mask.restype = _i32
_lib.orc_topk_mask.argtypes = [_vp, _i32, _i32, _vp, _vp]
_lib.orc_cache_update.restype = _i32
_lib.orc_cache_update.argtypes = [_vp, _vp, _vp, _i32, _i32, _vp, _vp]
_lib.orc_cache_update_lfu.restype = _i32
_lib.orc_cache_update_lfu.argtypes = [_vp, _vp, _vp, _vp, _i32, _i32, _vp, _vp]
_lib.orc_belady_hits.restype = C.c_longlong
_lib.orc_belady_hits.argtypes = [_vp, _i32, _i32, _i32, _vp]
_lib.orc_dip_ca_mask.restype = _i32
_lib.orc_dip_ca_mask.argtypes = [_vp, _i32, _i32, _f32, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp]
_lib.orc_masked_matvec.restype = None
_lib.orc_masked_matvec.argtypes = [_i32, _vp, _vp, _i32, _i32, _vp, _vp, _vp]
_lib.orc_dense_mlp.restype = None
_lib.orc_dense_mlp.argtypes = [_i32, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _vp, _vp, _vp]
_lib.orc_mlp_step.restype = _i32
_lib.orc_mlp_step.argtypes = ([_i32, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _vp, _i32, _i32, _f32]
                              + [_vp, _vp, _vp, _vp, _i32, _vp] * 2 + [_vp] * 6)
_lib.orc_neuron_pruned_step.restype = _i32
_lib.orc_neuron_pruned_step.argtypes = [_i32, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _vp, _i32, _i32,
                                        _vp, _vp, _vp, _vp, _vp]
_lib.orc_residual_rmsnorm.restype = None
_lib.orc_residual_rmsnorm.argtypes = [_vp, _vp, _i32, _vp]
_lib.orc_mask_union.restype = _i32
_lib.orc_mask_union.argtypes = [_vp, _i32, _i32, _vp]


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_vp)


def _chk(a: np.ndarray, dtype, n=None) -> np.ndarray:
    if a.dtype != dtype or not a.flags["C_CONTIGUOUS"]:
        raise TypeError("expected C-contiguous %s, got %s" % (np.dtype(dtype), a.dtype))
    if n is not None and a.size != n:
        raise ValueError("expected %d elements, got %d" % (n, a.size))
    return a


def num_threads() -> int:
    return int(_lib.orc_num_threads())


def set_num_threads(n: int) -> None:
    """Threads the oracle's parallel loops use from now on (timing legs only; results do not change)."""
    _lib.orc_set_num_threads(int(n))


def silu(z: float) -> float:
    return float(_lib.orc_silu(float(z)))


def glu(g: np.ndarray, u: np.ndarray) -> np.ndarray:
    """Eq. 2 element-wise: u * silu(g), fp64."""
    g = _chk(np.ascontiguousarray(g), np.float64)
    u = _chk(np.ascontiguousarray(u), np.float64, g.size)
    h = np.empty(g.size, dtype=np.float64)
    _lib.orc_glu(_p(g), _p(u), g.size, _p(h))
    return h


def rank_key(x: float, resident: bool, gamma: float) -> int:
    return int(_lib.orc_rank_key(float(np.float32(x)), int(bool(resident)), float(np.float32(gamma))))


@dataclass
class Matrix:
    """A stored weight matrix W[d_out, d_in] (canonical orientation).

    F32: w float32 [d_out, d_in].  BF16: w uint16 bit patterns [d_out, d_in].
    INT4_G128: w uint8 [d_out, d_in // 2] (even column in the low nibble),
    scales uint16 (binary16 bit patterns) [d_in // 128, d_out].
    """
    type: int
    w: np.ndarray
    scales: Optional[np.ndarray]
    d_out: int
    d_in: int

    def __post_init__(self):
        if self.type == W_F32:
            _chk(self.w, np.float32, self.d_out * self.d_in)
        elif self.type == W_BF16:
            _chk(self.w, np.uint16, self.d_out * self.d_in)
        elif self.type == W_INT4_G128:
            _chk(self.w, np.uint8, self.d_out * self.d_in // 2)
            _chk(self.scales, np.uint16, (self.d_in // GROUP) * self.d_out)
            if self.d_in % GROUP:
                raise ValueError("INT4 needs d_in % 128 == 0")
        else:
            raise ValueError("unknown weight type")

    def element(self, j: int, i: int) -> float:
        return float(_lib.orc_weight(self.type, _p(self.w), _p(self.scales), self.d_out, self.d_in, j, i))


class Cache:
    """LRU column-cache state of one masked linear-layer input (Alg. 1's c)."""

    def __init__(self, d: int, capacity: int, policy: str = "lru"):
        assert policy in ("lru", "lfu")
        self.d, self.capacity, self.policy = int(d), int(capacity), policy
        self.count = np.zeros(d, dtype=np.int32)      # LFU use counters
        self.stamp = np.full(d, -1, dtype=np.int32)
        self.n_resident = np.zeros(1, dtype=np.int32)
        self.step = np.zeros(1, dtype=np.int32)
        self.counters = np.zeros(4, dtype=np.int32)  # hits, misses, evictions, bypassed

    def resident(self) -> np.ndarray:
        return (self.stamp >= 0).astype(np.uint8)

    def copy(self) -> "Cache":
        c = Cache(self.d, self.capacity, self.policy)
        c.count[:] = self.count
        c.stamp[:] = self.stamp
        c.n_resident[:] = self.n_resident
        c.step[:] = self.step
        c.counters[:] = self.counters
        return c


def ca_score(x: np.ndarray, c: Optional[np.ndarray], gamma: float) -> np.ndarray:
    x = _chk(np.ascontiguousarray(x), np.float32)
    s = np.empty(x.size, dtype=np.float64)
    cc = None if c is None else _chk(np.ascontiguousarray(c), np.uint8, x.size)
    _lib.orc_ca_score(_p(x), _p(cc), float(gamma), x.size, _p(s))
    return s


def topk_mask(key: np.ndarray, k: int):
    key = _chk(np.ascontiguousarray(key), np.uint32)
    d = key.size
    m = np.empty(d, dtype=np.uint8)
    idx = np.empty(max(k, 0), dtype=np.int32)
    if _lib.orc_topk_mask(_p(key), d, int(k), _p(m), _p(idx)):
        raise ValueError("k outside [0, d]")
    return m, idx


def cache_update(cache: Cache, m: np.ndarray) -> None:
    m = _chk(np.ascontiguousarray(m), np.uint8, cache.d)
    if cache.policy == "lfu":
        rc = _lib.orc_cache_update_lfu(_p(cache.stamp), _p(cache.count), _p(cache.n_resident), _p(cache.step),
                                       cache.d, cache.capacity, _p(m), _p(cache.counters))
    else:
        rc = _lib.orc_cache_update(_p(cache.stamp), _p(cache.n_resident), _p(cache.step), cache.d,
                                   cache.capacity, _p(m), _p(cache.counters))
    if rc:
        raise ValueError("capacity outside [0, d]")


def belady_hits(masks: np.ndarray, capacity: int):
    """Offline Belady replay of a trace of masks uint8 [T, d]; returns (hits, misses)."""
    masks = _chk(np.ascontiguousarray(masks), np.uint8)
    T, d = masks.shape
    miss = C.c_longlong(0)
    hits = _lib.orc_belady_hits(_p(masks), T, d, int(capacity), C.byref(miss))
    return int(hits), int(miss.value)


def dip_ca_mask(x: np.ndarray, k: int, gamma: float = 1.0, cache: Optional[Cache] = None):
    """Alg. 1 for one linear-layer input; cache=None is plain DIP (Eq. 7-8)."""
    x = _chk(np.ascontiguousarray(x), np.float32)
    d = x.size
    m = np.empty(d, dtype=np.uint8)
    idx = np.empty(max(k, 0), dtype=np.int32)
    if cache is None:
        rc = _lib.orc_dip_ca_mask(_p(x), d, int(k), float(gamma), None, None, None, None, 0, _p(m), _p(idx), None)
    else:
        if cache.d != d:
            raise ValueError("cache size mismatch")
        rc = _lib.orc_dip_ca_mask(_p(x), d, int(k), float(gamma), _p(cache.stamp),
                                  _p(cache.count) if cache.policy == "lfu" else None, _p(cache.n_resident),
                                  _p(cache.step), cache.capacity, _p(m), _p(idx), _p(cache.counters))
    if rc:
        raise ValueError("invalid k or capacity")
    return m, idx


def masked_matvec(W: Matrix, v: np.ndarray, m: np.ndarray) -> np.ndarray:
    v = _chk(np.ascontiguousarray(v), np.float32, W.d_in)
    m = _chk(np.ascontiguousarray(m), np.uint8, W.d_in)
    out = np.empty(W.d_out, dtype=np.float64)
    _lib.orc_masked_matvec(W.type, _p(W.w), _p(W.scales), W.d_out, W.d_in, _p(v), _p(m), _p(out))
    return out


def dense_mlp(Wg: Matrix, Wu: Matrix, Wd: Matrix, x: np.ndarray):
    """Eq. 1-2.  Returns (GLU(x), MLP(x)) in fp64."""
    d_ff, d_model = Wg.d_out, Wg.d_in
    x = _chk(np.ascontiguousarray(x), np.float32, d_model)
    glu = np.empty(d_ff, dtype=np.float64)
    y = np.empty(d_model, dtype=np.float64)
    _lib.orc_dense_mlp(Wg.type, _p(Wg.w), _p(Wg.scales), _p(Wu.w), _p(Wu.scales), _p(Wd.w), _p(Wd.scales),
                       d_model, d_ff, _p(x), _p(glu), _p(y))
    return glu, y


@dataclass
class StepResult:
    m_x: np.ndarray
    idx_x: np.ndarray
    h32: np.ndarray
    m_h: np.ndarray
    idx_h: np.ndarray
    y: np.ndarray


def mlp_step(Wg: Matrix, Wu: Matrix, Wd: Matrix, x: np.ndarray, k_x: int, k_h: int, gamma: float = 1.0,
             cache_gu: Optional[Cache] = None, cache_d: Optional[Cache] = None) -> StepResult:
    """One sparse MLP step for one token (Eq. 3, 7, 8; Alg. 1 when caches are given)."""
    d_ff, d_model = Wg.d_out, Wg.d_in
    x = _chk(np.ascontiguousarray(x), np.float32, d_model)
    r = StepResult(np.empty(d_model, np.uint8), np.empty(k_x, np.int32), np.empty(d_ff, np.float32),
                   np.empty(d_ff, np.uint8), np.empty(k_h, np.int32), np.empty(d_model, np.float64))

    def cargs(c):
        if c is None:
            return [None, None, None, None, 0, None]
        return [_p(c.stamp), _p(c.count) if c.policy == "lfu" else None, _p(c.n_resident), _p(c.step), c.capacity,
                _p(c.counters)]

    rc = _lib.orc_mlp_step(Wg.type, _p(Wg.w), _p(Wg.scales), _p(Wu.w), _p(Wu.scales), _p(Wd.w), _p(Wd.scales),
                           d_model, d_ff, _p(x), int(k_x), int(k_h), float(gamma),
                           *cargs(cache_gu), *cargs(cache_d),
                           _p(r.m_x), _p(r.idx_x), _p(r.h32), _p(r.m_h), _p(r.idx_h), _p(r.y))
    if rc:
        raise ValueError("invalid k or capacity")
    return r


@dataclass
class NeuronPrunedResult:
    p32: np.ndarray
    m: np.ndarray
    idx: np.ndarray
    h32: np.ndarray
    y: np.ndarray


def neuron_pruned_step(Wg: Matrix, Wu: Matrix, Wd: Matrix, x: np.ndarray, k: int, by: str) -> NeuronPrunedResult:
    """Gate pruning (by="gate") or Up pruning (by="up") of Sec. 3.2 / Eq. 5 for one token."""
    assert by in ("gate", "up")
    d_ff, d_model = Wg.d_out, Wg.d_in
    x = _chk(np.ascontiguousarray(x), np.float32, d_model)
    r = NeuronPrunedResult(np.empty(d_ff, np.float32), np.empty(d_ff, np.uint8), np.empty(k, np.int32),
                           np.empty(d_ff, np.float32), np.empty(d_model, np.float64))
    rc = _lib.orc_neuron_pruned_step(Wg.type, _p(Wg.w), _p(Wg.scales), _p(Wu.w), _p(Wu.scales), _p(Wd.w),
                                     _p(Wd.scales), d_model, d_ff, _p(x), int(k), 0 if by == "gate" else 1,
                                     _p(r.p32), _p(r.m), _p(r.idx), _p(r.h32), _p(r.y))
    if rc:
        raise ValueError("invalid k")
    return r


def residual_rmsnorm(x: np.ndarray, y: np.ndarray) -> np.ndarray:
    x = _chk(np.ascontiguousarray(x), np.float32)
    y = _chk(np.ascontiguousarray(y), np.float64, x.size)
    out = np.empty(x.size, dtype=np.float32)
    _lib.orc_residual_rmsnorm(_p(x), _p(y), x.size, _p(out))
    return out


def mask_union(m: np.ndarray):
    """m: uint8 [B, d] per-token masks.  Returns (union mask [d], |U|)."""
    m = _chk(np.ascontiguousarray(m), np.uint8)
    b, d = m.shape
    u = np.empty(d, dtype=np.uint8)
    n = _lib.orc_mask_union(_p(m), b, d, _p(u))
    return u, int(n)
