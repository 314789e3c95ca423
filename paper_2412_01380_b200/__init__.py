"""Thin Python binding of the sm_100a DIP / DIP-CA sparse decode-MLP library (include/dip.h).

Argument marshalling only: every step of the method runs in the CUDA kernels of
`libdip.so`.  PyTorch supplies device memory and streams.  There is no CPU
fallback: importing this package without the built library raises ImportError.

Functions carry the names of the C entry points they call.
"""
import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdip.so")

W_F32, W_BF16, W_INT4_G128 = 0, 1, 2
MAX_D, MAX_BATCH, INT4_GROUP, CACHE_META_INTS = 32768, 16, 128, 8
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_WORKSPACE = 0, 1, 2, 3, 4
DEVICE_OK, DEVICE_WAIT_TIMEOUT, DEVICE_TIER_INCONSISTENT = 0, 1, 2

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "%s is missing: build it with `python paper_2412_01380_b200/build.py` "
        "(nvcc, sm_100a).  This package has no fallback path." % LIB_PATH)
_lib = C.CDLL(LIB_PATH)

_vp, _i32, _f32 = C.c_void_p, C.c_int, C.c_float


class MlpWeightsStruct(C.Structure):
    _fields_ = [("wtype", C.c_int32), ("d_model", C.c_int32), ("d_ff", C.c_int32), ("reserved", C.c_int32),
                ("gate_up", _vp), ("gate_up_scales", _vp), ("down", _vp), ("down_scales", _vp)]


class CacheStateStruct(C.Structure):
    _fields_ = [("d", C.c_int32), ("capacity", C.c_int32), ("stamp", _vp), ("meta", _vp), ("count", _vp),
                ("policy", C.c_int32), ("reserved", C.c_int32)]


class StepOutputsStruct(C.Structure):
    _fields_ = [("mask_x", _vp), ("idx_x", _vp), ("h", _vp), ("mask_h", _vp), ("idx_h", _vp),
                ("union_counts", _vp)]


class OptionsStruct(C.Structure):
    _fields_ = [("max_d", C.c_int32), ("max_batch", C.c_int32), ("gemv_segment_bytes", C.c_int32),
                ("gemv_copy_ring", C.c_int32), ("coarse_min_d", C.c_int32), ("wait_limit_us", C.c_int32),
                ("select_in_product", C.c_int32), ("reserved", C.c_int32 * 3)]


class StackProbeStruct(C.Structure):
    _fields_ = [("x", _vp), ("mask_x", _vp), ("h", _vp), ("mask_h", _vp), ("y", _vp)]


_lib.dip_create.restype = _i32
_lib.dip_create.argtypes = [C.POINTER(_vp), _i32]
_lib.dip_create_ex.restype = _i32
_lib.dip_create_ex.argtypes = [C.POINTER(_vp), _i32, C.POINTER(OptionsStruct)]
_lib.dip_reset_device_status.restype = _i32
_lib.dip_reset_device_status.argtypes = [_vp, _vp]
_lib.dip_selftest_bounded_wait.restype = _i32
_lib.dip_selftest_bounded_wait.argtypes = [_vp, _i32, _vp, _vp]
_lib.dip_destroy.restype = _i32
_lib.dip_destroy.argtypes = [_vp]
_lib.dip_status_string.restype = C.c_char_p
_lib.dip_status_string.argtypes = [_i32]
_lib.dip_last_error.restype = C.c_char_p
_lib.dip_last_error.argtypes = [_vp]
_lib.dip_sm_count.restype = _i32
_lib.dip_sm_count.argtypes = [_vp]
_lib.dip_device_status.restype = _i32
_lib.dip_device_status.argtypes = [_vp, C.POINTER(C.c_int), _vp]
_lib.dip_packed_bytes.restype = C.c_size_t
_lib.dip_packed_bytes.argtypes = [_i32, _i32, _i32, _i32]
_lib.dip_pack_weights.restype = _i32
_lib.dip_pack_weights.argtypes = [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp,
                                  C.POINTER(MlpWeightsStruct), _vp]
_lib.dip_mask_topk.restype = _i32
_lib.dip_mask_topk.argtypes = [_vp, _vp, _i32, _i32, _i32, _vp, _vp, _vp]
_lib.dip_ca_mask.restype = _i32
_lib.dip_ca_mask.argtypes = [_vp, _vp, _i32, _i32, _f32, C.POINTER(CacheStateStruct), _vp, _vp, _vp]
for _name in ("dip_sparse_gemv_gate_up", "dip_sparse_gemv_down"):
    getattr(_lib, _name).restype = _i32
    getattr(_lib, _name).argtypes = [_vp, C.POINTER(MlpWeightsStruct), _vp, _i32, _vp, _i32, _vp, _vp, _vp]
_lib.dip_select_gemv_gate_up.restype = _i32
_lib.dip_select_gemv_gate_up.argtypes = [_vp, C.POINTER(MlpWeightsStruct), _vp, _i32, _f32, C.POINTER(CacheStateStruct),
                                         C.POINTER(CacheStateStruct), _vp, _vp, _vp]
_lib.dip_select_gemv_down.restype = _i32
_lib.dip_select_gemv_down.argtypes = [_vp, C.POINTER(MlpWeightsStruct), _vp, _i32, _f32, C.POINTER(CacheStateStruct),
                                      _vp, _vp, _vp]
_lib.dip_mlp_step.restype = _i32
_lib.dip_mlp_step.argtypes = [_vp, C.POINTER(MlpWeightsStruct), _vp, _i32, _i32, _i32, _f32,
                              C.POINTER(CacheStateStruct), C.POINTER(CacheStateStruct), _vp,
                              C.POINTER(StepOutputsStruct), _vp]
_lib.dip_residual_rmsnorm.restype = _i32
_lib.dip_residual_rmsnorm.argtypes = [_vp, _vp, _vp, _i32, _i32, _vp, _vp]
_lib.dip_stack_step.restype = _i32
_lib.dip_stack_step.argtypes = [_vp, _i32, C.POINTER(MlpWeightsStruct), _vp, _i32, _i32, _i32, _f32,
                                C.POINTER(CacheStateStruct), C.POINTER(CacheStateStruct), _vp, _vp, _vp]
_lib.dip_stack_step_probed.restype = _i32
_lib.dip_stack_step_probed.argtypes = [_vp, _i32, C.POINTER(MlpWeightsStruct), _vp, _i32, _i32, _i32, _f32,
                                       C.POINTER(CacheStateStruct), C.POINTER(CacheStateStruct), _vp,
                                       C.POINTER(StackProbeStruct), _vp]


class TierStruct(C.Structure):
    _fields_ = [("d", C.c_int32), ("capacity", C.c_int32), ("staging", C.c_int32), ("reserved", C.c_int32),
                ("row_bytes", C.c_uint64), ("backing", _vp), ("arena", _vp), ("slot", _vp), ("loc", _vp),
                ("fetch", _vp), ("split", _vp), ("counters", _vp)]


_lib.dip_mlp_step_tiered.restype = _i32
_lib.dip_mlp_step_tiered.argtypes = [_vp, C.POINTER(MlpWeightsStruct), C.POINTER(TierStruct), C.POINTER(TierStruct),
                                     _vp, _i32, _i32, _f32, C.POINTER(CacheStateStruct),
                                     C.POINTER(CacheStateStruct), _vp, C.POINTER(StepOutputsStruct), _vp]


class NeuronWeightsStruct(C.Structure):
    _fields_ = [("wtype", C.c_int32), ("d_model", C.c_int32), ("d_ff", C.c_int32), ("reserved", C.c_int32),
                ("gate", _vp), ("up", _vp), ("down", _vp)]


PRUNE_BY_GATE, PRUNE_BY_UP = 0, 1
_lib.dip_mlp_step_neuron_pruned.restype = _i32
_lib.dip_mlp_step_neuron_pruned.argtypes = [_vp, C.POINTER(NeuronWeightsStruct), _i32, _vp, _i32, _vp,
                                            _vp, _vp, _vp, _vp, _vp]
_lib.dip_sparse_gemv_down_noalloc.restype = _i32
_lib.dip_sparse_gemv_down_noalloc.argtypes = [C.POINTER(MlpWeightsStruct), _vp, _vp, _i32, _vp, _vp]

EXPORTED = ["dip_create", "dip_create_ex", "dip_destroy", "dip_status_string", "dip_last_error", "dip_sm_count",
            "dip_device_status", "dip_reset_device_status", "dip_selftest_bounded_wait", "dip_stack_step_probed",
            "dip_trace_begin", "dip_trace_reset", "dip_trace_read", "dip_trace_end",
            "dip_packed_bytes", "dip_pack_weights", "dip_mask_topk", "dip_ca_mask",
            "dip_sparse_gemv_gate_up", "dip_sparse_gemv_down", "dip_select_gemv_gate_up", "dip_select_gemv_down",
            "dip_mlp_step",
            "dip_residual_rmsnorm", "dip_stack_step", "dip_mlp_step_tiered", "dip_mlp_step_neuron_pruned",
            "dip_sparse_gemv_down_noalloc"]


class TraceRecord(C.Structure):
    _fields_ = [("kind", C.c_int32), ("reserved", C.c_int32), ("t_start_ns", C.c_uint64),
                ("t_ready_ns", C.c_uint64), ("t_end_ns", C.c_uint64), ("t_aux_ns", C.c_uint64)]


TRACE_KINDS = {1: "select", 2: "select_ca", 3: "cache_update", 4: "gemv_gate_up", 5: "gemv_down",
               6: "tier_assign", 7: "tier_fetch", 8: "tier_split", 9: "rowdot", 10: "tier_install"}
for _name in ("dip_trace_begin", "dip_trace_reset", "dip_trace_end"):
    getattr(_lib, _name).restype = _i32
    getattr(_lib, _name).argtypes = [_vp]
_lib.dip_trace_read.restype = _i32
_lib.dip_trace_read.argtypes = [_vp, C.POINTER(TraceRecord), _i32, C.POINTER(C.c_int)]


class DipError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        msg = _lib.dip_status_string(status).decode()
        super().__init__("%s (status %d)%s" % (msg, status, (": " + detail) if detail else ""))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class Context:
    """A dip_ctx: scratch workspace on one device.  Not for concurrent use from several streams."""

    def __init__(self, device: int = 0, max_d: int = 0, max_batch: int = 0, gemv_segment_bytes: int = 0,
                 gemv_copy_ring: bool = False, coarse_min_d: int = 0, wait_limit_us: int = 0,
                 select_in_product: int = 0):
        """The keyword arguments are the fields of dip_options (0 = the library's default)."""
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2412_01380_b200 needs a CUDA device; there is no CPU path")
        h = _vp()
        opt = OptionsStruct(int(max_d), int(max_batch), int(gemv_segment_bytes), int(bool(gemv_copy_ring)),
                            int(coarse_min_d), int(wait_limit_us), int(select_in_product))
        st = _lib.dip_create_ex(C.byref(h), int(device), C.byref(opt))
        if st != OK:
            raise DipError(st, "dip_create_ex")
        self.handle = h
        self.device = int(device)

    def check(self, st: int) -> None:
        if st != OK:
            raise DipError(st, _lib.dip_last_error(self.handle).decode())

    @property
    def sm_count(self) -> int:
        return _lib.dip_sm_count(self.handle)

    def device_status(self) -> int:
        """Waits for the current stream; 0 unless a kernel gave up a bounded wait."""
        out = C.c_int(-1)
        self.check(_lib.dip_device_status(self.handle, C.byref(out), _stream()))
        return out.value

    def reset_device_status(self) -> None:
        self.check(_lib.dip_reset_device_status(self.handle, _stream()))

    def selftest_bounded_wait(self, limit_us: int, waited_ns: Optional[torch.Tensor] = None) -> None:
        """Enqueue the tiny kernel whose bounded wait runs out (device status becomes 1)."""
        self.check(_lib.dip_selftest_bounded_wait(self.handle, int(limit_us), _ptr(waited_ns), _stream()))

    def trace_begin(self) -> None:
        self.check(_lib.dip_trace_begin(self.handle))

    def trace_reset(self) -> None:
        self.check(_lib.dip_trace_reset(self.handle))

    def trace_end(self) -> None:
        self.check(_lib.dip_trace_end(self.handle))

    def trace_read(self):
        """Records of the launches that ran since the last reset: list of dicts with times in
        microseconds relative to the earliest start."""
        buf = (TraceRecord * 1024)()
        n = C.c_int(0)
        self.check(_lib.dip_trace_read(self.handle, buf, 1024, C.byref(n)))
        recs = [buf[i] for i in range(n.value)]
        if not recs:
            return []
        t0 = min(r.t_start_ns for r in recs)
        return [{"kind": TRACE_KINDS.get(r.kind, str(r.kind)), "start": (r.t_start_ns - t0) / 1e3,
                 "ready": (r.t_ready_ns - t0) / 1e3, "end": (r.t_end_ns - t0) / 1e3,
                 "aux": (r.t_aux_ns - t0) / 1e3 if r.t_aux_ns else None} for r in recs]

    def close(self) -> None:
        if self.handle:
            _lib.dip_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class MlpWeights:
    """Packed weights of one MLP block (device tensors owned here) plus the C struct naming them."""

    def __init__(self, wtype: int, d_model: int, d_ff: int, device):
        self.wtype, self.d_model, self.d_ff = int(wtype), int(d_model), int(d_ff)
        sizes = [_lib.dip_packed_bytes(wtype, d_model, d_ff, w) for w in range(4)]
        if sizes[0] == 0:
            raise DipError(ERR_INVALID_ARG, "unsupported weight type or shape")
        self.gate_up = torch.empty(sizes[0], dtype=torch.uint8, device=device)
        self.down = torch.empty(sizes[1], dtype=torch.uint8, device=device)
        self.gate_up_scales = torch.empty(sizes[2], dtype=torch.uint8, device=device) if sizes[2] else None
        self.down_scales = torch.empty(sizes[3], dtype=torch.uint8, device=device) if sizes[3] else None
        self.struct = MlpWeightsStruct(self.wtype, self.d_model, self.d_ff, 0, _ptr(self.gate_up),
                                       _ptr(self.gate_up_scales), _ptr(self.down), _ptr(self.down_scales))

    @property
    def nbytes(self) -> int:
        return sum(t.numel() for t in (self.gate_up, self.down, self.gate_up_scales, self.down_scales)
                   if t is not None)


class CacheState:
    """Column-cache state of one masked layer input: stamp int32[d], meta int32[8] on the device."""

    def __init__(self, d: int, capacity: int, device, policy: str = "lru"):
        assert policy in ("lru", "lfu")
        self.d, self.capacity, self.policy = int(d), int(capacity), policy
        self.stamp = torch.full((d,), -1, dtype=torch.int32, device=device)
        self.meta = torch.zeros(CACHE_META_INTS, dtype=torch.int32, device=device)
        self.count = torch.zeros(d, dtype=torch.int32, device=device) if policy == "lfu" else None
        self.struct = CacheStateStruct(self.d, self.capacity, _ptr(self.stamp), _ptr(self.meta), _ptr(self.count),
                                       1 if policy == "lfu" else 0, 0)

    def load(self, stamp, n_resident: int, step: int, counters=(0, 0, 0, 0)) -> None:
        self.stamp.copy_(torch.as_tensor(stamp, dtype=torch.int32))
        self.meta.copy_(torch.tensor([n_resident, step, *counters, 0, 0], dtype=torch.int32))


def dip_packed_bytes(wtype: int, d_model: int, d_ff: int, which: int) -> int:
    return int(_lib.dip_packed_bytes(wtype, d_model, d_ff, which))


def dip_pack_weights(ctx: Context, wtype: int, d_model: int, d_ff: int,
                     Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor,
                     Sg: Optional[torch.Tensor] = None, Su: Optional[torch.Tensor] = None,
                     Sd: Optional[torch.Tensor] = None, out: Optional[MlpWeights] = None) -> MlpWeights:
    """Canonical device tensors ([d_out, d_in] row-major) -> packed MlpWeights."""
    if out is None:
        out = MlpWeights(wtype, d_model, d_ff, Wg.device)
    for t in (Wg, Wu, Wd, Sg, Su, Sd):
        assert t is None or (t.is_cuda and t.is_contiguous())
    ctx.check(_lib.dip_pack_weights(ctx.handle, wtype, d_model, d_ff, _ptr(Wg), _ptr(Wu), _ptr(Wd),
                                    _ptr(Sg), _ptr(Su), _ptr(Sd), C.byref(out.struct), _stream()))
    return out


def dip_mask_topk(ctx: Context, x: torch.Tensor, k: int, mask_bits: Optional[torch.Tensor],
                  kept_idx: Optional[torch.Tensor]) -> None:
    batch, d = (1, x.numel()) if x.dim() == 1 else x.shape
    ctx.check(_lib.dip_mask_topk(ctx.handle, _ptr(x), batch, d, int(k), _ptr(mask_bits), _ptr(kept_idx),
                                 _stream()))


def dip_ca_mask(ctx: Context, x: torch.Tensor, k: int, gamma: float, st: CacheState,
                mask_bits: Optional[torch.Tensor], kept_idx: Optional[torch.Tensor]) -> None:
    ctx.check(_lib.dip_ca_mask(ctx.handle, _ptr(x), x.numel(), int(k), float(gamma), C.byref(st.struct),
                               _ptr(mask_bits), _ptr(kept_idx), _stream()))


def dip_sparse_gemv_gate_up(ctx: Context, w: MlpWeights, x: torch.Tensor, kept_idx: torch.Tensor, n_kept: int,
                            mask_bits: Optional[torch.Tensor], h: torch.Tensor) -> None:
    batch = 1 if x.dim() == 1 else x.shape[0]
    ctx.check(_lib.dip_sparse_gemv_gate_up(ctx.handle, C.byref(w.struct), _ptr(x), batch, _ptr(kept_idx),
                                           int(n_kept), _ptr(mask_bits), _ptr(h), _stream()))


def dip_sparse_gemv_down(ctx: Context, w: MlpWeights, h: torch.Tensor, kept_idx: torch.Tensor, n_kept: int,
                         mask_bits: Optional[torch.Tensor], y: torch.Tensor) -> None:
    batch = 1 if h.dim() == 1 else h.shape[0]
    ctx.check(_lib.dip_sparse_gemv_down(ctx.handle, C.byref(w.struct), _ptr(h), batch, _ptr(kept_idx),
                                        int(n_kept), _ptr(mask_bits), _ptr(y), _stream()))


def dip_select_gemv_gate_up(ctx: Context, w: MlpWeights, x: torch.Tensor, k_x: int, gamma: float,
                            cache_gu: Optional[CacheState], cache_d: Optional[CacheState],
                            mask_x: torch.Tensor, h: torch.Tensor) -> None:
    ctx.check(_lib.dip_select_gemv_gate_up(ctx.handle, C.byref(w.struct), _ptr(x), int(k_x), float(gamma),
                                           C.byref(cache_gu.struct) if cache_gu else None,
                                           C.byref(cache_d.struct) if cache_d else None,
                                           _ptr(mask_x), _ptr(h), _stream()))


def dip_select_gemv_down(ctx: Context, w: MlpWeights, h: torch.Tensor, k_h: int, gamma: float,
                         cache_d: Optional[CacheState], mask_h: torch.Tensor, y: torch.Tensor) -> None:
    ctx.check(_lib.dip_select_gemv_down(ctx.handle, C.byref(w.struct), _ptr(h), int(k_h), float(gamma),
                                        C.byref(cache_d.struct) if cache_d else None,
                                        _ptr(mask_h), _ptr(y), _stream()))


def dip_mlp_step(ctx: Context, w: MlpWeights, x: torch.Tensor, k_x: int, k_h: int, gamma: float,
                 cache_gu: Optional[CacheState], cache_d: Optional[CacheState], y: torch.Tensor,
                 mask_x=None, idx_x=None, h=None, mask_h=None, idx_h=None, union_counts=None) -> None:
    batch = 1 if x.dim() == 1 else x.shape[0]
    outs = StepOutputsStruct(_ptr(mask_x), _ptr(idx_x), _ptr(h), _ptr(mask_h), _ptr(idx_h), _ptr(union_counts))
    ctx.check(_lib.dip_mlp_step(ctx.handle, C.byref(w.struct), _ptr(x), batch, int(k_x), int(k_h), float(gamma),
                                C.byref(cache_gu.struct) if cache_gu else None,
                                C.byref(cache_d.struct) if cache_d else None,
                                _ptr(y), C.byref(outs), _stream()))


class Tier:
    """Where the columns of one masked input live: `backing` holds all d packed rows (pinned host
    memory, or a device tensor), the arena on the device holds the cache's columns.  Belongs to
    one CacheState; both start cold."""

    def __init__(self, cache: CacheState, backing: torch.Tensor, row_bytes: int, staging: int, device):
        assert backing.dtype == torch.uint8 and backing.is_contiguous()
        assert backing.numel() == cache.d * row_bytes
        assert backing.is_cuda or backing.is_pinned(), "the slow tier must be readable by the device"
        self.cache, self.backing = cache, backing
        self.d, self.capacity, self.staging, self.row_bytes = cache.d, cache.capacity, int(staging), int(row_bytes)
        words = (self.d + 31) // 32
        self.arena = torch.empty((self.capacity + self.staging) * self.row_bytes, dtype=torch.uint8, device=device)
        self.slot = torch.full((self.d,), -1, dtype=torch.int32, device=device)
        self.loc = torch.zeros(self.d, dtype=torch.int32, device=device)
        self.fetch = torch.zeros(4 + 2 * self.staging, dtype=torch.int32, device=device)
        self.split = torch.zeros(2 * words, dtype=torch.int32, device=device)
        self.counters = torch.zeros(2, dtype=torch.int64, device=device)
        self.struct = TierStruct(self.d, self.capacity, self.staging, 0, self.row_bytes, _ptr(backing),
                                 _ptr(self.arena), _ptr(self.slot), _ptr(self.loc), _ptr(self.fetch),
                                 _ptr(self.split), _ptr(self.counters))


def dip_mlp_step_tiered(ctx: Context, w: MlpWeights, tier_gu: Tier, tier_d: Tier, x: torch.Tensor,
                        k_x: int, k_h: int, gamma: float, y: torch.Tensor,
                        mask_x=None, idx_x=None, h=None, mask_h=None, idx_h=None) -> None:
    """One token through one block with both inputs' weights two-tiered; the caches are the tiers'."""
    outs = StepOutputsStruct(_ptr(mask_x), _ptr(idx_x), _ptr(h), _ptr(mask_h), _ptr(idx_h), None)
    ctx.check(_lib.dip_mlp_step_tiered(ctx.handle, C.byref(w.struct), C.byref(tier_gu.struct),
                                       C.byref(tier_d.struct), _ptr(x), int(k_x), int(k_h), float(gamma),
                                       C.byref(tier_gu.cache.struct), C.byref(tier_d.cache.struct),
                                       _ptr(y), C.byref(outs), _stream()))


class NeuronWeights:
    """Weights of one block laid out by neuron for Gate / Up pruning: gate and up as their own
    row-major [d_ff, d_model] matrices, down as [d_ff, d_model] with row j = W^d[:, j]."""

    def __init__(self, wtype: int, gate: torch.Tensor, up: torch.Tensor, down_t: torch.Tensor):
        d_ff, d_model = gate.shape
        assert up.shape == gate.shape and tuple(down_t.shape) == (d_ff, d_model)
        for t in (gate, up, down_t):
            assert t.is_cuda and t.is_contiguous()
        self.wtype, self.d_model, self.d_ff = int(wtype), int(d_model), int(d_ff)
        self.gate, self.up, self.down = gate, up, down_t
        self.struct = NeuronWeightsStruct(self.wtype, self.d_model, self.d_ff, 0, _ptr(gate), _ptr(up), _ptr(down_t))


def dip_mlp_step_neuron_pruned(ctx: Context, w: NeuronWeights, prune_by: str, x: torch.Tensor, k: int,
                               y: torch.Tensor, p=None, mask=None, idx=None, h=None) -> None:
    """Gate pruning (prune_by="gate") or Up pruning ("up") of one token through one block."""
    assert prune_by in ("gate", "up")
    ctx.check(_lib.dip_mlp_step_neuron_pruned(ctx.handle, C.byref(w.struct),
                                              PRUNE_BY_GATE if prune_by == "gate" else PRUNE_BY_UP, _ptr(x), int(k),
                                              _ptr(y), _ptr(p), _ptr(mask), _ptr(idx), _ptr(h), _stream()))


def dip_residual_rmsnorm(ctx: Context, x: torch.Tensor, y: torch.Tensor, x_next: torch.Tensor) -> None:
    batch, d = (1, x.numel()) if x.dim() == 1 else x.shape
    ctx.check(_lib.dip_residual_rmsnorm(ctx.handle, _ptr(x), _ptr(y), batch, d, _ptr(x_next), _stream()))


class Stack:
    """Host arrays naming the layers (and caches) of an MLP stack for dip_stack_step."""

    def __init__(self, layers: Sequence[MlpWeights], cache_gu: Optional[Sequence[CacheState]] = None,
                 cache_d: Optional[Sequence[CacheState]] = None):
        self.layers: List[MlpWeights] = list(layers)
        self.cache_gu = list(cache_gu) if cache_gu is not None else None
        self.cache_d = list(cache_d) if cache_d is not None else None
        n = len(self.layers)
        self.w_arr = (MlpWeightsStruct * n)(*[l.struct for l in self.layers])
        self.gu_arr = (CacheStateStruct * n)(*[c.struct for c in self.cache_gu]) if self.cache_gu else None
        self.d_arr = (CacheStateStruct * n)(*[c.struct for c in self.cache_d]) if self.cache_d else None


def dip_stack_step(ctx: Context, stack: Stack, x_in: torch.Tensor, k_x: int, k_h: int, gamma: float,
                   x_out: torch.Tensor, y_last: Optional[torch.Tensor] = None) -> None:
    batch = 1 if x_in.dim() == 1 else x_in.shape[0]
    ctx.check(_lib.dip_stack_step(ctx.handle, len(stack.layers), stack.w_arr, _ptr(x_in), batch, int(k_x),
                                  int(k_h), float(gamma), stack.gu_arr, stack.d_arr, _ptr(x_out),
                                  _ptr(y_last), _stream()))


class StackProbe:
    """Per-layer intermediates of one dip_stack_step_probed call (device tensors owned here)."""

    def __init__(self, n_layers: int, batch: int, d_model: int, d_ff: int, device):
        self.x = torch.empty((n_layers, batch, d_model), device=device)
        self.mask_x = torch.zeros((n_layers, batch, d_model // 32), dtype=torch.int32, device=device)
        self.h = torch.empty((n_layers, batch, d_ff), device=device)
        self.mask_h = torch.zeros((n_layers, batch, d_ff // 32), dtype=torch.int32, device=device)
        self.y = torch.empty((n_layers, batch, d_model), device=device)
        self.struct = StackProbeStruct(_ptr(self.x), _ptr(self.mask_x), _ptr(self.h), _ptr(self.mask_h), _ptr(self.y))


def dip_stack_step_probed(ctx: Context, stack: Stack, x_in: torch.Tensor, k_x: int, k_h: int, gamma: float,
                          x_out: torch.Tensor, probe: StackProbe) -> None:
    batch = 1 if x_in.dim() == 1 else x_in.shape[0]
    ctx.check(_lib.dip_stack_step_probed(ctx.handle, len(stack.layers), stack.w_arr, _ptr(x_in), batch, int(k_x),
                                         int(k_h), float(gamma), stack.gu_arr, stack.d_arr, _ptr(x_out),
                                         C.byref(probe.struct), _stream()))


def dip_sparse_gemv_down_noalloc(w: MlpWeights, h: torch.Tensor, kept_idx: torch.Tensor, n_kept: int,
                                 y: torch.Tensor) -> None:
    """y = W~d h without a Context and without any device allocation by the library.

    For callers that cannot let this library allocate: hosts whose memory pool is owned by a
    framework, serving loops that cannot afford the synchronisation an allocation implies, or
    processes with no free device memory left for a Context's workspace.  Scratch comes from a
    fixed ~4 MB array inside the library image, shared by every call on the device, so calls
    that overlap on the GPU race: keep them on one stream.  d_model is limited to 16384
    (ERR_WORKSPACE beyond); F32 and BF16 weights only.  The first call on a device does a
    one-off address look-up and should come before any stream capture.
    """
    st = _lib.dip_sparse_gemv_down_noalloc(C.byref(w.struct), _ptr(h), _ptr(kept_idx), int(n_kept), _ptr(y),
                                           _stream())
    if st == ERR_WORKSPACE:
        raise DipError(st, "d_model exceeds the no-allocation entry point's fixed scratch (max 16384)")
    if st != OK:
        raise DipError(st, "dip_sparse_gemv_down_noalloc")
