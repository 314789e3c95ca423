"""Helpers shared by the GPU parity tests: upload synthetic layers, wrap oracle matrices, error metric."""
import numpy as np
import torch

import dip_inputs as di
import oracle

REL_TOL = 2e-3   # max relative error, bf16/fp32 weights with binary32 accumulation vs the fp64 oracle


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max_j |got_j - ref_j| / max(|ref_j|, rms(ref)): element-wise relative error with the
    denominator floored at the vector's RMS so that near-zero outputs do not dominate."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref * ref)))
    den = np.maximum(np.abs(ref), max(rms, 1e-300))
    return float(np.max(np.abs(got - ref) / den))


def oracle_mats(lw: di.LayerWeights):
    t = lw.wtype
    return (oracle.Matrix(t, lw.gate, lw.gate_scales, lw.d_ff, lw.d_model),
            oracle.Matrix(t, lw.up, lw.up_scales, lw.d_ff, lw.d_model),
            oracle.Matrix(t, lw.down, lw.down_scales, lw.d_model, lw.d_ff))


def _dev(a, dtype=None):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.cuda()


def upload_layer(dip, ctx, lw: di.LayerWeights):
    """Canonical host arrays -> device -> dip_pack_weights."""
    if lw.wtype == di.W_BF16:
        args = [_dev(lw.gate.view(np.int16)), _dev(lw.up.view(np.int16)), _dev(lw.down.view(np.int16))]
        sc = [None, None, None]
    elif lw.wtype == di.W_F32:
        args = [_dev(lw.gate), _dev(lw.up), _dev(lw.down)]
        sc = [None, None, None]
    else:
        args = [_dev(lw.gate), _dev(lw.up), _dev(lw.down)]
        sc = [_dev(lw.gate_scales.view(np.int16)), _dev(lw.up_scales.view(np.int16)),
              _dev(lw.down_scales.view(np.int16))]
    w = dip.dip_pack_weights(ctx, lw.wtype, lw.d_model, lw.d_ff, *args, *sc)
    torch.cuda.synchronize()
    return w


def bits_to_mask(bits: torch.Tensor, d: int) -> np.ndarray:
    """uint32 words (as int32 tensor) -> uint8 [.., d] 0/1 array."""
    w = bits.cpu().numpy().view(np.uint32)
    m = ((w[..., :, None] >> np.arange(32, dtype=np.uint32)) & 1).astype(np.uint8)
    return m.reshape(*w.shape[:-1], -1)[..., :d]


def gpu_cache_from_oracle(dip, c: "oracle.Cache"):
    g = dip.CacheState(c.d, c.capacity, "cuda", c.policy)
    g.load(c.stamp, int(c.n_resident[0]), int(c.step[0]), tuple(int(v) for v in c.counters))
    if c.policy == "lfu":
        g.count.copy_(torch.from_numpy(c.count))
    return g


def cache_equal(g, c: "oracle.Cache") -> bool:
    meta = g.meta.cpu().numpy()
    if c.policy == "lfu" and not np.array_equal(g.count.cpu().numpy(), c.count):
        return False
    return (np.array_equal(g.stamp.cpu().numpy(), c.stamp) and meta[0] == c.n_resident[0]
            and meta[1] == c.step[0] and np.array_equal(meta[2:6], c.counters))


def check_step(dip, ctx, lw, w, x, k_x, k_h, gamma, ref_gu, ref_d, g_gu, g_d, tiers=None):
    """One dip_mlp_step (tiers given: one dip_mlp_step_tiered) against the oracle.  The first mask sees identical input and must be
    bit-exact; the second mask is checked bit-exactly against the oracle's top-k of the GPU's
    own h; outputs are compared on identical masks."""
    d_model, d_ff = lw.d_model, lw.d_ff
    Wg, Wu, Wd = oracle_mats(lw)
    dev = "cuda"
    y = torch.empty(d_model, device=dev)
    mask_x = torch.zeros((d_model + 31) // 32, dtype=torch.int32, device=dev)
    idx_x = torch.zeros(k_x, dtype=torch.int32, device=dev)
    h = torch.empty(d_ff, device=dev)
    mask_h = torch.zeros((d_ff + 31) // 32, dtype=torch.int32, device=dev)
    idx_h = torch.zeros(k_h, dtype=torch.int32, device=dev)
    if tiers is None:
        dip.dip_mlp_step(ctx, w, torch.from_numpy(x).cuda(), k_x, k_h, gamma, g_gu, g_d, y,
                         mask_x=mask_x, idx_x=idx_x, h=h, mask_h=mask_h, idx_h=idx_h)
    else:
        dip.dip_mlp_step_tiered(ctx, w, tiers[0], tiers[1], torch.from_numpy(x).cuda(), k_x, k_h, gamma, y,
                                mask_x=mask_x, idx_x=idx_x, h=h, mask_h=mask_h, idx_h=idx_h)
    torch.cuda.synchronize()
    # first half
    m_x, idx_x_ref = oracle.dip_ca_mask(x, k_x, gamma, ref_gu)
    assert np.array_equal(bits_to_mask(mask_x, d_model), m_x)
    assert np.array_equal(idx_x.cpu().numpy(), idx_x_ref)
    gg = oracle.masked_matvec(Wg, x, m_x)
    uu = oracle.masked_matvec(Wu, x, m_x)
    h_ref = oracle.glu(gg, uu)
    h_gpu = h.cpu().numpy()
    assert rel_err(h_gpu, h_ref) <= REL_TOL
    # second half, teacher-forced on the GPU's h
    m_h, idx_h_ref = oracle.dip_ca_mask(h_gpu, k_h, gamma, ref_d)
    assert np.array_equal(bits_to_mask(mask_h, d_ff), m_h)
    assert np.array_equal(idx_h.cpu().numpy(), idx_h_ref)
    y_ref = oracle.masked_matvec(Wd, h_gpu, m_h)
    assert rel_err(y.cpu().numpy(), y_ref) <= REL_TOL
    if ref_gu is not None:
        assert cache_equal(g_gu, ref_gu) and cache_equal(g_d, ref_d)
    return y.cpu().numpy()
