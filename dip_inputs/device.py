"""Device-side draw of the same weight recipe (N(0, 0.02), rounded to the storage type) for
full-size stacks, where drawing tens of GB on the host would take minutes.  Seeded per
(workload, layer, role) with torch's device generator; the bytes differ from the host
generator's, the distribution does not.  Draws numbers only: no method arithmetic here.
"""
import torch

from . import W_BF16, W_F32, W_INT4_G128, WEIGHT_STD, GROUP, Workload, _ROLE


def _gen(w: Workload, layer: int, role: str, device, rank: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((w.seed << 40) ^ (w.wid << 32) ^ (rank << 24) ^ (layer << 8) ^ _ROLE[role])
    return g


def _quantize_int4_g128(z: torch.Tensor):
    d_out, d_in = z.shape
    g = z.view(d_out, d_in // GROUP, GROUP)
    s16 = (g.abs().amax(dim=2) / 7.0).to(torch.float16)
    s16 = torch.where(s16 == 0, torch.full_like(s16, 6e-8), s16)
    q = torch.clamp(torch.round(g / s16.float().unsqueeze(2)), -7, 7).to(torch.int16) + 8
    q = q.view(d_out, d_in).to(torch.uint8)
    packed = (q[:, 0::2] | (q[:, 1::2] << 4)).contiguous()
    return packed, s16.t().contiguous()          # scales [d_in/128, d_out]


def matrix(w: Workload, layer: int, role: str, d_out: int, d_in: int, device, rank: int = 0):
    """Canonical [d_out, d_in] matrix in the workload's storage type; returns (tensor, scales or None)."""
    z = torch.randn((d_out, d_in), generator=_gen(w, layer, role, device, rank), device=device,
                    dtype=torch.float32) * WEIGHT_STD
    if w.wtype == W_F32:
        return z, None
    if w.wtype == W_BF16:
        return z.to(torch.bfloat16), None
    if w.wtype == W_INT4_G128:
        return _quantize_int4_g128(z)
    raise ValueError(w.wtype)
