"""GPU parity of the Gate pruning / Up pruning step (Sec. 3.2, Eq. 5) against the oracle.

The ranking activation p is compared within tolerance; the neuron mask must be bit-exact against
the oracle's top-k of the GPU's own p (both sides then rank identical binary32 values); h and y
are compared on that mask."""
import numpy as np
import pytest
import torch

import dip_inputs as di
import oracle
from gpu_util import REL_TOL, bits_to_mask, oracle_mats, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dip():
    import paper_2412_01380_b200 as m
    return m


@pytest.fixture(scope="module")
def ctx(dip):
    c = dip.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


def _neuron_weights(dip, lw):
    """Canonical host matrices -> the neuron-major device layout."""
    if lw.wtype == di.W_BF16:
        g, u = lw.gate.view(np.int16), lw.up.view(np.int16)
        dt = np.ascontiguousarray(lw.down.view(np.int16).T)
    else:
        g, u, dt = lw.gate, lw.up, np.ascontiguousarray(lw.down.T)
    return dip.NeuronWeights(lw.wtype, torch.from_numpy(np.ascontiguousarray(g)).cuda(),
                             torch.from_numpy(np.ascontiguousarray(u)).cuda(), torch.from_numpy(dt).cuda())


def _silu(z):
    return oracle.glu(z, np.ones_like(z))       # Eq. 2 with u = 1, through the oracle


@pytest.mark.parametrize("by", ["gate", "up"])
@pytest.mark.parametrize("wtype,d_model,d_ff,rho", [
    (di.W_BF16, 1024, 4096, 0.25),
    (di.W_BF16, 3072, 8192, 0.1),
    (di.W_F32, 1024, 2816, 0.5),
    (di.W_BF16, 5120, 17920, 0.25),        # Phi-3-Medium block
    (di.W_BF16, 96, 160, 0.3),             # rows shorter than one warp sweep, ragged
    (di.W_F32, 512, 1536, 1.0),            # every neuron kept: the dense MLP
])
def test_neuron_pruned_step_matches_oracle(dip, ctx, by, wtype, d_model, d_ff, rho):
    wl = di.WORKLOADS["phi3_mini"].scaled(seed=31 + d_ff, d_model=d_model, d_ff=d_ff, wtype=wtype)
    lw = di.layer_weights(wl, 0)
    nw = _neuron_weights(dip, lw)
    Wg, Wu, Wd = oracle_mats(lw)
    k = di.keep_count(rho, d_ff)
    xs = di.token_inputs(wl, n_tokens=3, batch=1, d=d_model)[:, 0]
    ones = np.ones(d_model, dtype=np.uint8)
    for x in xs:
        y = torch.empty(d_model, device="cuda")
        p = torch.empty(d_ff, device="cuda")
        h = torch.empty(d_ff, device="cuda")
        mask = torch.zeros((d_ff + 31) // 32, dtype=torch.int32, device="cuda")
        idx = torch.zeros(k, dtype=torch.int32, device="cuda")
        dip.dip_mlp_step_neuron_pruned(ctx, nw, by, torch.from_numpy(x).cuda(), k, y, p=p, mask=mask, idx=idx, h=h)
        torch.cuda.synchronize()
        g = oracle.masked_matvec(Wg, x, ones)
        u = oracle.masked_matvec(Wu, x, ones)
        p_ref = _silu(g) if by == "gate" else u
        p_gpu = p.cpu().numpy()
        assert rel_err(p_gpu, p_ref) <= REL_TOL
        # the mask, on the GPU's own p
        m, idx_ref = oracle.dip_ca_mask(p_gpu, k, 1.0, None)
        assert np.array_equal(bits_to_mask(mask, d_ff), m)
        assert np.array_equal(idx.cpu().numpy(), idx_ref)
        keep = m.astype(bool)
        h_ref = np.where(keep, p_gpu.astype(np.float64) * (u if by == "gate" else _silu(g)), 0.0)
        h_gpu = h.cpu().numpy()
        assert np.all(h_gpu[~keep] == 0.0)
        assert rel_err(h_gpu, h_ref) <= REL_TOL
        y_ref = oracle.masked_matvec(Wd, h_gpu, m)
        assert rel_err(y.cpu().numpy(), y_ref) <= REL_TOL
        # free running: the oracle's whole step, whenever no near-tie of p flipped the mask
        r = oracle.neuron_pruned_step(Wg, Wu, Wd, x, k, by)
        if np.array_equal(r.m, m):
            assert rel_err(y.cpu().numpy(), r.y) <= REL_TOL
    if rho == 1.0:
        _, y_dense = oracle.dense_mlp(Wg, Wu, Wd, xs[-1])
        assert rel_err(y.cpu().numpy(), y_dense) <= REL_TOL
    assert ctx.device_status() == 0


def test_neuron_pruned_step_rejects_bad_arguments(dip, ctx):
    wl = di.WORKLOADS["phi3_mini"].scaled(seed=1, d_model=256, d_ff=512)
    nw = _neuron_weights(dip, di.layer_weights(wl, 0))
    x = torch.zeros(256, device="cuda")
    y = torch.empty(256, device="cuda")
    with pytest.raises(dip.DipError):
        dip.dip_mlp_step_neuron_pruned(ctx, nw, "gate", x, 0, y)
    with pytest.raises(dip.DipError):
        dip.dip_mlp_step_neuron_pruned(ctx, nw, "up", x, 513, y)
    nw.struct.wtype = di.W_INT4_G128
    with pytest.raises(dip.DipError):
        dip.dip_mlp_step_neuron_pruned(ctx, nw, "gate", x, 8, y)
    torch.cuda.synchronize()
