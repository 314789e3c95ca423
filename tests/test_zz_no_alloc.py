"""The allocation-free down GEMV against the context-based one.

Some callers cannot let a library allocate device memory: they run inside a framework that
owns the device's memory pool, in a serving loop where an allocation (and the device
synchronisation it implies) is not acceptable, or with no free memory left for a context's
workspace.  `dip_sparse_gemv_down_noalloc` serves them from a fixed scratch array inside the
library image.  This test calls it through the C ABI twice in a row (the array keeps the
previous call's contents, so the second call checks that nothing stale leaks through) and
compares with `dip_sparse_gemv_down` on the same inputs, and with the CPU oracle's masked
product (Eq. 8) on the same kept set.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

import dip_inputs as di
import oracle
from gpu_util import REL_TOL, oracle_mats, rel_err, upload_layer

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wtype,d_model,d_ff,rhos", [
    (di.W_BF16, 5120, 17920, (0.25, 0.1)), (di.W_F32, 1024, 2816, (0.25, 0.1)), (di.W_BF16, 1056, 2848, (0.25, 0.1)),
    (di.W_BF16, 256, 64, (0.125, 0.05)),       # 8 and 3 kept columns: too few rows to split, one part per segment
])
def test_noalloc_down_gemv_matches_context_entry_point(wtype, d_model, d_ff, rhos):
    import paper_2412_01380_b200 as dip
    ctx = dip.Context(0)
    wl = di.WORKLOADS["phi3_mini"].scaled(seed=5, d_model=d_model, d_ff=d_ff, wtype=wtype)
    lw = di.layer_weights(wl, 0)
    w = upload_layer(dip, ctx, lw)
    Wd = oracle_mats(lw)[2]
    y_ref = torch.empty(d_model, device="cuda")
    y = torch.empty(d_model, device="cuda")
    # two calls in a row with different inputs and different numbers of kept columns
    for call, (seed, rho) in enumerate([(11, rhos[0]), (12, rhos[1])]):
        h_host = di.heavy_tail_vector(seed, d_ff)
        h = torch.from_numpy(h_host).cuda()
        k = di.keep_count(rho, d_ff)
        idx = torch.empty(k, dtype=torch.int32, device="cuda")
        dip.dip_mask_topk(ctx, h, k, None, idx)
        dip.dip_sparse_gemv_down(ctx, w, h, idx, k, None, y_ref)
        y.fill_(float("nan"))
        free_before = torch.cuda.mem_get_info()[0]
        dip.dip_sparse_gemv_down_noalloc(w, h, idx, k, y)
        torch.cuda.synchronize()
        if call > 0:
            # (the very first launch may make the driver load the kernel image, array included)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        got, ref = y.cpu().numpy(), y_ref.cpu().numpy()
        assert np.all(np.isfinite(got)), call
        assert rel_err(got, ref) <= REL_TOL, call
        m = np.zeros(d_ff, dtype=np.uint8)
        m[idx.cpu().numpy()] = 1
        assert rel_err(got, oracle.masked_matvec(Wd, h_host, m)) <= REL_TOL, call
    ctx.close()


def test_noalloc_skips_indices_that_name_no_column():
    """An entry outside [0, d_ff) is skipped instead of being read: the result is the product over
    the valid entries."""
    import paper_2412_01380_b200 as dip
    ctx = dip.Context(0)
    d_model, d_ff = 512, 1024
    wl = di.WORKLOADS["phi3_mini"].scaled(seed=6, d_model=d_model, d_ff=d_ff)
    lw = di.layer_weights(wl, 0)
    w = upload_layer(dip, ctx, lw)
    h_host = di.heavy_tail_vector(13, d_ff)
    good = np.arange(0, d_ff, 4, dtype=np.int32)
    bad = np.concatenate([good[:100], np.array([-1, d_ff, 2 ** 30, -2 ** 31], dtype=np.int32), good[100:]])
    y = torch.full((d_model,), float("nan"), device="cuda")
    dip.dip_sparse_gemv_down_noalloc(w, torch.from_numpy(h_host).cuda(), torch.from_numpy(bad).cuda(), bad.size, y)
    torch.cuda.synchronize()
    m = np.zeros(d_ff, dtype=np.uint8)
    m[good] = 1
    assert rel_err(y.cpu().numpy(), oracle.masked_matvec(oracle_mats(lw)[2], h_host, m)) <= REL_TOL
    ctx.close()


def test_noalloc_rejects_sizes_beyond_its_scratch():
    import paper_2412_01380_b200 as dip
    w = dip.MlpWeights(dip.W_BF16, 32768, 64, "cuda")      # d_model above the entry point's limit
    h = torch.zeros(64, device="cuda")
    idx = torch.arange(8, dtype=torch.int32, device="cuda")
    y = torch.zeros(32768, device="cuda")
    with pytest.raises(dip.DipError) as e:
        dip.dip_sparse_gemv_down_noalloc(w, h, idx, 8, y)
    assert e.value.status == dip.ERR_WORKSPACE
    with pytest.raises(dip.DipError):
        dip.dip_sparse_gemv_down_noalloc(w, h, idx, 0, y)   # n_kept out of range
    torch.cuda.synchronize()
