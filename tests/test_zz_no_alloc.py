"""The allocation-free down GEMV against the context-based one.

Some callers cannot let a library allocate device memory: they run inside a framework that
owns the device's memory pool, in a serving loop where an allocation (and the device
synchronisation it implies) is not acceptable, or with no free memory left for a context's
workspace.  `dip_sparse_gemv_down_noalloc` serves them from a fixed scratch array inside the
library image.  This test calls it through the C ABI twice in a row (the array keeps the
previous call's contents, so the second call checks that nothing stale leaks through) and
compares with `dip_sparse_gemv_down` on the same inputs.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

import dip_inputs as di
from gpu_util import REL_TOL, rel_err, upload_layer

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wtype,d_model,d_ff", [(di.W_BF16, 5120, 17920), (di.W_F32, 1024, 2816),
                                                (di.W_BF16, 1056, 2848)])
def test_noalloc_down_gemv_matches_context_entry_point(wtype, d_model, d_ff):
    import paper_2412_01380_b200 as dip
    ctx = dip.Context(0)
    wl = di.WORKLOADS["phi3_mini"].scaled(seed=5, d_model=d_model, d_ff=d_ff, wtype=wtype)
    w = upload_layer(dip, ctx, di.layer_weights(wl, 0))
    y_ref = torch.empty(d_model, device="cuda")
    y = torch.empty(d_model, device="cuda")
    # two calls in a row with different inputs and different numbers of kept columns
    for call, (seed, rho) in enumerate([(11, 0.25), (12, 0.1)]):
        h = torch.from_numpy(di.heavy_tail_vector(seed, d_ff)).cuda()
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
