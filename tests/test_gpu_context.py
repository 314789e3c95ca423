"""Contexts, options and failure paths of the C ABI on the GPU: workspace sizing, rejected
arguments (nothing is launched), and the bounded wait that every copy-ring kernel relies on."""
import numpy as np
import pytest
import torch

import dip_inputs as di
import oracle
from gpu_util import check_step, upload_layer

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dip():
    import paper_2412_01380_b200 as m
    return m


def test_bounded_wait_runs_out_and_the_context_stays_usable(dip):
    """A wait that nothing will ever satisfy gives up after its limit: the kernel returns, the
    sticky status word reads DEVICE_WAIT_TIMEOUT, and after a reset the same context computes a
    correct step."""
    c = dip.Context(0)
    try:
        assert c.device_status() == dip.DEVICE_OK
        waited = torch.zeros(1, dtype=torch.int64, device="cuda")
        c.selftest_bounded_wait(1000, waited)                  # one millisecond
        assert c.device_status() == dip.DEVICE_WAIT_TIMEOUT
        assert 1_000_000 <= int(waited.item()) < 200_000_000   # it waited its limit, and not much more
        assert c.device_status() == dip.DEVICE_WAIT_TIMEOUT    # sticky
        c.reset_device_status()
        assert c.device_status() == dip.DEVICE_OK
        # the copy-ring kernel (INT4) on the same context right after
        wl = di.WORKLOADS["llama3_8b_int4"].scaled(seed=3, d_model=512, d_ff=1024)
        lw = di.layer_weights(wl, 0)
        w = upload_layer(dip, c, lw)
        x = di.token_inputs(wl, n_tokens=1, batch=1)[0, 0]
        check_step(dip, c, lw, w, x, wl.k_x, wl.k_h, 1.0, None, None, None, None)
        assert c.device_status() == dip.DEVICE_OK
        with pytest.raises(dip.DipError):
            c.selftest_bounded_wait(0)
        with pytest.raises(dip.DipError):
            c.selftest_bounded_wait(2_000_000)
    finally:
        torch.cuda.synchronize()
        c.close()


def test_options_size_the_workspace_and_pick_the_kernels(dip):
    wl = di.WORKLOADS["phi3_mini"].scaled(seed=8, d_model=1024, d_ff=2816)
    lw = di.layer_weights(wl, 0)
    x = di.token_inputs(wl, n_tokens=1, batch=1)[0, 0]
    free0 = torch.cuda.mem_get_info()[0]
    small = dip.Context(0, max_d=2816, max_batch=1)
    used_small = free0 - torch.cuda.mem_get_info()[0]
    try:
        w = upload_layer(dip, small, lw)
        check_step(dip, small, lw, w, x, wl.k_x, wl.k_h, 1.0, None, None, None, None)
        # beyond what the workspace was sized for
        big = torch.zeros(4096, device="cuda")
        with pytest.raises(dip.DipError) as e:
            dip.dip_mask_topk(small, big, 8, torch.zeros(128, dtype=torch.int32, device="cuda"), None)
        assert e.value.status == dip.ERR_WORKSPACE
        with pytest.raises(dip.DipError) as e:
            xb = torch.zeros((2, 1024), device="cuda")
            dip.dip_mlp_step(small, w, xb, 8, 8, 1.0, None, None, torch.zeros((2, 1024), device="cuda"))
        assert e.value.status == dip.ERR_WORKSPACE
    finally:
        torch.cuda.synchronize()
        small.close()
    free1 = torch.cuda.mem_get_info()[0]
    full = dip.Context(0)
    used_full = free1 - torch.cuda.mem_get_info()[0]
    full.close()
    assert used_small < used_full
    # forced kernels: copy ring with each segment width, and the 16-bit keys at every size
    for kw in ({"gemv_copy_ring": True}, {"gemv_copy_ring": True, "gemv_segment_bytes": 512},
               {"gemv_copy_ring": True, "gemv_segment_bytes": 1024}, {"coarse_min_d": -1}):
        c = dip.Context(0, **kw)
        try:
            w = upload_layer(dip, c, lw)
            ref_gu, ref_d = oracle.Cache(1024, 512), oracle.Cache(2816, 1408)
            g_gu, g_d = dip.CacheState(1024, 512, "cuda"), dip.CacheState(2816, 1408, "cuda")
            for t in range(2):
                check_step(dip, c, lw, w, x, wl.k_x, wl.k_h, 0.2, ref_gu, ref_d, g_gu, g_d)
            assert c.device_status() == dip.DEVICE_OK
        finally:
            torch.cuda.synchronize()
            c.close()
    for bad in ({"max_d": 40000}, {"max_batch": 17}, {"gemv_segment_bytes": 100}, {"wait_limit_us": -1}):
        with pytest.raises(dip.DipError):
            dip.Context(0, **bad)


def test_misaligned_pointers_are_rejected_before_any_launch(dip):
    """Every vector and mask is read with 16-byte loads somewhere: a tensor slice at a 4-byte offset
    must come back as an error code, not as a misaligned-address fault."""
    c = dip.Context(0)
    try:
        wl = di.WORKLOADS["phi3_mini"].scaled(seed=9, d_model=256, d_ff=512)
        w = upload_layer(dip, c, di.layer_weights(wl, 0))
        f = lambda n: torch.zeros(n + 4, device="cuda")
        i = lambda n: torch.zeros(n + 4, dtype=torch.int32, device="cuda")
        x, y, h = f(256), f(256), f(512)
        mx, mh, idx = i(8), i(16), i(64)

        def rejected(fn):
            with pytest.raises(dip.DipError) as e:
                fn()
            assert e.value.status == dip.ERR_INVALID_ARG

        rejected(lambda: dip.dip_mask_topk(c, x[:256], 8, mx[1:9], None))
        st = dip.CacheState(256, 128, "cuda")
        rejected(lambda: dip.dip_ca_mask(c, x[:256], 8, 0.2, st, mx[1:9], None))
        rejected(lambda: dip.dip_sparse_gemv_gate_up(c, w, x[:256], None, 64, mx[1:9], h[:512]))
        rejected(lambda: dip.dip_sparse_gemv_gate_up(c, w, x[1:257], None, 64, mx[:8], h[:512]))
        rejected(lambda: dip.dip_sparse_gemv_down(c, w, h[:512], None, 64, mh[1:17], y[:256]))
        rejected(lambda: dip.dip_sparse_gemv_down(c, w, h[:512], None, 64, mh[:16], y[1:257]))
        rejected(lambda: dip.dip_mlp_step(c, w, x[:256], 64, 128, 1.0, None, None, y[:256], mask_x=mx[1:9]))
        rejected(lambda: dip.dip_mlp_step(c, w, x[:256], 64, 128, 1.0, None, None, y[:256], mask_h=mh[1:17]))
        rejected(lambda: dip.dip_mlp_step(c, w, x[:256], 64, 128, 1.0, None, None, y[:256], h=h[1:513]))
        rejected(lambda: dip.dip_residual_rmsnorm(c, x[1:257], y[:256], x[:256]))
        rejected(lambda: dip.dip_residual_rmsnorm(c, x[:256], y[1:257], x[:256]))
        rejected(lambda: dip.dip_residual_rmsnorm(c, x[:256], y[:256], x[1:257]))
        stack = dip.Stack([w])
        rejected(lambda: dip.dip_stack_step(c, stack, x[1:257], 64, 128, 1.0, y[:256]))
        rejected(lambda: dip.dip_stack_step(c, stack, x[:256], 64, 128, 1.0, y[1:257]))
        torch.cuda.synchronize()
        # and the aligned calls still work on the same context
        dip.dip_mlp_step(c, w, x[:256], 64, 128, 1.0, None, None, y[:256], mask_x=mx[:8], mask_h=mh[:16], h=h[:512])
        torch.cuda.synchronize()
        assert c.device_status() == dip.DEVICE_OK
    finally:
        torch.cuda.synchronize()
        c.close()
