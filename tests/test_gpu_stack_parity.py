"""Multi-layer parity at the shapes the benchmark times: dip_stack_step (fused rmsnorm select, 16-bit
rank keys from the gate/up product, cache updates on side streams) against the CPU oracle.

Three views of the same run:
  * teacher-forced, layer by layer: the oracle is fed the GPU's own x_l and h_l (binary32), so every
    layer of every token stays comparable: masks, kept sets, cache state and counters bit-exact,
    h, y and the chained x within REL_TOL (Eq. 7-8, Algorithm 1, chaining R13);
  * the same tokens through a captured and replayed CUDA graph of dip_stack_step: x_out and every
    cache state bit-equal to the eager run;
  * free running: the oracle chains its own fp64 results; the first mask that differs must be a
    near-tie of rank keys (relative gap < 1e-3), and is printed.
"""
import numpy as np
import pytest
import torch

import dip_inputs as di
import oracle
from gpu_util import REL_TOL, bits_to_mask, cache_equal, oracle_mats, rel_err, upload_layer

pytestmark = pytest.mark.gpu

NEAR_TIE = 1e-3


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


_LAYER_CACHE = {}


def _layers(dip, ctx, wl, L):
    """Host layers, their oracle views and their packed device copies (kept for the module)."""
    key = (wl.name, wl.seed, wl.d_model, wl.d_ff, wl.wtype, L)
    if key not in _LAYER_CACHE:
        lws = [di.layer_weights(wl, l) for l in range(L)]
        _LAYER_CACHE[key] = (lws, [oracle_mats(lw) for lw in lws], [upload_layer(dip, ctx, lw) for lw in lws])
    return _LAYER_CACHE[key]


def _caches(dip, wl, L, rho, beta, policy="lru"):
    if beta is None:
        return None, None, None, None
    cg, cd = di.cache_capacity(beta, wl.d_model), di.cache_capacity(beta, wl.d_ff)
    return ([oracle.Cache(wl.d_model, cg, policy) for _ in range(L)], [oracle.Cache(wl.d_ff, cd, policy) for _ in range(L)],
            [dip.CacheState(wl.d_model, cg, "cuda", policy) for _ in range(L)],
            [dip.CacheState(wl.d_ff, cd, "cuda", policy) for _ in range(L)])


def _teacher_forced_token(probe, x_in, x_out, mats, k_x, k_h, gamma, ref_gu, ref_d, g_gu, g_d, batch):
    """Check one probed dip_stack_step call layer by layer.  Returns the per-layer masks."""
    L = len(mats)
    X, MX, H, MH, Y = (t.cpu().numpy() for t in (probe.x, probe.mask_x, probe.h, probe.mask_h, probe.y))
    d_model, d_ff = X.shape[2], H.shape[2]
    mx_all, mh_all = bits_to_mask(probe.mask_x, d_model), bits_to_mask(probe.mask_h, d_ff)
    assert np.array_equal(X[0], np.asarray(x_in).reshape(batch, d_model))
    for l in range(L):
        Wg, Wu, Wd = mats[l]
        for b in range(batch):
            x = X[l, b]
            m_x, _ = oracle.dip_ca_mask(x, k_x, gamma, ref_gu[l] if ref_gu else None)
            assert np.array_equal(mx_all[l, b], m_x), ("mask_x", l, b)
            h_ref = oracle.glu(oracle.masked_matvec(Wg, x, m_x), oracle.masked_matvec(Wu, x, m_x))
            assert rel_err(H[l, b], h_ref) <= REL_TOL, ("h", l, b)
            m_h, _ = oracle.dip_ca_mask(H[l, b], k_h, gamma, ref_d[l] if ref_d else None)
            assert np.array_equal(mh_all[l, b], m_h), ("mask_h", l, b)
            y_ref = oracle.masked_matvec(Wd, H[l, b], m_h)
            assert rel_err(Y[l, b], y_ref) <= REL_TOL, ("y", l, b)
            # chaining x_{l+1} = rmsnorm(x_l + y_l) on the GPU's own x_l, y_l
            nxt = X[l + 1, b] if l + 1 < L else x_out.cpu().numpy().reshape(batch, d_model)[b]
            assert rel_err(nxt, oracle.residual_rmsnorm(x, Y[l, b].astype(np.float64))) <= REL_TOL, ("x_next", l, b)
        if ref_gu:
            assert cache_equal(g_gu[l], ref_gu[l]) and cache_equal(g_d[l], ref_d[l]), ("cache", l)
    return mx_all, mh_all


def _free_running_report(xs, mats, k_x, k_h, gamma, caps, gpu_masks, gpu_vecs, gpu_out):
    """The oracle chains its own results; the first differing mask must be a near-tie."""
    L = len(mats)
    d_model, d_ff = mats[0][0].d_in, mats[0][0].d_out
    cg = [oracle.Cache(d_model, caps[0]) for _ in range(L)] if caps else [None] * L
    cd = [oracle.Cache(d_ff, caps[1]) for _ in range(L)] if caps else [None] * L
    for t, x in enumerate(xs):
        cur = x
        for l in range(L):
            res_x = cg[l].resident().copy() if caps else np.ones(d_model, np.uint8)
            res_h = cd[l].resident().copy() if caps else np.ones(d_ff, np.uint8)
            r = oracle.mlp_step(*mats[l], cur, k_x, k_h, gamma, cg[l], cd[l])
            for name, got, ref_m, vec, res in (("x", gpu_masks[t][0][l, 0], r.m_x, gpu_vecs[t][0][l, 0], res_x),
                                               ("h", gpu_masks[t][1][l, 0], r.m_h, gpu_vecs[t][1][l, 0], res_h)):
                diff = np.nonzero(got != ref_m)[0]
                if len(diff):
                    keys = np.array([oracle.rank_key(float(vec[i]), bool(res[i]), gamma) for i in diff],
                                    dtype=np.uint32).view(np.float32)
                    gap = float(keys.max() / keys.min() - 1.0) if keys.min() > 0 else float("inf")
                    print("first mask flip: token %d layer %d input %s columns %s keys %s relative gap %.3g"
                          % (t, l, name, diff.tolist(), keys.tolist(), gap))
                    assert len(diff) % 2 == 0
                    assert gap < NEAR_TIE
                    return (t, l, name)
            cur = oracle.residual_rmsnorm(cur, r.y)
        assert rel_err(gpu_out[t], cur) <= REL_TOL, ("x_out", t)
    print("free-running run: no mask flip in %d tokens x %d layers" % (len(xs), L))
    return None


def _run_stack_case(dip, ctx, wl, L, n_tok, rho, beta, graph=True, free_running=True):
    lws, mats, ws = _layers(dip, ctx, wl, L)
    d_model, d_ff = wl.d_model, wl.d_ff
    k_x, k_h = di.keep_count(rho, d_model), di.keep_count(rho, d_ff)
    gamma = wl.gamma if beta is not None else 1.0
    ref_gu, ref_d, g_gu, g_d = _caches(dip, wl, L, rho, beta)
    xs = di.token_inputs(wl, n_tokens=n_tok, batch=1)[:, 0]
    stack = dip.Stack(ws, g_gu, g_d)
    probe = dip.StackProbe(L, 1, d_model, d_ff, "cuda")
    x_cur = torch.empty(d_model, device="cuda")
    x_out = torch.empty(d_model, device="cuda")

    # the timed route: dip_stack_step captured once, replayed per token, on cache states of its own
    if graph:
        _, _, r_gu, r_d = _caches(dip, wl, L, rho, beta)
        stack_r = dip.Stack(ws, r_gu, r_d)
        x_out_r = torch.empty(d_model, device="cuda")
        side = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            x_cur.copy_(torch.from_numpy(xs[0]).cuda())
            dip.dip_stack_step(ctx, stack_r, x_cur, k_x, k_h, gamma, x_out_r)     # prime outside the capture
            side.synchronize()
            if r_gu:
                for c in r_gu + r_d:                                              # back to cold
                    c.stamp.fill_(-1)
                    c.meta.zero_()
            side.synchronize()
            with torch.cuda.graph(g, stream=side):
                dip.dip_stack_step(ctx, stack_r, x_cur, k_x, k_h, gamma, x_out_r)
        torch.cuda.synchronize()

    masks, vecs, outs = [], [], []
    for t, x in enumerate(xs):
        x_cur.copy_(torch.from_numpy(x).cuda())
        dip.dip_stack_step_probed(ctx, stack, x_cur, k_x, k_h, gamma, x_out, probe)
        torch.cuda.synchronize()
        mx, mh = _teacher_forced_token(probe, x, x_out, mats, k_x, k_h, gamma, ref_gu, ref_d, g_gu, g_d, 1)
        masks.append((mx, mh))
        vecs.append((probe.x.cpu().numpy().copy(), probe.h.cpu().numpy().copy()))
        outs.append(x_out.cpu().numpy().copy())
        if graph:
            g.replay()
            torch.cuda.synchronize()
            assert torch.equal(x_out_r, x_out), ("graph replay differs from the eager run", t)
            if r_gu:
                for l in range(L):
                    assert torch.equal(r_gu[l].stamp, g_gu[l].stamp) and torch.equal(r_gu[l].meta, g_gu[l].meta), (t, l)
                    assert torch.equal(r_d[l].stamp, g_d[l].stamp) and torch.equal(r_d[l].meta, g_d[l].meta), (t, l)
    assert ctx.device_status() == 0
    if free_running:
        caps = (ref_gu[0].capacity, ref_d[0].capacity) if ref_gu else None
        _free_running_report(xs, mats, k_x, k_h, gamma, caps, masks, vecs, outs)


@pytest.mark.parametrize("rho,beta", [(0.25, 0.5), (0.5, 0.25)])
def test_phi3_medium_stack_matches_oracle_eager_and_graph(dip, ctx, rho, beta):
    """The benchmark's configuration (5120 / 17920, bf16, DIP-CA) on 4 layers x 6 tokens: at this
    width the default context ranks h from the 16-bit keys; beta 0.25 with rho 0.5 has k > capacity."""
    _run_stack_case(dip, ctx, di.WORKLOADS["phi3_medium"], 4, 6, rho, beta)


def test_phi3_mini_stack_matches_oracle(dip, ctx):
    wl = di.WORKLOADS["phi3_mini"]
    _run_stack_case(dip, ctx, wl, 3, 8, wl.keep_ratio, wl.cache_budget)


def test_phi3_mini_stack_with_select_kernels_in_front(dip):
    """The same stack on a context created with select_in_product < 0: four launches per layer."""
    wl = di.WORKLOADS["phi3_mini"]
    c = dip.Context(0, select_in_product=-1)
    try:
        _run_stack_case(dip, c, wl, 2, 4, wl.keep_ratio, wl.cache_budget)
    finally:
        torch.cuda.synchronize()
        c.close()


def test_llama3_8b_int4_stack_matches_oracle(dip, ctx):
    wl = di.WORKLOADS["llama3_8b_int4"]
    _run_stack_case(dip, ctx, wl, 2, 6, wl.keep_ratio, wl.cache_budget)


def test_block_f32_all_tokens_match_oracle(dip, ctx):
    """Configuration 1: one fp32 block, all 64 tokens, keep ratio 0.5, no cache."""
    wl = di.WORKLOADS["block_f32"]
    _run_stack_case(dip, ctx, wl, 1, wl.n_tokens, wl.keep_ratio, None)


@pytest.mark.parametrize("batch", [2, 4, 8])
def test_phi3_medium_batched_stack_matches_oracle(dip, ctx, batch):
    """Batched decode through 2 layers at 5120 / 17920: every token against its own oracle run."""
    wl = di.WORKLOADS["phi3_medium_batched"]
    L = 2
    lws, mats, ws = _layers(dip, ctx, wl, L)
    k_x, k_h = wl.k_x, wl.k_h
    xs = di.token_inputs(wl, n_tokens=2, batch=batch)
    stack = dip.Stack(ws)
    probe = dip.StackProbe(L, batch, wl.d_model, wl.d_ff, "cuda")
    x_out = torch.empty((batch, wl.d_model), device="cuda")
    x_plain = torch.empty_like(x_out)
    for x in xs:
        xg = torch.from_numpy(np.ascontiguousarray(x)).cuda()
        dip.dip_stack_step_probed(ctx, stack, xg, k_x, k_h, 1.0, x_out, probe)
        dip.dip_stack_step(ctx, stack, xg, k_x, k_h, 1.0, x_plain)
        torch.cuda.synchronize()
        assert torch.equal(x_plain, x_out)
        _teacher_forced_token(probe, x, x_out, mats, k_x, k_h, 1.0, None, None, None, None, batch)
    assert ctx.device_status() == 0


def test_stack_deeper_than_the_mask_ring(dip, ctx):
    """More layers than the stack runner has per-layer mask slots (the cache updates of early layers
    are joined before their slots are reused): same bits as the probed run, which is checked
    against the oracle layer by layer."""
    L, d_model, d_ff = 131, 128, 256
    wl = di.WORKLOADS["phi3_mini"].scaled(seed=91, n_layers=L, d_model=d_model, d_ff=d_ff)
    base = [di.layer_weights(wl, l) for l in range(3)]
    lws = [base[l % 3] for l in range(L)]
    mats = [oracle_mats(lw) for lw in lws]
    wdev = [upload_layer(dip, ctx, lw) for lw in base]
    ws = [wdev[l % 3] for l in range(L)]
    k_x, k_h, gamma = wl.k_x, wl.k_h, wl.gamma
    ref_gu, ref_d, g_gu, g_d = _caches(dip, wl, L, wl.keep_ratio, wl.cache_budget)
    _, _, p_gu, p_d = _caches(dip, wl, L, wl.keep_ratio, wl.cache_budget)
    xs = di.token_inputs(wl, n_tokens=3, batch=1)[:, 0]
    plain, probed = dip.Stack(ws, p_gu, p_d), dip.Stack(ws, g_gu, g_d)
    probe = dip.StackProbe(L, 1, d_model, d_ff, "cuda")
    x_out, x_plain = torch.empty(d_model, device="cuda"), torch.empty(d_model, device="cuda")
    for x in xs:
        xg = torch.from_numpy(x).cuda()
        dip.dip_stack_step_probed(ctx, probed, xg, k_x, k_h, gamma, x_out, probe)
        dip.dip_stack_step(ctx, plain, xg, k_x, k_h, gamma, x_plain)
        torch.cuda.synchronize()
        _teacher_forced_token(probe, x, x_out, mats, k_x, k_h, gamma, ref_gu, ref_d, g_gu, g_d, 1)
        assert torch.equal(x_plain, x_out)
        for l in range(L):
            assert torch.equal(p_gu[l].stamp, g_gu[l].stamp) and torch.equal(p_d[l].stamp, g_d[l].stamp), l
            assert torch.equal(p_gu[l].meta, g_gu[l].meta) and torch.equal(p_d[l].meta, g_d[l].meta), l


def test_saved_and_restored_cache_state_continues_bit_exactly(dip, ctx):
    """2N tokens in one go == N tokens, a copy of the state buffers into fresh ones, N more tokens."""
    L, d_model, d_ff, N = 3, 1024, 4096, 5
    wl = di.WORKLOADS["phi3_mini"].scaled(seed=93, n_layers=L, d_model=d_model, d_ff=d_ff)
    ws = [upload_layer(dip, ctx, di.layer_weights(wl, l)) for l in range(L)]
    k_x, k_h, gamma = wl.k_x, wl.k_h, wl.gamma
    xs = di.token_inputs(wl, n_tokens=2 * N, batch=1)[:, 0]
    for policy in ("lru", "lfu"):
        _, _, a_gu, a_d = _caches(dip, wl, L, wl.keep_ratio, wl.cache_budget, policy)
        _, _, b_gu, b_d = _caches(dip, wl, L, wl.keep_ratio, wl.cache_budget, policy)
        sa, sb = dip.Stack(ws, a_gu, a_d), dip.Stack(ws, b_gu, b_d)
        out_a, out_b = torch.empty(d_model, device="cuda"), torch.empty(d_model, device="cuda")
        outs_a = []
        for x in xs:
            dip.dip_stack_step(ctx, sa, torch.from_numpy(x).cuda(), k_x, k_h, gamma, out_a)
            torch.cuda.synchronize()
            outs_a.append(out_a.clone())
        for x in xs[:N]:
            dip.dip_stack_step(ctx, sb, torch.from_numpy(x).cuda(), k_x, k_h, gamma, out_b)
        torch.cuda.synchronize()
        # save = copy the buffers out; restore = copy them into brand-new state objects
        _, _, c_gu, c_d = _caches(dip, wl, L, wl.keep_ratio, wl.cache_budget, policy)
        for src, dst in zip(b_gu + b_d, c_gu + c_d):
            saved = (src.stamp.cpu(), src.meta.cpu(), src.count.cpu() if policy == "lfu" else None)
            dst.stamp.copy_(saved[0])
            dst.meta.copy_(saved[1])
            if policy == "lfu":
                dst.count.copy_(saved[2])
        sc = dip.Stack(ws, c_gu, c_d)
        for t, x in enumerate(xs[N:]):
            dip.dip_stack_step(ctx, sc, torch.from_numpy(x).cuda(), k_x, k_h, gamma, out_b)
            torch.cuda.synchronize()
            assert torch.equal(out_b, outs_a[N + t]), (policy, t)
        for l in range(L):
            assert torch.equal(c_gu[l].stamp, a_gu[l].stamp) and torch.equal(c_gu[l].meta, a_gu[l].meta)
            assert torch.equal(c_d[l].stamp, a_d[l].stamp) and torch.equal(c_d[l].meta, a_d[l].meta)
            if policy == "lfu":
                assert torch.equal(c_gu[l].count, a_gu[l].count) and torch.equal(c_d[l].count, a_d[l].count)
