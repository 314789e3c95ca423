#!/usr/bin/env python
"""Benchmark of the sparse SwiGLU decode-MLP path (DIP / DIP-CA) on B200.

A step is one decode token through the whole MLP stack of the workload (n_layers MLP-steps:
mask x, gate/up GEMV + silu*up, mask h, down GEMV, residual + rmsnorm per layer).  The layers
are distinct and the stack is far larger than L2, so every step streams its kept weight
columns from HBM.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload NAME] [--keep-ratio R] [--cache-budget B] [--no-sweep]

With N > 1 (torchrun) every rank runs an independent replica of the stack on its own
sequence ("replicas only": the path has no exchange step); value = MLP-steps of all ranks
divided by the slowest rank's time.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import dip_inputs as di  # noqa: E402

METRIC = "sparse_swiglu_decode_mlp_steps_per_s"
UNIT = "MLP-steps/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="phi3_medium", choices=sorted(di.WORKLOADS))
    ap.add_argument("--keep-ratio", type=float, default=None)
    ap.add_argument("--cache-budget", type=float, default=None)
    ap.add_argument("--batch", type=int, default=1, help="tokens per step (batched decode; cache-aware masking off)")
    ap.add_argument("--policy", default="lru", choices=["lru", "lfu"], help="eviction policy of the column caches")
    ap.add_argument("--layers", type=int, default=None, help="use fewer layers (debugging; not a valid bench)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--min-timed-s", type=float, default=0.5,
                    help="repeat the timed region of --steps steps until this much time has been timed (profiling runs: 0)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--report", default=None, metavar="FILE",
                    help="run every workload of the five configurations (fewer steps) and write a markdown table")
    ap.add_argument("--two-tier", action="store_true",
                    help="time the two-tier step instead: cache arena in HBM, all weights in pinned host memory")
    ap.add_argument("--schedule", default="dip", choices=["dip", "gate", "up"],
                    help="dip: input pruning (the headline); gate / up: Gate / Up pruning of Eq. 5 (neuron-wise)")
    ap.add_argument("--token-correlation", type=float, default=0.0,
                    help="mix consecutive tokens (x_t = c x_{t-1} + sqrt(1-c^2) draw); 0 = independent tokens")
    ap.add_argument("--timeline", action="store_true",
                    help="print the device-side timeline of one graph replay (per kernel: start, ready, end) and exit")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def weight_bytes(wtype):
    return {di.W_F32: 4.0, di.W_BF16: 2.0, di.W_INT4_G128: 0.5}[wtype]


def algorithmic_bytes(w, k_x, k_h, ca):
    """Bytes the method has to move per MLP-step: the kept weight columns plus activations,
    index lists and (cache-aware masking on) the cache stamps.  INT4 adds the scale rows of the
    groups touched (bounded by all groups)."""
    bw = weight_bytes(w.wtype)
    gu = k_x * 2 * w.d_ff * bw + 4 * w.d_model + 4 * k_x + 4 * w.d_ff
    dn = k_h * w.d_model * bw + 4 * w.d_ff + 4 * k_h + 4 * w.d_model
    if w.wtype == di.W_INT4_G128:
        gu += min(k_x, w.d_model // di.GROUP) * 2 * w.d_ff * 2
        dn += min(k_h, w.d_ff // di.GROUP) * w.d_model * 2
    masks = 4 * (w.d_model + w.d_ff) + 4 * (k_x + k_h)
    if ca:
        masks += 8 * (w.d_model + w.d_ff)
    return {"gate_up": gu, "down": dn, "step": gu + dn + masks}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# dram__bytes_read.sum + dram__bytes_write.sum of one gate/up GEMV launch at Phi-3-Medium shapes, keep
# ratio 0.25, one token, from the committed ncu capture (profiles/): bytes, and the kernel it is of.
NCU_TRAFFIC = {"kernel": "gemv_fused_kernel", "bytes": 94.1e6,
               "source": "profiles/kernels_fused_phi3_medium_4layers_rho025.md"}


def ncu_traffic(w, keep_ratio, batch, kernel_name):
    """The committed capture's DRAM traffic per launch, only for the exact kernel, workload and keep
    ratio it was taken on; null for anything else (nothing is extrapolated)."""
    if w.name != "phi3_medium" or batch != 1 or abs(keep_ratio - 0.25) > 1e-9:
        return None
    if not kernel_name.startswith(NCU_TRAFFIC["kernel"]):
        return None
    return NCU_TRAFFIC["bytes"]


def median_repeat(ms_list):
    """The median of the repeats' times (the upper one for an even count, so it is a measured repeat)."""
    s = sorted(ms_list)
    return s[len(s) // 2]


def GATE_UP_KERNEL(w, batch, select_in_product=True):
    """Name of the kernel that computes the gate/up product for this workload."""
    if w.wtype == di.W_INT4_G128:
        return "gemv_int4_kernel"
    if batch == 1:
        return "gemv_fused_kernel" if select_in_product else "gemv_direct_kernel"
    return "gemv_kernel" if batch == 2 else "gemv_tc_kernel"


def max_over_ranks(ms, dist, torch, device):
    """Slowest rank's time (the job is as fast as its slowest replica)."""
    if dist is None:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank, world, ms):
    """Units processed by all ranks (replicas, equal work each) per second of the slowest rank."""
    return units_per_rank * world / (ms * 1e-3)


def simulator_view(w, n_layers, meta_gu, meta_d, dram_gbs=60.0, flash_gbs=1.0, bytes_per_weight=0.5):
    """The run's hit/miss counters pushed through the paper's memory model (Sec. 6, App. A: a phone
    with DRAM 60 GB/s and Flash 1 GB/s, INT4 weights, compute ignored; MLP weights only): every
    kept column is read from DRAM, every missed column is first loaded from Flash.  Context for
    the paper's simulated tok/s, not a measurement of this machine."""
    used_gu, used_d = meta_gu[2] + meta_gu[3], meta_d[2] + meta_d[3]
    tokens = max(1, meta_gu[1] // max(1, n_layers))
    col_gu, col_d = 2 * w.d_ff * bytes_per_weight, w.d_model * bytes_per_weight
    dram = (used_gu * col_gu + used_d * col_d) / tokens
    flash = (meta_gu[3] * col_gu + meta_d[3] * col_d) / tokens
    dense = n_layers * 3 * w.d_model * w.d_ff * bytes_per_weight
    t_sparse = dram / (dram_gbs * 1e9) + flash / (flash_gbs * 1e9)
    # dense model with the same cache budget: the cached share from DRAM, the rest from Flash each token
    return {"dram_gbs": dram_gbs, "flash_gbs": flash_gbs, "bytes_per_weight": bytes_per_weight,
            "dram_bytes_per_token": dram, "flash_bytes_per_token": flash,
            "mlp_tokens_per_s": 1.0 / t_sparse if t_sparse > 0 else None,
            "dense_mlp_bytes_per_token": dense}


def build_stack(dip, ctx, torch, w, n_layers, rank):
    """Draw and pack the stack's weights on the device (one canonical layer at a time)."""
    from dip_inputs import device as dd
    dev = "cuda"
    layers = []
    for l in range(n_layers):
        g, gs = dd.matrix(w, l, "gate", w.d_ff, w.d_model, dev, rank)
        u, us = dd.matrix(w, l, "up", w.d_ff, w.d_model, dev, rank)
        d_, ds = dd.matrix(w, l, "down", w.d_model, w.d_ff, dev, rank)
        layers.append(dip.dip_pack_weights(ctx, w.wtype, w.d_model, w.d_ff, g, u, d_, gs, us, ds))
        torch.cuda.synchronize()
        del g, u, d_, gs, us, ds
    return layers


def run_config(dip, ctx, torch, w, layers, xs_host, keep_ratio, budget, steps, warmup, use_graph=True,
               kernel_pass=True, e2e_pass=True, sampler=None, dist=None, policy="lru", min_timed_s=0.5, min_repeats=3):
    """Time `steps` decode tokens through the stack at one (keep ratio, cache budget)."""
    L, d_model, d_ff = len(layers), w.d_model, w.d_ff
    k_x, k_h = di.keep_count(keep_ratio, d_model), di.keep_count(keep_ratio, d_ff)
    ca = budget is not None
    gamma = w.gamma if ca else 1.0

    def fresh_stack():
        if not ca:
            return dip.Stack(layers)
        cg = [dip.CacheState(d_model, di.cache_capacity(budget, d_model), "cuda", policy) for _ in range(L)]
        cd = [dip.CacheState(d_ff, di.cache_capacity(budget, d_ff), "cuda", policy) for _ in range(L)]
        return dip.Stack(layers, cg, cd)

    n_tok = xs_host.shape[0]
    xs_dev = xs_host.cuda()
    # xs_host is [tokens, d_model] (one sequence) or [tokens, batch, d_model] (batched decode)
    batch = 1 if xs_host.dim() == 2 else xs_host.shape[1]
    x_cur = torch.empty(tuple(xs_host.shape[1:]), device="cuda")
    x_out = torch.empty_like(x_cur)
    out_host = torch.empty(tuple(xs_host.shape[1:])).pin_memory()
    stack = fresh_stack()
    stream = torch.cuda.current_stream()

    graph = None
    if use_graph:
        # capture one token through the stack; replays read x_cur and update the caches in place
        x_cur.copy_(xs_dev[0])
        dip.dip_stack_step(ctx, stack, x_cur, k_x, k_h, gamma, x_out)      # prime outside capture
        torch.cuda.synchronize()
        stack = fresh_stack()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            dip.dip_stack_step(ctx, stack, x_cur, k_x, k_h, gamma, x_out)

    def one_step(t):
        x_cur.copy_(xs_dev[t % n_tok], non_blocking=True)
        if graph is not None:
            graph.replay()
        else:
            dip.dip_stack_step(ctx, stack, x_cur, k_x, k_h, gamma, x_out)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def check_status(where):
        st = ctx.device_status()
        if st != 0:
            raise SystemExit("device status %d after %s: a kernel gave up a bounded wait; no number is printed"
                             % (st, where))

    # ---- device-resident timing: the region of `steps` steps is repeated until at least
    #      min_timed_s have been timed (and at least 3 times); the median repeat is reported ----
    for t in range(warmup):
        one_step(t)
    barrier()
    if sampler:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps, tok = [], warmup
    while len(reps) < min_repeats or (sum(reps) < min_timed_s * 1e3 and len(reps) < 64):
        barrier()
        e0.record(stream)
        for t in range(steps):
            one_step(tok + t)
        e1.record(stream)
        barrier()
        tok += steps
        reps.append(max_over_ranks(e0.elapsed_time(e1), dist, torch, "cuda"))
    clocks = sampler.stop() if sampler else None
    check_status("the timed region")
    ms = median_repeat(reps)
    res = {"keep_ratio": keep_ratio, "cache_budget": budget, "k_x": k_x, "k_h": k_h, "ms_total": ms,
           "ms_per_step": ms / steps, "mlp_steps_per_s": L * steps / (ms * 1e-3), "clocks": clocks,
           "repeats": {"n": len(reps), "ms_min": min(reps), "ms_median": ms, "ms_max": max(reps),
                       "timed_s": sum(reps) * 1e-3},
           "bytes": algorithmic_bytes(w, k_x, k_h, ca)}
    res["step_gbs"] = res["bytes"]["step"] * L * steps / (ms * 1e-3) / 1e9
    res["batch"] = batch
    if batch > 1:
        # density of the union of the tokens' masks (measured on layer 0): the share of a layer's
        # columns that a batched step reads
        counts = torch.zeros(2, dtype=torch.int32, device="cuda")
        y_tmp = torch.empty_like(x_cur)
        dip.dip_mlp_step(ctx, layers[0], xs_dev[0], k_x, k_h, gamma, None, None, y_tmp, union_counts=counts)
        ux, uh = counts.cpu().tolist()
        res["union_density"] = {"x": ux / d_model, "h": uh / d_ff}
        ub = weight_bytes(w.wtype)
        res["union_bytes"] = ux * 2 * d_ff * ub + uh * d_model * ub
        res["union_gbs"] = res["union_bytes"] * L * steps / (ms * 1e-3) / 1e9
    if ca:
        mg = torch.stack([c.meta for c in stack.cache_gu]).sum(0).cpu().tolist()
        md = torch.stack([c.meta for c in stack.cache_d]).sum(0).cpu().tolist()
        res["hit_rate"] = (mg[2] + md[2]) / max(1, mg[2] + mg[3] + md[2] + md[3])
        res["paper_simulator_view"] = simulator_view(w, L, mg, md)

    # ---- end to end: host buffers in, host result out, every step ----
    if e2e_pass:
        xs_pin = xs_host.pin_memory()
        n_e2e = min(steps, 128)
        for t in range(3):
            one_step(t)
        barrier()
        t0 = time.perf_counter()
        e0.record(stream)
        for t in range(n_e2e):
            x_cur.copy_(xs_pin[(warmup + t) % n_tok], non_blocking=True)
            if graph is not None:
                graph.replay()
            else:
                dip.dip_stack_step(ctx, stack, x_cur, k_x, k_h, gamma, x_out)
            out_host.copy_(x_out, non_blocking=True)
            stream.synchronize()          # a decode loop needs the result before the next token
        e1.record(stream)
        barrier()
        ms_e = e0.elapsed_time(e1)
        ms_e = max_over_ranks(ms_e, dist, torch, "cuda")
        check_status("the end-to-end region")
        res["e2e"] = {"value": L * n_e2e / (ms_e * 1e-3), "unit": UNIT, "steps": n_e2e,
                      "h2d_bytes_per_step": 4 * d_model * batch, "d2h_bytes_per_step": 4 * d_model * batch,
                      "wall_ms": (time.perf_counter() - t0) * 1e3}

    # ---- per-kernel durations (separate instrumented pass, one event pair per launch) ----
    if kernel_pass and batch == 1:
        st2 = fresh_stack()
        mask_x = torch.zeros((d_model + 31) // 32, dtype=torch.int32, device="cuda")
        idx_x = torch.zeros(k_x, dtype=torch.int32, device="cuda")
        mask_h = torch.zeros((d_ff + 31) // 32, dtype=torch.int32, device="cuda")
        idx_h = torch.zeros(k_h, dtype=torch.int32, device="cuda")
        h = torch.empty(d_ff, device="cuda")
        y = torch.empty(d_model, device="cuda")
        n_pass_tok = 6
        # A step of this configuration runs each mask together with its product (one launch each) when the
        # library supports that for the weights and shape; otherwise a select kernel precedes each product.
        try:
            dip.dip_select_gemv_gate_up(ctx, layers[0], xs_dev[0].clone(), k_x, gamma,
                                        st2.cache_gu[0] if ca else None, st2.cache_d[0] if ca else None, mask_x, h)
            fused = True
        except dip.DipError:
            fused = False
        res["select_in_product"] = fused
        cg = (lambda l: st2.cache_gu[l]) if ca else (lambda l: None)
        cd = (lambda l: st2.cache_d[l]) if ca else (lambda l: None)
        if fused:
            names = ["select_gate_up", "select_down", "rmsnorm"]
        else:
            names = ["mask_x", "gate_up", "mask_h", "down", "rmsnorm"]   # mask_* = select (+ cache update when on)
        evs = []
        for t in range(n_pass_tok):
            cur = xs_dev[t % n_tok].clone()
            for l in range(L):
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)]
                ev[0].record(stream)
                if fused:
                    dip.dip_select_gemv_gate_up(ctx, layers[l], cur, k_x, gamma, cg(l), cd(l), mask_x, h)
                    ev[1].record(stream)
                    dip.dip_select_gemv_down(ctx, layers[l], h, k_h, gamma, cd(l), mask_h, y)
                    ev[2].record(stream)
                else:
                    if ca:
                        dip.dip_ca_mask(ctx, cur, k_x, gamma, st2.cache_gu[l], mask_x, None)
                    else:
                        dip.dip_mask_topk(ctx, cur, k_x, mask_x, None)
                    ev[1].record(stream)
                    dip.dip_sparse_gemv_gate_up(ctx, layers[l], cur, None, k_x, mask_x, h)
                    ev[2].record(stream)
                    if ca:
                        dip.dip_ca_mask(ctx, h, k_h, gamma, st2.cache_d[l], mask_h, None)
                    else:
                        dip.dip_mask_topk(ctx, h, k_h, mask_h, None)
                    ev[3].record(stream)
                    dip.dip_sparse_gemv_down(ctx, layers[l], h, None, k_h, mask_h, y)
                    ev[4].record(stream)
                dip.dip_residual_rmsnorm(ctx, cur, y, cur)
                ev[len(names)].record(stream)
                if t >= 2:
                    evs.append(ev)
        torch.cuda.synchronize()
        kern = {}
        for i, n in enumerate(names):
            kern[n + "_us"] = float(np.mean([e[i].elapsed_time(e[i + 1]) for e in evs])) * 1e3
        # The products again as a train of launches: one event pair around the launch of every
        # layer (distinct weights, so each launch streams from HBM), twice.  The mean is the
        # kernel's launch duration without the event pair's own overhead on every launch.  With
        # select_in_product the launch is the step's own kernel: the select of the input and the product.
        if fused:
            calls = (("gate_up", lambda l: dip.dip_select_gemv_gate_up(ctx, layers[l], cur, k_x, gamma, cg(l), cd(l), mask_x, h)),
                     ("down", lambda l: dip.dip_select_gemv_down(ctx, layers[l], h, k_h, gamma, cd(l), mask_h, y)))
        else:
            calls = (("gate_up", lambda l: dip.dip_sparse_gemv_gate_up(ctx, layers[l], cur, None, k_x, mask_x, h)),
                     ("down", lambda l: dip.dip_sparse_gemv_down(ctx, layers[l], h, None, k_h, mask_h, y)))
        for name, call in calls:
            for l in range(min(L, 3)):
                call(l)
            ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ea.record(stream)
            for rep in range(2):
                for l in range(L):
                    call(l)
            eb.record(stream)
            torch.cuda.synchronize()
            kern[name + "_train_us"] = ea.elapsed_time(eb) * 1e3 / (2 * L)
        check_status("the per-kernel pass")
        res["kernels"] = kern
    return res


def host_link_peak(torch):
    """Bandwidth of large copies from pinned host memory to the device, measured here (GB/s)."""
    n = 256 << 20
    src = torch.empty(n, dtype=torch.uint8).pin_memory()
    dst = torch.empty(n, dtype=torch.uint8, device="cuda")
    for _ in range(2):
        dst.copy_(src, non_blocking=True)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(4):
        dst.copy_(src, non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    return 4 * n / (e0.elapsed_time(e1) * 1e-3) / 1e9


def print_records(recs):
    print("%-14s %9s %9s %9s %9s %9s" % ("kernel", "start", "ready", "stream", "end", "end-ready"))
    for r in recs:
        print("%-14s %9.2f %9.2f %9s %9.2f %9.2f" % (r["kind"], r["start"], r["ready"],
              "%.2f" % r["aux"] if r["aux"] is not None else "-", r["end"], r["end"] - r["ready"]))


def run_two_tier(dip, ctx, torch, w, L, rank, xs_host, keep_ratio, budget, steps, warmup, policy, sampler=None,
                 timeline=False):
    """Decode tokens through a stack whose weights live in pinned host memory; each layer keeps
    the columns its cache holds in an arena in device memory and fetches the misses of every
    mask over the host link."""
    from dip_inputs import device as dd
    d_model, d_ff = w.d_model, w.d_ff
    k_x, k_h = di.keep_count(keep_ratio, d_model), di.keep_count(keep_ratio, d_ff)
    ws, backs = [], []
    for l in range(L):
        g, gs = dd.matrix(w, l, "gate", d_ff, d_model, "cuda", rank)
        u, us = dd.matrix(w, l, "up", d_ff, d_model, "cuda", rank)
        d_, ds = dd.matrix(w, l, "down", d_model, d_ff, "cuda", rank)
        pw = dip.dip_pack_weights(ctx, w.wtype, d_model, d_ff, g, u, d_, gs, us, ds)
        torch.cuda.synchronize()
        backs.append((pw.gate_up.cpu().pin_memory(), pw.down.cpu().pin_memory()))
        # only the shapes and the INT4 scales stay on the device
        pw.gate_up = pw.down = None
        pw.struct.gate_up = None
        pw.struct.down = None
        ws.append(pw)
        del g, u, d_, gs, us, ds
    torch.cuda.empty_cache()

    def fresh():
        tg, td = [], []
        for l in range(L):
            cg = dip.CacheState(d_model, di.cache_capacity(budget, d_model), "cuda", policy)
            cd = dip.CacheState(d_ff, di.cache_capacity(budget, d_ff), "cuda", policy)
            tg.append(dip.Tier(cg, backs[l][0], backs[l][0].numel() // d_model, k_x, "cuda"))
            td.append(dip.Tier(cd, backs[l][1], backs[l][1].numel() // d_ff, k_h, "cuda"))
        return tg, td

    n_tok = xs_host.shape[0]
    xs_dev = xs_host.cuda()
    xa, xb = torch.empty(d_model, device="cuda"), torch.empty(d_model, device="cuda")
    y = torch.empty(d_model, device="cuda")
    out_host = torch.empty(d_model).pin_memory()
    stream = torch.cuda.current_stream()

    def token(tg, td):
        cur, nxt = xa, xb
        for l in range(L):
            dip.dip_mlp_step_tiered(ctx, ws[l], tg[l], td[l], cur, k_x, k_h, w.gamma, y)
            dip.dip_residual_rmsnorm(ctx, cur, y, nxt)
            cur, nxt = nxt, cur
        return cur

    tg, td = fresh()
    xa.copy_(xs_dev[0])
    token(tg, td)                                    # prime outside capture
    torch.cuda.synchronize()
    del tg, td
    tg, td = fresh()
    if timeline:
        ctx.trace_begin()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        x_last = token(tg, td)

    def fetched():
        return sum(int(t.counters[1]) for t in tg + td)

    for t in range(warmup):
        xa.copy_(xs_dev[t % n_tok], non_blocking=True)
        graph.replay()
    torch.cuda.synchronize()
    if timeline:
        ctx.trace_reset()
        xa.copy_(xs_dev[warmup % n_tok])
        graph.replay()
        recs = ctx.trace_read()
        ctx.trace_end()
        print("# %s two-tier, keep_ratio %g cache_budget %s: one graph replay of %d layers; times in us"
              % (w.name, keep_ratio, budget, L))
        print_records(recs)
        print("# per layer: %.2f us" % ((max(r["end"] for r in recs) - recs[0]["ready"]) / L))
        return None
    b0 = fetched()
    m0 = [torch.stack([t.cache.meta for t in ts]).sum(0).cpu().tolist() for ts in (tg, td)]
    if sampler:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for t in range(steps):
        xa.copy_(xs_dev[(warmup + t) % n_tok], non_blocking=True)
        graph.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    ms = e0.elapsed_time(e1)
    b1 = fetched()
    m1 = [torch.stack([t.cache.meta for t in ts]).sum(0).cpu().tolist() for ts in (tg, td)]
    hits = sum(a[2] - b[2] for a, b in zip(m1, m0))
    misses = sum(a[3] - b[3] for a, b in zip(m1, m0))
    # end to end: the token comes from the host and the result goes back, every step
    xs_pin = xs_host.pin_memory()
    n_e2e = min(steps, 64)
    torch.cuda.synchronize()
    e0.record(stream)
    for t in range(n_e2e):
        xa.copy_(xs_pin[(warmup + steps + t) % n_tok], non_blocking=True)
        graph.replay()
        out_host.copy_(x_last, non_blocking=True)
        stream.synchronize()
    e1.record(stream)
    torch.cuda.synchronize()
    ms_e = e0.elapsed_time(e1)
    # the fetch kernel by itself: a second capture with the device-side timeline on, a few replays
    ctx.trace_begin()
    graph_t = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph_t):
        token(tg, td)
    fetch_us, fetch_bytes = 0.0, 0
    for t in range(8):
        xa.copy_(xs_dev[(warmup + steps + n_e2e + t) % n_tok])
        torch.cuda.synchronize()
        c0 = fetched()
        ctx.trace_reset()
        graph_t.replay()
        recs = ctx.trace_read()
        fetch_us += sum(r["end"] - r["ready"] for r in recs if r["kind"] == "tier_fetch")
        fetch_bytes += fetched() - c0
    ctx.trace_end()
    status = ctx.device_status()
    if status != 0:
        raise SystemExit("device status %d after the two-tier run" % status)
    arena = sum(t.arena.numel() for t in tg + td)
    return {"ms_total": ms, "ms_per_step": ms / steps, "k_x": k_x, "k_h": k_h, "clocks": clocks,
            "fetched_bytes": b1 - b0, "fetch_gbs": (b1 - b0) / (ms * 1e-3) / 1e9,
            "fetch_kernel_gbs": fetch_bytes / max(fetch_us, 1e-9) / 1e3, "fetch_kernel_us": fetch_us / (8 * 2 * L),
            "fetch_kernel_bytes": fetch_bytes / (8 * 2 * L),
            "hit_rate": hits / max(1, hits + misses), "arena_bytes": arena,
            "backing_bytes": sum(a.numel() + b.numel() for a, b in backs),
            "e2e": {"value": L * n_e2e / (ms_e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 4 * d_model,
                    "d2h_bytes_per_step": 4 * d_model}}


def main_neuron_pruned(args, dip, ctx, torch, w, keep_ratio, rank, world, local):
    """Gate pruning / Up pruning (Eq. 5): per layer one dense neuron-major product ranks the
    neurons, the other first-layer matrix and W^d are read for the kept neurons only."""
    from dip_inputs import device as dd
    if world > 1 or args.batch > 1 or w.wtype == di.W_INT4_G128:
        raise SystemExit("--schedule gate|up is a single-GPU, single-token, F32/BF16 measurement")
    by = args.schedule
    L = args.layers if args.layers else w.n_layers
    d_model, d_ff = w.d_model, w.d_ff
    k = di.keep_count(keep_ratio, d_ff)
    layers = []
    for l in range(L):
        g, _ = dd.matrix(w, l, "gate", d_ff, d_model, "cuda", rank)
        u, _ = dd.matrix(w, l, "up", d_ff, d_model, "cuda", rank)
        d_, _ = dd.matrix(w, l, "down", d_model, d_ff, "cuda", rank)
        layers.append(dip.NeuronWeights(w.wtype, g, u, d_.t().contiguous()))
        del d_
    n_tok = min(w.n_tokens, args.steps + args.warmup)
    xs_dev = torch.from_numpy(di.token_inputs(w, n_tokens=n_tok, batch=1)[:, 0].copy()).cuda()
    xa, xb = torch.empty(d_model, device="cuda"), torch.empty(d_model, device="cuda")
    y = torch.empty(d_model, device="cuda")
    stream = torch.cuda.current_stream()

    def token():
        cur, nxt = xa, xb
        for l in range(L):
            dip.dip_mlp_step_neuron_pruned(ctx, layers[l], by, cur, k, y)
            dip.dip_residual_rmsnorm(ctx, cur, y, nxt)
            cur, nxt = nxt, cur
        return cur

    xa.copy_(xs_dev[0])
    token()
    torch.cuda.synchronize()
    ctx.trace_begin()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        x_last = token()
    # per-kernel durations from the device-side timeline of two replays
    dense_us = kept_us = 0.0
    for t in range(2):
        xa.copy_(xs_dev[t % n_tok])
        torch.cuda.synchronize()
        ctx.trace_reset()
        graph.replay()
        recs = [r for r in ctx.trace_read() if r["kind"] == "rowdot"]
        dense_us += sum(r["end"] - r["ready"] for r in recs[0::2])
        kept_us += sum(r["end"] - r["ready"] for r in recs[1::2])
    dense_us /= 2 * L
    kept_us /= 2 * L
    if args.timeline:
        print_records(ctx.trace_read()[:10])
        ctx.trace_end()
        return
    ctx.trace_end()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        x_last = token()
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ
                           else int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local]))
    for t in range(args.warmup):
        xa.copy_(xs_dev[t % n_tok], non_blocking=True)
        graph.replay()
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for t in range(args.steps):
        xa.copy_(xs_dev[(args.warmup + t) % n_tok], non_blocking=True)
        graph.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    xs_pin = xs_dev.cpu().pin_memory()
    out_host = torch.empty(d_model).pin_memory()
    n_e2e = min(args.steps, 128)
    e0.record(stream)
    for t in range(n_e2e):
        xa.copy_(xs_pin[t % n_tok], non_blocking=True)
        graph.replay()
        out_host.copy_(x_last, non_blocking=True)
        stream.synchronize()
    e1.record(stream)
    torch.cuda.synchronize()
    ms_e = e0.elapsed_time(e1)
    bw = weight_bytes(w.wtype)
    dense_bytes = d_ff * d_model * bw + 4 * (d_model + d_ff)
    step_bytes = dense_bytes + 2 * k * d_model * bw + 4 * (3 * d_ff + 2 * d_model + k)
    peak, peak_kind = measured_peak()
    step_gbs = step_bytes * L * args.steps / (ms * 1e-3) / 1e9
    achieved = dense_bytes / (dense_us * 1e-6) / 1e9
    line = {
        "metric": METRIC, "value": L * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None,
        "dtype": {di.W_F32: "f32", di.W_BF16: "bf16 weights, f32 accumulate"}[w.wtype], "data": "synthetic",
        "config": {"workload": "%s, %s pruning (Eq. 5)" % (w.name, by), "n_layers": L, "d_model": d_model,
                   "d_ff": d_ff, "keep_ratio": keep_ratio, "k": k,
                   "step": "one decode token through %d layers = %d MLP-steps" % (L, L),
                   "l2": "inputs larger than L2: %.1f GB of distinct layer weights cycled"
                         % (3 * L * d_ff * d_model * bw / 1e9),
                   "launch": "CUDA graph of dip_mlp_step_neuron_pruned + dip_residual_rmsnorm per layer",
                   "parallelism": "replicas only"},
        "mlp_step_us": ms * 1e3 / (L * args.steps), "step_gbs": step_gbs, "step_frac_of_measured_hbm": step_gbs / peak,
        "clocks": clocks,
        "e2e": {"value": L * n_e2e / (ms_e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 4 * d_model,
                "d2h_bytes_per_step": 4 * d_model},
        # per layer: 2 row products, select, mask->list, memset, down GEMV, rmsnorm
        "gpu_launches": 6 * L * args.steps,
        "roofline": {"bound": "hbm", "kernel": "rowdot_kernel (dense ranking product)", "achieved": achieved,
                     "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "bytes_per_launch": dense_bytes, "us_per_launch": dense_us, "traffic": None},
        "kernels_us": {"rowdot_dense": dense_us, "rowdot_kept": kept_us},
    }
    print(json.dumps(line))


def main_two_tier(args, dip, ctx, torch, w, keep_ratio, budget, rank, world, local):
    if world > 1 or args.batch > 1 or budget is None:
        raise SystemExit("--two-tier is a single-GPU, single-token, cache-aware measurement")
    L = args.layers if args.layers else 4
    n_tok = min(w.n_tokens, args.steps + args.warmup + 64)
    xs_host = torch.from_numpy(di.token_inputs(w, n_tokens=n_tok, batch=1,
                                               correlation=args.token_correlation)[:, 0].copy())
    link = host_link_peak(torch)
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ
                           else int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local]))
    if args.timeline:
        run_two_tier(dip, ctx, torch, w, L, rank, xs_host, keep_ratio, budget, args.steps, args.warmup, args.policy,
                     timeline=True)
        return
    r = run_two_tier(dip, ctx, torch, w, L, rank, xs_host, keep_ratio, budget, args.steps, args.warmup, args.policy,
                     sampler=sampler)
    line = {
        "metric": METRIC, "value": L * args.steps / (r["ms_total"] * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": {di.W_F32: "f32", di.W_BF16: "bf16 weights, f32 accumulate",
                  di.W_INT4_G128: "int4 weights, f32 accumulate"}[w.wtype],
        "data": "synthetic",
        "config": {"workload": w.name + " two-tier: cache arena in HBM, all weights in pinned host memory",
                   "n_layers": L, "d_model": w.d_model, "d_ff": w.d_ff, "keep_ratio": keep_ratio, "k_x": r["k_x"],
                   "k_h": r["k_h"], "cache_budget": budget, "gamma": w.gamma, "cache_policy": args.policy,
                   "token_correlation": args.token_correlation,
                   "step": "one decode token through %d layers = %d MLP-steps" % (L, L),
                   "l2": "inputs larger than L2: %.1f GB of arenas, %.1f GB of host weights"
                         % (r["arena_bytes"] / 1e9, r["backing_bytes"] / 1e9),
                   "launch": "CUDA graph of dip_mlp_step_tiered + dip_residual_rmsnorm per layer",
                   "parallelism": "replicas only"},
        "mlp_step_us": r["ms_per_step"] * 1e3 / L, "hit_rate": r["hit_rate"], "clocks": r["clocks"],
        "e2e": r["e2e"],
        # per layer: 2 selects, 2 cache updates, 2 slot assignments, 2 fetches, 4 GEMVs, 2 combines, 1 rmsnorm
        "gpu_launches": 15 * L * args.steps,
        # the fetch kernel: bytes it brought in / its own device time (timeline of 8 replays); the
        # same bytes over the whole step's time are in fetch_gbs_over_step
        "roofline": {"bound": "host_link", "kernel": "tier_fetch_kernel", "achieved": r["fetch_kernel_gbs"],
                     "peak": link, "peak_kind": "of a pinned host-to-device copy measured in this run",
                     "unit": "GB/s", "frac": r["fetch_kernel_gbs"] / link,
                     "bytes_per_launch": r["fetch_kernel_bytes"], "us_per_launch": r["fetch_kernel_us"],
                     "traffic": None},
        "fetch_gbs_over_step": r["fetch_gbs"],
        "fetched_bytes_per_mlp_step": r["fetched_bytes"] / (L * args.steps),
    }
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = {k: v for k, v in oracle_rate(w, keep_ratio, budget, 1, 60).items()
                                if k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line))


def print_timeline(dip, ctx, torch, w, layers, xs_host, keep_ratio, budget):
    """One decode token through the stack as a CUDA graph, with the library's device-side
    timeline on: per kernel, when it started, when its inputs were ready, when it ended."""
    L, d_model, d_ff = len(layers), w.d_model, w.d_ff
    k_x, k_h = di.keep_count(keep_ratio, d_model), di.keep_count(keep_ratio, d_ff)
    ca = budget is not None
    gamma = w.gamma if ca else 1.0
    if ca:
        stack = dip.Stack(layers, [dip.CacheState(d_model, di.cache_capacity(budget, d_model), "cuda") for _ in range(L)],
                          [dip.CacheState(d_ff, di.cache_capacity(budget, d_ff), "cuda") for _ in range(L)])
    else:
        stack = dip.Stack(layers)
    xs = xs_host.cuda()
    x_cur = torch.empty(tuple(xs.shape[1:]), device="cuda")
    x_out = torch.empty_like(x_cur)
    x_cur.copy_(xs[0])
    dip.dip_stack_step(ctx, stack, x_cur, k_x, k_h, gamma, x_out)
    torch.cuda.synchronize()
    ctx.trace_begin()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        dip.dip_stack_step(ctx, stack, x_cur, k_x, k_h, gamma, x_out)
    for t in range(6):
        x_cur.copy_(xs[t % xs.shape[0]])
        g.replay()
    torch.cuda.synchronize()
    ctx.trace_reset()
    x_cur.copy_(xs[6 % xs.shape[0]])
    g.replay()
    recs = ctx.trace_read()
    ctx.trace_end()
    print("# %s keep_ratio %g cache_budget %s: one graph replay of %d layers; times in us" % (w.name, keep_ratio, budget, L))
    print_records(recs)
    main_path = [r for r in recs if r["kind"] != "cache_update"]
    print("# critical path per layer: %.2f us" % ((main_path[-1]["end"] - main_path[0]["ready"]) / L))


def write_report(dip, ctx, torch, path, steps):
    """All five configurations (bench workloads), one row each: MLP-steps/s, effective GB/s on the
    kept-column bytes, fraction of the measured and nominal HBM peak."""
    peak, kind = measured_peak()
    rows = []

    def row(name, r, L, extra=""):
        gbs = r.get("union_gbs", r["step_gbs"])
        rows.append("| %s | %g | %s | %d | %.0f | %.1f | %.0f | %.1f %% | %.1f %% | %s |" % (
            name, r["keep_ratio"], r["cache_budget"], r["batch"], r["mlp_steps_per_s"], r["ms_per_step"] * 1e3 / L,
            gbs, 100 * gbs / NOMINAL_HBM_GBS, 100 * gbs / peak, extra))

    for name in ("block_f32", "phi3_mini", "phi3_medium", "llama3_8b_int4", "phi3_medium_batched"):
        w = di.WORKLOADS[name]
        L = 8 if name == "block_f32" else w.n_layers      # 8 distinct blocks cycled: HBM-cold
        layers = build_stack(dip, ctx, torch, w, L, 0)
        n_tok = min(w.n_tokens, steps + 8)
        if name == "phi3_medium_batched":
            for B in di.BATCH_SIZES:
                xs = torch.from_numpy(di.token_inputs(w, n_tokens=n_tok, batch=B).copy())
                xs = xs[:, 0] if B == 1 else xs
                r = run_config(dip, ctx, torch, w, layers, xs, w.keep_ratio, None, min(steps, 64), 4,
                               kernel_pass=False, e2e_pass=False, min_timed_s=0.1)
                ud = r.get("union_density")
                row(name, r, L, "union density x %.2f h %.2f" % (ud["x"], ud["h"]) if ud else "")
        else:
            xs = torch.from_numpy(di.token_inputs(w, n_tokens=n_tok, batch=1)[:, 0].copy())
            combos = [(w.keep_ratio, w.cache_budget)]
            if name == "phi3_medium":
                combos = [(r_, b_) for r_ in di.PHI3_MEDIUM_KEEP_RATIOS for b_ in di.PHI3_MEDIUM_CACHE_BUDGETS]
            for rho, beta in combos:
                r = run_config(dip, ctx, torch, w, layers, xs, rho, beta, steps, 4, kernel_pass=False, e2e_pass=False,
                               min_timed_s=0.1)
                extra = "hit rate %.2f" % r["hit_rate"] if "hit_rate" in r else ""
                if name == "block_f32":
                    extra = "8 distinct blocks cycled (one block alone fits L2)"
                row(name, r, L, extra)
        del layers
        torch.cuda.empty_cache()
    with open(path, "w") as f:
        f.write("| workload | keep ratio | cache budget | batch | MLP-steps/s | us per MLP-step | GB/s (kept-column bytes) | of 8 TB/s | of %s %.0f GB/s | notes |\n" % (kind, peak))
        f.write("|---|---|---|---|---|---|---|---|---|---|\n")
        f.write("\n".join(rows) + "\n")


def oracle_rate(w, keep_ratio, budget, n_layers_sample, n_steps, warmup=0, threads=None):
    """The CPU oracle as it stands, timed on this machine's host cores on a bounded sample of the
    workload: `n_steps` MLP-steps cycling over `n_layers_sample` host-generated layers.
    threads: None = all cores the OpenMP runtime gives it; 1 = the single-thread leg."""
    import oracle
    all_threads = oracle.num_threads()
    if threads is not None:
        oracle.set_num_threads(threads)
    k_x, k_h = di.keep_count(keep_ratio, w.d_model), di.keep_count(keep_ratio, w.d_ff)
    ca = budget is not None
    gamma = w.gamma if ca else 1.0
    lws = [di.layer_weights(w, l) for l in range(n_layers_sample)]
    mats = [(oracle.Matrix(lw.wtype, lw.gate, lw.gate_scales, w.d_ff, w.d_model),
             oracle.Matrix(lw.wtype, lw.up, lw.up_scales, w.d_ff, w.d_model),
             oracle.Matrix(lw.wtype, lw.down, lw.down_scales, w.d_model, w.d_ff)) for lw in lws]
    cg = [oracle.Cache(w.d_model, di.cache_capacity(budget, w.d_model)) if ca else None for _ in lws]
    cd = [oracle.Cache(w.d_ff, di.cache_capacity(budget, w.d_ff)) if ca else None for _ in lws]
    n_tok = (warmup + n_steps + n_layers_sample - 1) // n_layers_sample + 1
    xs = di.token_inputs(w, n_tokens=n_tok, batch=1)[:, 0]
    cur, t_idx, times = xs[0], 0, []
    for s in range(warmup + n_steps):
        l = s % n_layers_sample
        if l == 0:
            t_idx += 1
            cur = xs[t_idx % n_tok]
        t0 = time.perf_counter()
        r = oracle.mlp_step(*mats[l], cur, k_x, k_h, gamma, cg[l], cd[l])
        cur = oracle.residual_rmsnorm(cur, r.y)
        if s >= warmup:
            times.append(time.perf_counter() - t0)
    total = float(np.sum(times))
    used = oracle.num_threads()
    if threads is not None:
        oracle.set_num_threads(all_threads)
    return {"value": n_steps / total, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": "%d MLP-steps over %d host-generated layer(s) of %s, keep ratio %g, cache budget %s"
                      % (n_steps, n_layers_sample, w.name, keep_ratio, budget),
            "ms_per_mlp_step": total / n_steps * 1e3}


def main_reference(args, w, keep_ratio, budget):
    """The reference arm: the CPU oracle timed on the host cores; a step is one MLP-step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    r = oracle_rate(w, keep_ratio, budget, 1, args.steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["ms_per_mlp_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": w.name, "keep_ratio": keep_ratio, "cache_budget": budget,
                       "d_model": w.d_model, "d_ff": w.d_ff, "step": "one MLP-step (1 layer x 1 token) of the CPU oracle"},
            "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    args = parse_args()
    w = di.WORKLOADS[args.workload]
    keep_ratio = args.keep_ratio if args.keep_ratio is not None else w.keep_ratio
    budget = args.cache_budget if args.cache_budget is not None else w.cache_budget
    if args.impl == "reference":
        return main_reference(args, w, keep_ratio, budget)

    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_mod

    import paper_2412_01380_b200 as dip
    ctx = dip.Context(local)
    if args.report:
        write_report(dip, ctx, torch, args.report, min(args.steps, 128))
        return
    if args.schedule != "dip":
        return main_neuron_pruned(args, dip, ctx, torch, w, keep_ratio, rank, world, local)
    if args.two_tier:
        return main_two_tier(args, dip, ctx, torch, w, keep_ratio, budget, rank, world, local)
    L = args.layers if args.layers else w.n_layers
    layers = build_stack(dip, ctx, torch, w, L, rank)
    n_tok = w.n_tokens                                  # the repeats cycle through the workload's tokens
    wl_rank = w.scaled(seed=w.seed + 1000 * rank)
    if args.batch > 1:
        budget = None                                   # Algorithm 1 is per token
        xs_host = torch.from_numpy(di.token_inputs(wl_rank, n_tokens=n_tok, batch=args.batch).copy())
    else:
        xs_host = torch.from_numpy(di.token_inputs(wl_rank, n_tokens=n_tok, batch=1)[:, 0].copy())

    if args.timeline:
        print_timeline(dip, ctx, torch, w, layers, xs_host, keep_ratio, budget)
        return
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ
                           else int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local])) if rank == 0 else None
    head = run_config(dip, ctx, torch, w, layers, xs_host, keep_ratio, budget, args.steps, args.warmup,
                      sampler=sampler, dist=dist, policy=args.policy, min_timed_s=args.min_timed_s,
                      min_repeats=3 if args.min_timed_s > 0 else 1)

    sweep = []
    if not args.no_sweep and world == 1 and w.name == "phi3_medium":
        for rho in di.PHI3_MEDIUM_KEEP_RATIOS:
            for beta in di.PHI3_MEDIUM_CACHE_BUDGETS:
                r = run_config(dip, ctx, torch, w, layers, xs_host, rho, beta, min(args.steps, 64), 4,
                               kernel_pass=True, e2e_pass=False, min_timed_s=0.1)
                sweep.append(r)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    gu_bytes = head["bytes"]["gate_up"]
    if "kernels" in head:
        gu_us = head["kernels"]["gate_up_train_us"]
        achieved = gu_bytes / (gu_us * 1e-6) / 1e9
    else:
        # batched decode: no per-kernel pass; the whole step on the bytes of the union of the masks
        gu_us = None
        achieved = head.get("union_gbs", head["step_gbs"])
    fused = bool(head.get("select_in_product"))
    # per layer: two selects and two products (or two launches that do both), two cache updates when a
    # cache is on; one residual + rmsnorm closes the stack
    # (with a cache the last layer's down half keeps its select kernel: one launch more per token)
    launches_per_step = L * ((2 if fused else 4) + (2 if budget is not None else 0)) + 1 + (1 if fused and budget is not None else 0)
    kernel_name = GATE_UP_KERNEL(w, args.batch, fused) + (" (select of x + gate/up bundle)" if fused else " (gate/up bundle)")
    line = {
        "metric": METRIC, "value": whole_job_rate(L * args.steps, world, head["ms_total"]), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": head["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {di.W_F32: "f32", di.W_BF16: "bf16 weights, f32 accumulate", di.W_INT4_G128: "int4 weights, f32 accumulate"}[w.wtype],
        "data": "synthetic",
        "config": {"workload": w.name, "n_layers": L, "d_model": w.d_model, "d_ff": w.d_ff,
                   "keep_ratio": keep_ratio, "k_x": head["k_x"], "k_h": head["k_h"], "cache_budget": budget,
                   "gamma": w.gamma if budget is not None else 1.0, "cache_policy": args.policy, "batch": args.batch,
                   "step": "one decode token through %d layers = %d MLP-steps" % (L, L),
                   "l2": "inputs larger than L2: %.1f GB of distinct layer weights cycled" % (sum(l.nbytes for l in layers) / 1e9),
                   "launch": "CUDA graph of dip_stack_step", "parallelism": "replicas only"},
        "mlp_step_us": head["ms_per_step"] * 1e3 / L,
        "repeats": head["repeats"],
        "step_gbs": head["step_gbs"] * world,
        "step_frac_of_measured_hbm": head["step_gbs"] / peak,
        "step_frac_of_nominal_8tbs": head["step_gbs"] / NOMINAL_HBM_GBS,
        "hit_rate": head.get("hit_rate"),
        "paper_simulator_view": head.get("paper_simulator_view"),
        "clocks": head["clocks"],
        "e2e": {k: head["e2e"][k] for k in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step")},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                     "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8tbs": achieved / NOMINAL_HBM_GBS, "bytes_per_launch": gu_bytes,
                     "us_per_launch": gu_us, "traffic": ncu_traffic(w, keep_ratio, args.batch, kernel_name),
                     "traffic_source": "committed ncu capture (%s); null when this run's kernel or workload differs"
                                       % NCU_TRAFFIC["source"]},
        "kernels_us": head.get("kernels"),
        "union_density": head.get("union_density"),
    }
    line["e2e"]["value"] *= world
    if sweep:
        line["sweep"] = [{"keep_ratio": r["keep_ratio"], "cache_budget": r["cache_budget"],
                          "mlp_steps_per_s": r["mlp_steps_per_s"], "mlp_step_us": r["ms_per_step"] * 1e3 / L,
                          "step_gbs": r["step_gbs"], "frac_of_measured": r["step_gbs"] / peak,
                          "frac_of_nominal_8tbs": r["step_gbs"] / NOMINAL_HBM_GBS, "hit_rate": r.get("hit_rate"),
                          "gate_up_gbs": r["bytes"]["gate_up"] / (r["kernels"]["gate_up_train_us"] * 1e-6) / 1e9,
                          "down_gbs": r["bytes"]["down"] / (r["kernels"]["down_train_us"] * 1e-6) / 1e9,
                          "kernels_us": r["kernels"]} for r in sweep]
    if world == 1 and not args.no_cpu_baseline:
        del layers
        torch.cuda.empty_cache()
        line["cpu_baseline"] = {k: v for k, v in oracle_rate(w, keep_ratio, budget, 1, 60).items()
                                if k in ("value", "unit", "cores", "kind", "sample")}
        one = oracle_rate(w, keep_ratio, budget, 1, 8, threads=1)
        line["cpu_baseline"]["single_thread"] = {k: one[k] for k in ("value", "unit", "cores", "sample")}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
