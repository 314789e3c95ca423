// C ABI of the library (see include/dip.h): context, argument validation, and the
// composition of the kernels into the sparse MLP step of Eq. 3 / 7 / 8.
#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace {

constexpr size_t PARTIALS_FLOATS = (size_t)8 << 20;   // 32 MB of split-row partial sums
constexpr int N_TICKETS = 4096;

bool dims_ok(int wtype, int d_model, int d_ff)
{
    if (wtype != DIP_W_F32 && wtype != DIP_W_BF16 && wtype != DIP_W_INT4_G128) return false;
    if (d_model < 32 || d_ff < 32 || d_model > DIP_MAX_D || d_ff > DIP_MAX_D) return false;
    if (d_model % 32 || d_ff % 32) return false;
    if (wtype == DIP_W_INT4_G128 && (d_model % DIP_INT4_GROUP || d_ff % DIP_INT4_GROUP)) return false;
    return true;
}

bool weights_ok(const dip_mlp_weights *w)
{
    if (!w || !dims_ok(w->wtype, w->d_model, w->d_ff)) return false;
    if (!w->gate_up || !w->down || !dip_aligned16(w->gate_up) || !dip_aligned16(w->down)) return false;
    if (w->wtype == DIP_W_INT4_G128 &&
        (!w->gate_up_scales || !w->down_scales || !dip_aligned16(w->gate_up_scales) ||
         !dip_aligned16(w->down_scales)))
        return false;
    return true;
}

bool cache_ok(const dip_cache_state *c, int d)
{
    if (!(c && c->d == d && c->capacity >= 0 && c->capacity <= d && c->stamp && c->meta &&
          dip_aligned16(c->stamp) && dip_aligned16(c->meta)))
        return false;
    if (c->policy == DIP_CACHE_LFU) return c->count && dip_aligned16(c->count);
    return c->policy == DIP_CACHE_LRU;
}

size_t packed_row_bytes(int wtype, size_t row_elems)
{
    return wtype == DIP_W_F32 ? row_elems * 4 : wtype == DIP_W_BF16 ? row_elems * 2 : row_elems / 2;
}

bool tier_ok(const dip_tier *t, const dip_cache_state *c, size_t row_bytes, int k)
{
    if (!t || !c || t->d != c->d || t->capacity != c->capacity) return false;
    if (t->staging < k || t->row_bytes != row_bytes || (row_bytes & 15)) return false;
    if (!t->backing || !t->arena || !t->slot || !t->loc || !t->fetch || !t->split || !t->counters) return false;
    return dip_aligned16(t->backing) && dip_aligned16(t->arena) && dip_aligned16(t->split);
}

template <typename T> dip_status dev_alloc(dip_ctx *ctx, T **p, size_t n)
{
    DIP_CUDA_TRY(ctx, cudaMalloc((void **)p, n * sizeof(T)));
    return DIP_OK;
}

// The context exists and its device is the calling thread's current one.
bool ctx_ok(const dip_ctx *ctx)
{
    int dev = -1;
    return ctx && cudaGetDevice(&dev) == cudaSuccess && dev == ctx->device;
}

// Shapes within what the context's workspace was sized for.
bool fits(const dip_ctx *ctx, int d_a, int d_b, int batch)
{
    return d_a <= ctx->max_d && d_b <= ctx->max_d && batch <= ctx->max_batch;
}

bool opt_aligned16(const void *p) { return !p || dip_aligned16(p); }

bool outputs_aligned(const dip_step_outputs *o)
{
    return !o || (opt_aligned16(o->mask_x) && opt_aligned16(o->mask_h) && opt_aligned16(o->h));
}

}  // namespace

extern "C" {

const char *dip_status_string(dip_status s)
{
    switch (s) {
    case DIP_OK: return "ok";
    case DIP_ERR_INVALID_ARG: return "invalid argument";
    case DIP_ERR_UNSUPPORTED: return "unsupported request";
    case DIP_ERR_CUDA: return "CUDA runtime failure";
    case DIP_ERR_WORKSPACE: return "problem exceeds the context workspace";
    }
    return "unknown status";
}

const char *dip_last_error(const dip_ctx *ctx) { return ctx ? ctx->err : ""; }
int dip_sm_count(const dip_ctx *ctx) { return ctx ? ctx->sm_count : 0; }

dip_status dip_create(dip_ctx **out, int device) { return dip_create_ex(out, device, nullptr); }

dip_status dip_create_ex(dip_ctx **out, int device, const dip_options *opt)
{
    if (!out) return DIP_ERR_INVALID_ARG;
    *out = nullptr;
    dip_options o = {};
    if (opt) o = *opt;
    if (o.max_d < 0 || o.max_d > DIP_MAX_D || o.max_batch < 0 || o.max_batch > DIP_MAX_BATCH) return DIP_ERR_INVALID_ARG;
    if (o.gemv_segment_bytes != 0 && o.gemv_segment_bytes != 512 && o.gemv_segment_bytes != 1024 &&
        o.gemv_segment_bytes != 2048)
        return DIP_ERR_INVALID_ARG;
    if (o.wait_limit_us < 0) return DIP_ERR_INVALID_ARG;
    int prev_device = -1;
    if (cudaGetDevice(&prev_device) != cudaSuccess) return DIP_ERR_CUDA;
    dip_ctx *ctx = new (std::nothrow) dip_ctx();
    if (!ctx) return DIP_ERR_CUDA;
    memset(ctx, 0, sizeof(*ctx));
    ctx->device = device;
    dip_status st = DIP_OK;
    auto fail = [&](dip_status s) {
        dip_destroy(ctx);
        cudaSetDevice(prev_device);
        return s;
    };
    if (cudaSetDevice(device) != cudaSuccess) return fail(DIP_ERR_CUDA);
    if (cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
        return fail(DIP_ERR_CUDA);
    ctx->max_d = o.max_d ? (o.max_d + 127) / 128 * 128 : DIP_MAX_D;
    ctx->max_batch = o.max_batch ? o.max_batch : DIP_MAX_BATCH;
    ctx->gemv_seg = o.gemv_segment_bytes;
    ctx->gemv_direct = o.gemv_copy_ring ? 0 : 1;
    // below ~4096 columns the whole of h and its stamps is a few KB and the plain select is as fast
    ctx->coarse_min_d = o.coarse_min_d == 0 ? 4096 : (o.coarse_min_d < 0 ? 0 : o.coarse_min_d);
    ctx->fuse_select = o.select_in_product < 0 ? 0 : 1;
    ctx->wait_limit_ns = o.wait_limit_us ? 1000ull * (unsigned long long)o.wait_limit_us : 1000000000ull;
    // split-row partial sums: up to one part per SM of a whole output row per token
    ctx->partials_floats = PARTIALS_FLOATS;
    ctx->n_tickets = N_TICKETS;
    const size_t vec = (size_t)ctx->max_batch * ctx->max_d;
    if ((st = dev_alloc(ctx, &ctx->partials, ctx->partials_floats)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->tickets, (size_t)N_TICKETS)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->h, vec)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->y, vec)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->y2, vec)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->xa, vec)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->xb, vec)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->p, (size_t)ctx->max_d)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->mask, vec / 32)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->idx, vec)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->mask_h, vec / 32)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->idx_h, vec)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->union_idx, (size_t)ctx->max_d)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->counts, (size_t)8)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->mask_ring, (size_t)2 * DIP_RING_LAYERS * (ctx->max_d / 32))) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->mask_tmp, (size_t)(ctx->max_d / 32))) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->coarse, vec)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->xt, (size_t)ctx->max_d * 32)) != DIP_OK) return fail(st);
    if ((st = dev_alloc(ctx, &ctx->status, (size_t)1)) != DIP_OK) return fail(st);
    if (cudaMemset(ctx->status, 0, sizeof(int)) != cudaSuccess) return fail(DIP_ERR_CUDA);
    if ((st = dev_alloc(ctx, &ctx->trace, (size_t)DIP_TRACE_SLOTS * DIP_TRACE_WORDS)) != DIP_OK) return fail(st);
    for (int i = 0; i < 2; ++i) {
        if (cudaStreamCreateWithFlags(&ctx->tier_fetch[i], cudaStreamNonBlocking) != cudaSuccess) return fail(DIP_ERR_CUDA);
        if (cudaStreamCreateWithFlags(&ctx->tier_book[i], cudaStreamNonBlocking) != cudaSuccess) return fail(DIP_ERR_CUDA);
        if (cudaEventCreateWithFlags(&ctx->ev_tier_fork[i], cudaEventDisableTiming) != cudaSuccess) return fail(DIP_ERR_CUDA);
        if (cudaEventCreateWithFlags(&ctx->ev_tier_fetched[i], cudaEventDisableTiming) != cudaSuccess) return fail(DIP_ERR_CUDA);
        if (cudaEventCreateWithFlags(&ctx->ev_tier_booked[i], cudaEventDisableTiming) != cudaSuccess) return fail(DIP_ERR_CUDA);
    }
    for (int i = 0; i < 2; ++i) {
        if (cudaStreamCreateWithFlags(&ctx->side[i], cudaStreamNonBlocking) != cudaSuccess) return fail(DIP_ERR_CUDA);
        if (cudaEventCreateWithFlags(&ctx->ev_fork[i], cudaEventDisableTiming) != cudaSuccess) return fail(DIP_ERR_CUDA);
        if (cudaEventCreateWithFlags(&ctx->ev_join[i], cudaEventDisableTiming) != cudaSuccess) return fail(DIP_ERR_CUDA);
    }
    if (cudaMemset(ctx->tickets, 0, N_TICKETS * sizeof(unsigned int)) != cudaSuccess) return fail(DIP_ERR_CUDA);
    if (cudaMemset(ctx->counts, 0, 8 * sizeof(int32_t)) != cudaSuccess) return fail(DIP_ERR_CUDA);
    if ((st = dip_init_mask_kernels(ctx)) != DIP_OK) return fail(st);
    if (cudaSetDevice(prev_device) != cudaSuccess) return fail(DIP_ERR_CUDA);
    *out = ctx;
    return DIP_OK;
}

dip_status dip_destroy(dip_ctx *ctx)
{
    if (!ctx) return DIP_ERR_INVALID_ARG;
    cudaFree(ctx->partials);
    cudaFree(ctx->tickets);
    cudaFree(ctx->h);
    cudaFree(ctx->y);
    cudaFree(ctx->y2);
    cudaFree(ctx->xa);
    cudaFree(ctx->xb);
    cudaFree(ctx->p);
    cudaFree(ctx->mask);
    cudaFree(ctx->idx);
    cudaFree(ctx->mask_h);
    cudaFree(ctx->idx_h);
    cudaFree(ctx->union_idx);
    cudaFree(ctx->counts);
    cudaFree(ctx->mask_ring);
    cudaFree(ctx->mask_tmp);
    cudaFree(ctx->coarse);
    cudaFree(ctx->xt);
    cudaFree(ctx->status);
    cudaFree(ctx->trace);
    for (int i = 0; i < 2; ++i) {
        if (ctx->side[i]) cudaStreamDestroy(ctx->side[i]);
        if (ctx->ev_fork[i]) cudaEventDestroy(ctx->ev_fork[i]);
        if (ctx->ev_join[i]) cudaEventDestroy(ctx->ev_join[i]);
        if (ctx->tier_fetch[i]) cudaStreamDestroy(ctx->tier_fetch[i]);
        if (ctx->tier_book[i]) cudaStreamDestroy(ctx->tier_book[i]);
        if (ctx->ev_tier_fork[i]) cudaEventDestroy(ctx->ev_tier_fork[i]);
        if (ctx->ev_tier_fetched[i]) cudaEventDestroy(ctx->ev_tier_fetched[i]);
        if (ctx->ev_tier_booked[i]) cudaEventDestroy(ctx->ev_tier_booked[i]);
    }
    delete ctx;
    return DIP_OK;
}

size_t dip_packed_bytes(int wtype, int d_model, int d_ff, int which)
{
    if (!dims_ok(wtype, d_model, d_ff) || which < 0 || which > 3) return 0;
    const size_t n_gu = (size_t)d_model * 2 * (size_t)d_ff, n_d = (size_t)d_ff * (size_t)d_model;
    if (which == 0) return wtype == DIP_W_F32 ? n_gu * 4 : wtype == DIP_W_BF16 ? n_gu * 2 : n_gu / 2;
    if (which == 1) return wtype == DIP_W_F32 ? n_d * 4 : wtype == DIP_W_BF16 ? n_d * 2 : n_d / 2;
    if (wtype != DIP_W_INT4_G128) return 0;
    if (which == 2) return (size_t)(d_model / DIP_INT4_GROUP) * 2 * (size_t)d_ff * 2;
    return (size_t)(d_ff / DIP_INT4_GROUP) * (size_t)d_model * 2;
}

dip_status dip_pack_weights(dip_ctx *ctx, int wtype, int d_model, int d_ff,
                            const void *Wg, const void *Wu, const void *Wd,
                            const void *Sg, const void *Su, const void *Sd,
                            const dip_mlp_weights *out, void *stream)
{
    if (!ctx_ok(ctx) || !Wg || !Wu || !Wd || !out) return DIP_ERR_INVALID_ARG;
    if (!dip_aligned16(Wg) || !dip_aligned16(Wu) || !dip_aligned16(Wd) || !opt_aligned16(Sg) || !opt_aligned16(Su) ||
        !opt_aligned16(Sd))
        return DIP_ERR_INVALID_ARG;
    if (!weights_ok(out) || out->wtype != wtype || out->d_model != d_model || out->d_ff != d_ff)
        return DIP_ERR_INVALID_ARG;
    if (wtype == DIP_W_INT4_G128 && (!Sg || !Su || !Sd)) return DIP_ERR_INVALID_ARG;
    return dip_launch_pack(ctx, wtype, d_model, d_ff, Wg, Wu, Wd, Sg, Su, Sd, out, (cudaStream_t)stream);
}

dip_status dip_device_status(dip_ctx *ctx, int *status_out, void *stream)
{
    if (!ctx_ok(ctx) || !status_out) return DIP_ERR_INVALID_ARG;
    DIP_CUDA_TRY(ctx, cudaMemcpyAsync(status_out, ctx->status, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    DIP_CUDA_TRY(ctx, cudaStreamSynchronize((cudaStream_t)stream));
    return DIP_OK;
}

dip_status dip_reset_device_status(dip_ctx *ctx, void *stream)
{
    if (!ctx_ok(ctx)) return DIP_ERR_INVALID_ARG;
    DIP_CUDA_TRY(ctx, cudaMemsetAsync(ctx->status, 0, sizeof(int), (cudaStream_t)stream));
    return DIP_OK;
}

dip_status dip_selftest_bounded_wait(dip_ctx *ctx, int limit_us, unsigned long long *waited_ns, void *stream)
{
    if (!ctx_ok(ctx) || limit_us < 1 || limit_us > 1000000) return DIP_ERR_INVALID_ARG;
    return dip_launch_bounded_wait_selftest(ctx, 1000ull * (unsigned long long)limit_us, waited_ns, (cudaStream_t)stream);
}

// Run the cache update of one masked input beside the main stream (side stream `which`).
static dip_status fork_cache_update(dip_ctx *ctx, int which, const uint32_t *mask_bits, const dip_cache_state *c,
                                    cudaStream_t main)
{
    DIP_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_fork[which], main));
    DIP_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->side[which], ctx->ev_fork[which], 0));
    dip_status st = dip_launch_cache_update(ctx, mask_bits, c->d, c->stamp, c->policy == DIP_CACHE_LFU ? c->count : nullptr, c->meta,
                                            c->capacity, ctx->side[which]);
    ctx->side_busy[which] = true;
    return st;
}

// Make the main stream wait for the side streams' updates.
static dip_status join_cache_updates(dip_ctx *ctx, cudaStream_t main)
{
    for (int i = 0; i < 2; ++i) {
        if (!ctx->side_busy[i]) continue;
        DIP_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_join[i], ctx->side[i]));
        DIP_CUDA_TRY(ctx, cudaStreamWaitEvent(main, ctx->ev_join[i], 0));
        ctx->side_busy[i] = false;
    }
    return DIP_OK;
}

dip_status dip_mask_topk(dip_ctx *ctx, const float *x, int batch, int d, int k,
                         uint32_t *mask_bits, int32_t *kept_idx, void *stream)
{
    if (!ctx_ok(ctx) || !x || !dip_aligned16(x) || !opt_aligned16(mask_bits)) return DIP_ERR_INVALID_ARG;
    if (batch < 1 || batch > DIP_MAX_BATCH || d < 1 || d > DIP_MAX_D || k < 1 || k > d) return DIP_ERR_INVALID_ARG;
    if (!fits(ctx, d, 0, batch)) return DIP_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    uint32_t *m = mask_bits ? mask_bits : ctx->mask;
    dip_status st = dip_launch_select(ctx, x, nullptr, nullptr, batch, d, k, 1.0f, nullptr, m, s);
    if (st == DIP_OK && kept_idx) st = dip_launch_mask_to_idx(ctx, m, batch, 1, d, kept_idx, k, nullptr, s);
    return st;
}

dip_status dip_ca_mask(dip_ctx *ctx, const float *x, int d, int k, float gamma,
                       const dip_cache_state *st,
                       uint32_t *mask_bits, int32_t *kept_idx, void *stream)
{
    if (!ctx_ok(ctx) || !x || !dip_aligned16(x) || !opt_aligned16(mask_bits)) return DIP_ERR_INVALID_ARG;
    if (d < 1 || d > DIP_MAX_D || k < 1 || k > d) return DIP_ERR_INVALID_ARG;
    if (!(gamma >= 0.0f) || !isfinite(gamma)) return DIP_ERR_INVALID_ARG;
    if (!cache_ok(st, d)) return DIP_ERR_INVALID_ARG;
    if (!fits(ctx, d, 0, 1)) return DIP_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    uint32_t *m = mask_bits ? mask_bits : ctx->mask;
    dip_status rc = dip_launch_select(ctx, x, nullptr, nullptr, 1, d, k, gamma, st->stamp, m, s);
    if (rc == DIP_OK) rc = dip_launch_cache_update(ctx, m, d, st->stamp, st->policy == DIP_CACHE_LFU ? st->count : nullptr, st->meta,
                                                   st->capacity, s);
    if (rc == DIP_OK && kept_idx) rc = dip_launch_mask_to_idx(ctx, m, 1, 1, d, kept_idx, k, nullptr, s);
    return rc;
}

static dip_status gemv_entry(dip_ctx *ctx, const dip_mlp_weights *w, int which, const float *v, int batch,
                             const int32_t *kept_idx, int n_kept, const uint32_t *mask_bits,
                             float *out, void *stream)
{
    if (!ctx_ok(ctx) || !weights_ok(w) || !v || !out) return DIP_ERR_INVALID_ARG;
    if (!kept_idx && !mask_bits) return DIP_ERR_INVALID_ARG;
    if (!dip_aligned16(v) || !dip_aligned16(out) || !opt_aligned16(mask_bits)) return DIP_ERR_INVALID_ARG;
    if (!fits(ctx, w->d_model, w->d_ff, batch)) return DIP_ERR_WORKSPACE;
    const int d_in = which == 0 ? w->d_model : w->d_ff;
    if (batch < 1 || batch > DIP_MAX_BATCH || n_kept < 1 || n_kept > d_in) return DIP_ERR_INVALID_ARG;
    if (batch > 1 && !mask_bits) return DIP_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    if (batch == 1 && kept_idx) {
        // the kernels take the kept columns as a bit set
        dip_status st = dip_launch_idx_to_mask(ctx, kept_idx, n_kept, d_in, ctx->mask_tmp, s);
        if (st != DIP_OK) return st;
        mask_bits = ctx->mask_tmp;
    }
    return dip_launch_gemv(ctx, w, which, v, batch, mask_bits, n_kept, out, s);
}

dip_status dip_sparse_gemv_gate_up(dip_ctx *ctx, const dip_mlp_weights *w, const float *x, int batch,
                                   const int32_t *kept_idx, int n_kept, const uint32_t *mask_bits,
                                   float *h, void *stream)
{
    return gemv_entry(ctx, w, 0, x, batch, kept_idx, n_kept, mask_bits, h, stream);
}

dip_status dip_sparse_gemv_down(dip_ctx *ctx, const dip_mlp_weights *w, const float *h, int batch,
                                const int32_t *kept_idx, int n_kept, const uint32_t *mask_bits,
                                float *y, void *stream)
{
    return gemv_entry(ctx, w, 1, h, batch, kept_idx, n_kept, mask_bits, y, stream);
}

dip_status dip_select_gemv_gate_up(dip_ctx *ctx, const dip_mlp_weights *w, const float *x, int k_x, float gamma,
                                   const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                                   uint32_t *mask_x, float *h, void *stream)
{
    if (!ctx_ok(ctx) || !weights_ok(w) || !x || !mask_x || !h) return DIP_ERR_INVALID_ARG;
    if (!dip_aligned16(x) || !dip_aligned16(mask_x) || !dip_aligned16(h)) return DIP_ERR_INVALID_ARG;
    if (k_x < 1 || k_x > w->d_model || !(gamma >= 0.0f) || !isfinite(gamma)) return DIP_ERR_INVALID_ARG;
    if (cache_gu && !cache_ok(cache_gu, w->d_model)) return DIP_ERR_INVALID_ARG;
    if (cache_d && !cache_ok(cache_d, w->d_ff)) return DIP_ERR_INVALID_ARG;
    if (!fits(ctx, w->d_model, w->d_ff, 1)) return DIP_ERR_WORKSPACE;
    if (!dip_gemv_fused_supported(ctx, w, 0, false) || !dip_gemv_fused_supported(ctx, w, 1, false)) return DIP_ERR_UNSUPPORTED;
    dip_gemv_keys hk = {ctx->coarse, cache_d ? cache_d->stamp : nullptr, gamma, 0};
    const dip_fused_select sx = {x, nullptr, nullptr, nullptr, k_x, gamma, cache_gu ? cache_gu->stamp : nullptr, mask_x};
    return dip_launch_gemv_fused(ctx, w, 0, &sx, h, (cudaStream_t)stream, &hk);
}

dip_status dip_select_gemv_down(dip_ctx *ctx, const dip_mlp_weights *w, const float *h, int k_h, float gamma,
                                const dip_cache_state *cache_d, uint32_t *mask_h, float *y, void *stream)
{
    if (!ctx_ok(ctx) || !weights_ok(w) || !h || !mask_h || !y) return DIP_ERR_INVALID_ARG;
    if (!dip_aligned16(h) || !dip_aligned16(mask_h) || !dip_aligned16(y)) return DIP_ERR_INVALID_ARG;
    if (k_h < 1 || k_h > w->d_ff || !(gamma >= 0.0f) || !isfinite(gamma)) return DIP_ERR_INVALID_ARG;
    if (cache_d && !cache_ok(cache_d, w->d_ff)) return DIP_ERR_INVALID_ARG;
    if (!fits(ctx, w->d_model, w->d_ff, 1)) return DIP_ERR_WORKSPACE;
    if (!dip_gemv_fused_supported(ctx, w, 1, false)) return DIP_ERR_UNSUPPORTED;
    const dip_fused_select sh = {h, nullptr, nullptr, ctx->coarse, k_h, gamma, cache_d ? cache_d->stamp : nullptr, mask_h};
    return dip_launch_gemv_fused(ctx, w, 1, &sh, y, (cudaStream_t)stream, nullptr);
}

// One sparse MLP step.  xb != nullptr: the step's input is formed first as
// x = (xa + xb) / rms(xa + xb), written to x_norm, in the same launch as its mask.
// slot_x / slot_h: where the masks go when the caller did not ask for them.  defer_join: leave
// the cache updates running on the side streams (the caller joins them later).
static dip_status step_impl(dip_ctx *ctx, const dip_mlp_weights *w,
                            const float *xa, const float *xb, float *x_norm,
                            int batch, int k_x, int k_h, float gamma,
                            const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                            float *y, const dip_step_outputs *out,
                            uint32_t *slot_x, uint32_t *slot_h, bool defer_join, bool join_follows, void *stream)
{
    const float *x = xb ? x_norm : xa;
    if (!ctx || !weights_ok(w) || !xa || !x || !y || !dip_aligned16(xa) || !dip_aligned16(x) || !dip_aligned16(y))
        return DIP_ERR_INVALID_ARG;
    if (batch < 1 || batch > DIP_MAX_BATCH || !outputs_aligned(out)) return DIP_ERR_INVALID_ARG;
    if (k_x < 1 || k_x > w->d_model || k_h < 1 || k_h > w->d_ff) return DIP_ERR_INVALID_ARG;
    if (!(gamma >= 0.0f) || !isfinite(gamma)) return DIP_ERR_INVALID_ARG;
    if (!fits(ctx, w->d_model, w->d_ff, batch)) return DIP_ERR_WORKSPACE;
    if (cache_gu && !cache_ok(cache_gu, w->d_model)) return DIP_ERR_INVALID_ARG;
    if (cache_d && !cache_ok(cache_d, w->d_ff)) return DIP_ERR_INVALID_ARG;
    if (batch > 1 && (cache_gu || cache_d)) return DIP_ERR_UNSUPPORTED;   // Algorithm 1 is per token

    cudaStream_t s = (cudaStream_t)stream;
    uint32_t *mask_x = out && out->mask_x ? out->mask_x : slot_x;
    float *h = out && out->h ? out->h : ctx->h;
    uint32_t *mask_h = out && out->mask_h ? out->mask_h : slot_h;
    const long long cap_x = (long long)batch * k_x, cap_h = (long long)batch * k_h;
    const int nmax_x = cap_x < w->d_model ? (int)cap_x : w->d_model;
    const int nmax_h = cap_h < w->d_ff ? (int)cap_h : w->d_ff;
    dip_status st;

    if (batch == 1 && dip_gemv_fused_supported(ctx, w, 0, xb != nullptr) && dip_gemv_fused_supported(ctx, w, 1, false)) {
        // The same four operations in two launches: each product builds the mask of its own input
        // (Eq. 7 / Eq. 8, or the ranking of Algorithm 1) while it already streams the rows that are
        // certain to be kept; the cache updates follow the launch that wrote their mask.
        dip_gemv_keys hk = {ctx->coarse, cache_d ? cache_d->stamp : nullptr, gamma, 0};
        const dip_fused_select sx = {xa, xb, x_norm, nullptr, k_x, gamma, cache_gu ? cache_gu->stamp : nullptr, mask_x};
        if ((st = dip_launch_gemv_fused(ctx, w, 0, &sx, h, s, &hk)) != DIP_OK) return st;
        if (cache_gu && (st = fork_cache_update(ctx, 0, mask_x, cache_gu, s)) != DIP_OK) return st;
        if (cache_d && join_follows) {
            // The caller waits for this step's cache updates right after it: the update of the down input
            // (the long one) then has to run BESIDE the down product, which it can only with the mask
            // from a select kernel of its own.
            st = dip_launch_select(ctx, h, nullptr, nullptr, 1, w->d_ff, k_h, gamma, cache_d->stamp, mask_h, s, ctx->coarse);
            if (st != DIP_OK) return st;
            if ((st = fork_cache_update(ctx, 1, mask_h, cache_d, s)) != DIP_OK) return st;
            if ((st = dip_launch_gemv(ctx, w, 1, h, 1, mask_h, nmax_h, y, s)) != DIP_OK) return st;
        } else {
            const dip_fused_select sh = {h, nullptr, nullptr, ctx->coarse, k_h, gamma, cache_d ? cache_d->stamp : nullptr, mask_h};
            if ((st = dip_launch_gemv_fused(ctx, w, 1, &sh, y, s, nullptr)) != DIP_OK) return st;
            if (cache_d && (st = fork_cache_update(ctx, 1, mask_h, cache_d, s)) != DIP_OK) return st;
        }
    } else {
        // m_x = topK(score(x))            (Eq. 7; the ranking of Algorithm 1 when a cache is given)
        st = dip_launch_select(ctx, xa, xb, x_norm, batch, w->d_model, k_x, gamma,
                               cache_gu ? cache_gu->stamp : nullptr, mask_x, s);
        if (st != DIP_OK) return st;
        // c' = cache_update(c, m_x)       (Algorithm 1; beside the products, which do not need it)
        if (cache_gu && (st = fork_cache_update(ctx, 0, mask_x, cache_gu, s)) != DIP_OK) return st;
        // h = (W~u x) * silu(W~g x)       (Eq. 2 inside Eq. 3)
        // (a single-token product also leaves the top bits of the rank keys of h for the next launch)
        dip_gemv_keys hk = {ctx->coarse, cache_d ? cache_d->stamp : nullptr, gamma, 0};
        st = dip_launch_gemv(ctx, w, 0, x, batch, mask_x, nmax_x, h, s, nullptr,
                             w->d_ff >= ctx->coarse_min_d && (w->d_ff & 31) == 0 ? &hk : nullptr);
        if (st != DIP_OK) return st;
        // m_h = topK(score(h))            (Eq. 8: the GLU of the already sparsified gate/up)
        st = dip_launch_select(ctx, h, nullptr, nullptr, batch, w->d_ff, k_h, gamma,
                               cache_d ? cache_d->stamp : nullptr, mask_h, s, hk.written ? ctx->coarse : nullptr);
        if (st != DIP_OK) return st;
        if (cache_d && (st = fork_cache_update(ctx, 1, mask_h, cache_d, s)) != DIP_OK) return st;
        // y = W~d h                       (Eq. 1 inside Eq. 3)
        st = dip_launch_gemv(ctx, w, 1, h, batch, mask_h, nmax_h, y, s);
        if (st != DIP_OK) return st;
    }

    if (out && out->idx_x && (st = dip_launch_mask_to_idx(ctx, mask_x, batch, 1, w->d_model, out->idx_x, k_x, nullptr, s)) != DIP_OK)
        return st;
    if (out && out->idx_h && (st = dip_launch_mask_to_idx(ctx, mask_h, batch, 1, w->d_ff, out->idx_h, k_h, nullptr, s)) != DIP_OK)
        return st;
    if (out && out->union_counts && batch > 1) {
        if ((st = dip_launch_mask_to_idx(ctx, mask_x, 1, batch, w->d_model, nullptr, 0, out->union_counts, s)) != DIP_OK) return st;
        if ((st = dip_launch_mask_to_idx(ctx, mask_h, 1, batch, w->d_ff, nullptr, 0, out->union_counts + 1, s)) != DIP_OK) return st;
    }
    return defer_join ? DIP_OK : join_cache_updates(ctx, s);
}

dip_status dip_mlp_step(dip_ctx *ctx, const dip_mlp_weights *w,
                        const float *x, int batch, int k_x, int k_h, float gamma,
                        const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                        float *y, const dip_step_outputs *out, void *stream)
{
    if (!ctx_ok(ctx)) return DIP_ERR_INVALID_ARG;
    return step_impl(ctx, w, x, nullptr, nullptr, batch, k_x, k_h, gamma, cache_gu, cache_d, y, out,
                     ctx->mask, ctx->mask_h, false, true, stream);
}

// One masked input of the two-tier step.  On the step's path: the hit / miss split, the list of
// the misses, the hits' product; beside it one stream fetches the misses into the staging rows
// (the misses' product waits for that) and another keeps the books: cache update, slot
// assignment, and the move of the staged rows of the inserted columns into their slots.  The
// book-keeping is joined at the end of the call.
static dip_status tiered_half(dip_ctx *ctx, const dip_mlp_weights *w, int which, const dip_tier *t,
                              const dip_cache_state *c, const float *v, const uint32_t *mask_bits, int k,
                              float *out, cudaStream_t s)
{
    const int words = (t->d + 31) / 32;
    dip_status st = dip_launch_tier_split(ctx, t, mask_bits, s);
    if (st != DIP_OK) return st;
    // the misses as an ascending list: fetch[0] = how many, fetch[4 ..] = their columns
    if ((st = dip_launch_mask_to_idx(ctx, t->split + words, 1, 1, t->d, t->fetch + 4, 0, t->fetch, s)) != DIP_OK) return st;
    cudaStream_t sf = ctx->tier_fetch[which], sb = ctx->tier_book[which];
    DIP_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_tier_fork[which], s));
    DIP_CUDA_TRY(ctx, cudaStreamWaitEvent(sf, ctx->ev_tier_fork[which], 0));
    DIP_CUDA_TRY(ctx, cudaStreamWaitEvent(sb, ctx->ev_tier_fork[which], 0));
    if ((st = dip_launch_tier_fetch(ctx, t, sf)) != DIP_OK) return st;
    DIP_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_tier_fetched[which], sf));
    st = dip_launch_cache_update(ctx, mask_bits, c->d, c->stamp, c->policy == DIP_CACHE_LFU ? c->count : nullptr,
                                 c->meta, c->capacity, sb);
    if (st != DIP_OK) return st;
    if ((st = dip_launch_tier_assign(ctx, t, mask_bits, c->stamp, sb)) != DIP_OK) return st;
    DIP_CUDA_TRY(ctx, cudaStreamWaitEvent(sb, ctx->ev_tier_fetched[which], 0));
    if ((st = dip_launch_tier_install(ctx, t, sb)) != DIP_OK) return st;
    DIP_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_tier_booked[which], sb));
    dip_gemv_rows rows = {t->arena, t->loc, 1};
    if ((st = dip_launch_gemv(ctx, w, which, v, 1, t->split, k, out, s, &rows)) != DIP_OK) return st;
    DIP_CUDA_TRY(ctx, cudaStreamWaitEvent(s, ctx->ev_tier_fetched[which], 0));
    rows.mode = 2;
    return dip_launch_gemv(ctx, w, which, v, 1, t->split + words, k, out, s, &rows);
}

dip_status dip_mlp_step_tiered(dip_ctx *ctx, const dip_mlp_weights *w,
                               const dip_tier *tier_gu, const dip_tier *tier_d,
                               const float *x, int k_x, int k_h, float gamma,
                               const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                               float *y, const dip_step_outputs *out, void *stream)
{
    if (!ctx_ok(ctx) || !w || !dims_ok(w->wtype, w->d_model, w->d_ff) || !x || !y || !dip_aligned16(x) ||
        !dip_aligned16(y) || !outputs_aligned(out))
        return DIP_ERR_INVALID_ARG;
    if (!fits(ctx, w->d_model, w->d_ff, 1)) return DIP_ERR_WORKSPACE;
    if (w->wtype == DIP_W_INT4_G128 &&
        (!w->gate_up_scales || !w->down_scales || !dip_aligned16(w->gate_up_scales) || !dip_aligned16(w->down_scales)))
        return DIP_ERR_INVALID_ARG;
    if (k_x < 1 || k_x > w->d_model || k_h < 1 || k_h > w->d_ff) return DIP_ERR_INVALID_ARG;
    if (!(gamma >= 0.0f) || !isfinite(gamma)) return DIP_ERR_INVALID_ARG;
    if (!cache_ok(cache_gu, w->d_model) || !cache_ok(cache_d, w->d_ff)) return DIP_ERR_INVALID_ARG;
    if (!tier_ok(tier_gu, cache_gu, packed_row_bytes(w->wtype, (size_t)2 * w->d_ff), k_x) ||
        !tier_ok(tier_d, cache_d, packed_row_bytes(w->wtype, (size_t)w->d_model), k_h))
        return DIP_ERR_INVALID_ARG;
    if (ctx->side_busy[0] || ctx->side_busy[1]) return DIP_ERR_INVALID_ARG;   // side streams are in use

    cudaStream_t s = (cudaStream_t)stream;
    uint32_t *mask_x = out && out->mask_x ? out->mask_x : ctx->mask;
    float *h = out && out->h ? out->h : ctx->h;
    uint32_t *mask_h = out && out->mask_h ? out->mask_h : ctx->mask_h;
    dip_status st;
    // m_x from the cache-aware ranking (Algorithm 1), then the gate/up half out of the two tiers
    st = dip_launch_select(ctx, x, nullptr, nullptr, 1, w->d_model, k_x, gamma, cache_gu->stamp, mask_x, s);
    if (st != DIP_OK) return st;
    if ((st = tiered_half(ctx, w, 0, tier_gu, cache_gu, x, mask_x, k_x, h, s)) != DIP_OK) return st;
    // m_h likewise (Eq. 8), then the down half
    st = dip_launch_select(ctx, h, nullptr, nullptr, 1, w->d_ff, k_h, gamma, cache_d->stamp, mask_h, s);
    if (st != DIP_OK) return st;
    if ((st = tiered_half(ctx, w, 1, tier_d, cache_d, h, mask_h, k_h, y, s)) != DIP_OK) return st;
    if (out && out->idx_x && (st = dip_launch_mask_to_idx(ctx, mask_x, 1, 1, w->d_model, out->idx_x, k_x, nullptr, s)) != DIP_OK)
        return st;
    if (out && out->idx_h && (st = dip_launch_mask_to_idx(ctx, mask_h, 1, 1, w->d_ff, out->idx_h, k_h, nullptr, s)) != DIP_OK)
        return st;
    // the book-keeping of both inputs has to be through before the call's work ends
    DIP_CUDA_TRY(ctx, cudaStreamWaitEvent(s, ctx->ev_tier_booked[0], 0));
    DIP_CUDA_TRY(ctx, cudaStreamWaitEvent(s, ctx->ev_tier_booked[1], 0));
    return DIP_OK;
}

dip_status dip_mlp_step_neuron_pruned(dip_ctx *ctx, const dip_neuron_weights *w, int prune_by,
                                      const float *x, int k, float *y,
                                      float *p_out, uint32_t *mask_out, int32_t *idx_out, float *h_out,
                                      void *stream)
{
    if (!ctx_ok(ctx) || !w || !x || !y || !dip_aligned16(x) || !dip_aligned16(y) || !opt_aligned16(mask_out))
        return DIP_ERR_INVALID_ARG;
    if (w->wtype == DIP_W_INT4_G128) return DIP_ERR_UNSUPPORTED;
    if (!dims_ok(w->wtype, w->d_model, w->d_ff)) return DIP_ERR_INVALID_ARG;
    if (!fits(ctx, w->d_model, w->d_ff, 1)) return DIP_ERR_WORKSPACE;
    if (!w->gate || !w->up || !w->down || !dip_aligned16(w->gate) || !dip_aligned16(w->up) || !dip_aligned16(w->down))
        return DIP_ERR_INVALID_ARG;
    if (prune_by != DIP_PRUNE_BY_GATE && prune_by != DIP_PRUNE_BY_UP) return DIP_ERR_INVALID_ARG;
    if (k < 1 || k > w->d_ff) return DIP_ERR_INVALID_ARG;
    if ((p_out && !dip_aligned16(p_out)) || (h_out && !dip_aligned16(h_out))) return DIP_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    float *p = p_out ? p_out : ctx->p;
    float *h = h_out ? h_out : ctx->h;
    uint32_t *mask = mask_out ? mask_out : ctx->mask_h;
    int32_t *idx = idx_out ? idx_out : ctx->idx_h;
    const bool by_gate = prune_by == DIP_PRUNE_BY_GATE;
    dip_status st;
    // the dense, ranking activation: p = silu(W^g x) (Gate pruning) or W^u x (Up pruning)
    st = dip_launch_rowdot(ctx, w->wtype, by_gate ? w->gate : w->up, w->d_model, w->d_ff, x, nullptr, w->d_ff,
                           by_gate ? 1 : 0, nullptr, p, s);
    if (st != DIP_OK) return st;
    // m = topK(|p|) over the neurons (Eq. 5), as a bit set and as an ascending list
    if ((st = dip_launch_select(ctx, p, nullptr, nullptr, 1, w->d_ff, k, 1.0f, nullptr, mask, s)) != DIP_OK) return st;
    if ((st = dip_launch_mask_to_idx(ctx, mask, 1, 1, w->d_ff, idx, k, nullptr, s)) != DIP_OK) return st;
    // the kept rows of the other matrix: h_j = p_j * (W^u x)_j, or p_j * silu((W^g x)_j); 0 elsewhere
    DIP_CUDA_TRY(ctx, cudaMemsetAsync(h, 0, sizeof(float) * (size_t)w->d_ff, s));
    st = dip_launch_rowdot(ctx, w->wtype, by_gate ? w->up : w->gate, w->d_model, w->d_ff, x, idx, k,
                           by_gate ? 0 : 1, p, h, s);
    if (st != DIP_OK) return st;
    // y = sum over the kept neurons of W^d[:, j] h_j
    dip_mlp_weights wd = {};
    wd.wtype = w->wtype;
    wd.d_model = w->d_model;
    wd.d_ff = w->d_ff;
    wd.down = w->down;
    return dip_launch_gemv(ctx, &wd, 1, h, 1, mask, k, y, s);
}

dip_status dip_residual_rmsnorm(dip_ctx *ctx, const float *x, const float *y,
                                int batch, int d, float *x_next, void *stream)
{
    if (!ctx_ok(ctx) || !x || !y || !x_next) return DIP_ERR_INVALID_ARG;
    if (!dip_aligned16(x) || !dip_aligned16(y) || !dip_aligned16(x_next)) return DIP_ERR_INVALID_ARG;
    if (batch < 1 || batch > DIP_MAX_BATCH || d < 1 || d > DIP_MAX_D) return DIP_ERR_INVALID_ARG;
    return dip_launch_residual_rmsnorm(ctx, x, y, batch, d, x_next, (cudaStream_t)stream);
}

static dip_status stack_impl(dip_ctx *ctx, int n_layers, const dip_mlp_weights *layers,
                             const float *x_in, int batch, int k_x, int k_h, float gamma,
                             const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                             float *x_out, float *y_last, const dip_stack_probe *probe, void *stream)
{
    if (!ctx_ok(ctx) || n_layers < 1 || !layers || !x_in || !x_out) return DIP_ERR_INVALID_ARG;
    if (!dip_aligned16(x_in) || !dip_aligned16(x_out) || !opt_aligned16(y_last)) return DIP_ERR_INVALID_ARG;
    if (batch < 1 || batch > DIP_MAX_BATCH) return DIP_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l) {
        if (!weights_ok(&layers[l])) return DIP_ERR_INVALID_ARG;
        if (layers[l].d_model != layers[0].d_model || layers[l].d_ff != layers[0].d_ff) return DIP_ERR_INVALID_ARG;
    }
    const int d = layers[0].d_model, d_ff = layers[0].d_ff;
    if (!fits(ctx, d, d_ff, batch)) return DIP_ERR_WORKSPACE;
    if (probe && (!probe->x || !probe->mask_x || !probe->h || !probe->mask_h || !probe->y || !dip_aligned16(probe->x) ||
                  !dip_aligned16(probe->mask_x) || !dip_aligned16(probe->h) || !dip_aligned16(probe->mask_h) ||
                  !dip_aligned16(probe->y) || (d & 127) || (d_ff & 127)))
        return DIP_ERR_INVALID_ARG;      // (per-layer slices of the arrays stay 16-byte aligned)
    cudaStream_t s = (cudaStream_t)stream;
    const size_t ring_words = (size_t)ctx->max_d / 32;
    // x_0 = x_in; for l > 0 the chaining x_l = rmsnorm(x_{l-1} + y_{l-1}) runs inside layer l's
    // first mask launch.  x and y ping-pong between two workspace buffers each.
    const float *x_prev = x_in;
    const float *y_prev = nullptr;
    const bool ca = cache_gu || cache_d;
    if (probe) DIP_CUDA_TRY(ctx, cudaMemcpyAsync(probe->x, x_in, sizeof(float) * (size_t)batch * d, cudaMemcpyDeviceToDevice, s));
    for (int l = 0; l < n_layers; ++l) {
        float *y = (l == n_layers - 1 && y_last) ? y_last : ((l & 1) ? ctx->y2 : ctx->y);
        float *x_l = (l & 1) ? ctx->xb : ctx->xa;
        // with caches each layer's masks get their own slot: the updates that read them run
        // beside later layers
        const int slot = ca ? l % DIP_RING_LAYERS : 0;
        uint32_t *slot_x = batch == 1 ? ctx->mask_ring + (size_t)slot * ring_words : ctx->mask;
        uint32_t *slot_h = batch == 1 ? ctx->mask_ring + (size_t)(DIP_RING_LAYERS + slot) * ring_words : ctx->mask_h;
        dip_step_outputs po = {};
        if (probe) {
            y = probe->y + (size_t)l * batch * d;
            x_l = probe->x + (size_t)l * batch * d;
            po.mask_x = probe->mask_x + (size_t)l * batch * (d / 32);
            po.mask_h = probe->mask_h + (size_t)l * batch * (d_ff / 32);
            po.h = probe->h + (size_t)l * batch * d_ff;
        }
        dip_status st = step_impl(ctx, &layers[l], x_prev, y_prev, y_prev ? x_l : nullptr, batch, k_x, k_h, gamma,
                                  cache_gu ? &cache_gu[l] : nullptr, cache_d ? &cache_d[l] : nullptr,
                                  y, probe ? &po : nullptr, slot_x, slot_h, true,
                                  l == n_layers - 1 || (ca && slot == DIP_RING_LAYERS - 1), stream);
        if (st != DIP_OK) return st;
        if (ca && slot == DIP_RING_LAYERS - 1 && (st = join_cache_updates(ctx, s)) != DIP_OK) return st;
        if (y_prev) x_prev = x_l;
        y_prev = y;
    }
    dip_status st = dip_residual_rmsnorm(ctx, x_prev, y_prev, batch, d, x_out, stream);
    if (st != DIP_OK) return st;
    return join_cache_updates(ctx, s);
}

dip_status dip_stack_step(dip_ctx *ctx, int n_layers, const dip_mlp_weights *layers,
                          const float *x_in, int batch, int k_x, int k_h, float gamma,
                          const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                          float *x_out, float *y_last, void *stream)
{
    return stack_impl(ctx, n_layers, layers, x_in, batch, k_x, k_h, gamma, cache_gu, cache_d, x_out, y_last, nullptr,
                      stream);
}

dip_status dip_stack_step_probed(dip_ctx *ctx, int n_layers, const dip_mlp_weights *layers,
                                 const float *x_in, int batch, int k_x, int k_h, float gamma,
                                 const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                                 float *x_out, const dip_stack_probe *probe, void *stream)
{
    if (!probe) return DIP_ERR_INVALID_ARG;
    return stack_impl(ctx, n_layers, layers, x_in, batch, k_x, k_h, gamma, cache_gu, cache_d, x_out, nullptr, probe,
                      stream);
}

// ---- device-side timeline (diagnostics) ----
static dip_status trace_clear(dip_ctx *ctx)
{
    static unsigned long long init[DIP_TRACE_SLOTS * DIP_TRACE_WORDS];
    for (int i = 0; i < DIP_TRACE_SLOTS; ++i) {
        init[DIP_TRACE_WORDS * i + 0] = ~0ull;
        init[DIP_TRACE_WORDS * i + 1] = ~0ull;
        init[DIP_TRACE_WORDS * i + 2] = 0;
        init[DIP_TRACE_WORDS * i + 3] = 0;
    }
    DIP_CUDA_TRY(ctx, cudaDeviceSynchronize());
    DIP_CUDA_TRY(ctx, cudaMemcpy(ctx->trace, init, sizeof(init), cudaMemcpyHostToDevice));
    return DIP_OK;
}

dip_status dip_trace_begin(dip_ctx *ctx)
{
    if (!ctx_ok(ctx)) return DIP_ERR_INVALID_ARG;
    ctx->trace_on = 1;
    ctx->trace_next = 0;
    return trace_clear(ctx);
}

dip_status dip_trace_reset(dip_ctx *ctx)
{
    if (!ctx_ok(ctx)) return DIP_ERR_INVALID_ARG;
    return trace_clear(ctx);
}

dip_status dip_trace_read(dip_ctx *ctx, dip_trace_record *out, int max_records, int *n_out)
{
    if (!ctx_ok(ctx) || !out || !n_out || max_records < 0) return DIP_ERR_INVALID_ARG;
    static unsigned long long host[DIP_TRACE_SLOTS * DIP_TRACE_WORDS];
    DIP_CUDA_TRY(ctx, cudaDeviceSynchronize());
    DIP_CUDA_TRY(ctx, cudaMemcpy(host, ctx->trace, sizeof(host), cudaMemcpyDeviceToHost));
    int n = 0;
    for (int i = 0; i < ctx->trace_next && n < max_records; ++i) {
        const unsigned long long *w = host + (size_t)DIP_TRACE_WORDS * i;
        if (w[0] == ~0ull) continue;               // that launch has not run since the last reset
        out[n].kind = ctx->trace_kind[i];
        out[n].t_start_ns = w[0];
        out[n].t_ready_ns = w[1];
        out[n].t_end_ns = w[2];
        out[n].t_aux_ns = w[3];
        ++n;
    }
    *n_out = n;
    return DIP_OK;
}

dip_status dip_trace_end(dip_ctx *ctx)
{
    if (!ctx_ok(ctx)) return DIP_ERR_INVALID_ARG;
    ctx->trace_on = 0;
    return DIP_OK;
}

}  // extern "C"
