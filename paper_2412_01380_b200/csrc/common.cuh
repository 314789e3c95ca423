// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include <atomic>

#include "dip.h"

constexpr int DIP_RING_LAYERS = 128;
constexpr int DIP_TRACE_SLOTS = 1024;
constexpr int DIP_TRACE_WORDS = 4;   // first start, dependency ready, last end, auxiliary

// Scratch workspace of a context.  All device memory the library itself owns.
struct dip_ctx {
    int device;
    int sm_count;
    int max_d;           // largest masked dimension the workspace was sized for
    int max_batch;       // most tokens per call the workspace was sized for
    int gemv_seg;        // 0 = choose per launch; else force the GEMV segment width (dip_options)
    int gemv_direct;     // one token, F32/BF16: plain-load kernel instead of the copy ring
    unsigned long long wait_limit_ns;   // bound of every in-kernel wait
    // split-row partial sums of the two GEMVs (binary32)
    float *partials;
    size_t partials_floats;
    // one arrival counter per output slab; zero between launches
    unsigned int *tickets;
    int n_tickets;
    // intermediates of dip_mlp_step when the caller does not ask for them
    float *h;            // [max_batch][max_d]
    float *y;            // [max_batch][max_d]   (stack runner, even layers)
    float *y2;           // [max_batch][max_d]   (stack runner, odd layers)
    float *xa;           // [max_batch][max_d]   (stack runner ping)
    float *xb;           // [max_batch][max_d]   (stack runner pong)
    float *p;            // [max_d]   ranking activation of Gate / Up pruning
    uint32_t *mask;      // [max_batch][max_d/32]  masks of x
    int32_t *idx;        // [max_batch][max_d]     kept indices of x
    uint32_t *mask_h;    // same for h
    int32_t *idx_h;
    int32_t *union_idx;  // [max_d]
    int32_t *counts;     // [8] device scalars (union sizes)
    uint32_t *mask_ring; // [2][DIP_RING_LAYERS][max_d/32] per-layer mask slots of the stack runner
    uint32_t *mask_tmp;  // [max_d/32] list-based GEMV entry points
    uint16_t *coarse;    // [max_batch][max_d] top 16 bits of the rank keys of h, left by the gate/up product
    uint16_t *xt;        // [max_d][32] batched decode: per row of the union, the tokens' values as bfloat16 (16 high, 16 low halves)
    int coarse_min_d;    // smallest d_ff for which the step ranks h from those
    int *status;         // sticky device status word (0 = fine)
    int fuse_select;     // single-token F32 / BF16 steps: the products build their own masks
    // the cache updates run beside the GEMVs: one side stream per cache kind
    cudaStream_t side[2];
    cudaEvent_t ev_fork[2], ev_join[2];
    bool side_busy[2];
    // two-tier step, per masked input: a stream that fetches the misses and one that keeps the books
    cudaStream_t tier_fetch[2], tier_book[2];
    cudaEvent_t ev_tier_fork[2], ev_tier_fetched[2], ev_tier_booked[2];
    // device-side timeline (diagnostics): one slot of DIP_TRACE_WORDS words per launch
    unsigned long long *trace;
    int trace_on;
    int trace_next;
    unsigned char trace_kind[DIP_TRACE_SLOTS];
    char err[256];
};

// Slot of the next launch, or nullptr when tracing is off.
static inline unsigned long long *dip_trace_slot(dip_ctx *ctx, int kind)
{
    if (!ctx->trace_on || ctx->trace_next >= DIP_TRACE_SLOTS) return nullptr;
    ctx->trace_kind[ctx->trace_next] = (unsigned char)kind;
    return ctx->trace + (size_t)DIP_TRACE_WORDS * ctx->trace_next++;
}


#define DIP_CUDA_TRY(ctx, call)                                                        \
    do {                                                                               \
        cudaError_t e_ = (call);                                                       \
        if (e_ != cudaSuccess) {                                                       \
            snprintf((ctx)->err, sizeof((ctx)->err), "%s: %s", #call,                  \
                     cudaGetErrorString(e_));                                          \
            return DIP_ERR_CUDA;                                                       \
        }                                                                              \
    } while (0)

#ifdef __CUDACC__
// Timeline stamps (nanoseconds of %globaltimer) taken by thread 0 of each CTA when tr != nullptr:
// word 0 = earliest kernel entry, 1 = earliest return from the dependency wait, 2 = latest exit,
// 3 = latest auxiliary mark.
__device__ __forceinline__ unsigned long long dip_gtime()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define DIP_TRACE_MIN(tr, i) do { if ((tr) && threadIdx.x == 0) atomicMin(&(tr)[i], dip_gtime()); } while (0)
#define DIP_TRACE_MAX(tr, i) do { if ((tr) && threadIdx.x == 0) atomicMax(&(tr)[i], dip_gtime()); } while (0)

// Programmatic dependent launch: a kernel may be scheduled before its predecessor in the stream
// has finished; it must not touch the predecessor's results before this wait returns.
__device__ __forceinline__ void dip_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel in the stream be scheduled early (it still waits as above).
__device__ __forceinline__ void dip_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }


// Launch on `stream` with programmatic dependent launch enabled: the kernel may start while the
// previous kernel in the stream drains; it orders itself with dip_grid_dependency_wait().
template <typename... KArgs, typename... Args>
static inline cudaError_t dip_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                         cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

static inline bool dip_aligned16(const void *p) { return (((uintptr_t)p) & 15u) == 0; }

// cudaFuncSetAttribute applies to the current device only, so "this kernel's dynamic shared memory
// limit has been raised" is remembered per device (one object per kernel instantiation).
constexpr int DIP_MAX_DEVICES = 64;
struct dip_per_device_once {
    std::atomic<unsigned char> done[DIP_MAX_DEVICES];
};
template <typename K>
static inline cudaError_t dip_raise_smem_limit(dip_per_device_once &once, int device, K kernel, size_t bytes)
{
    const bool tracked = device >= 0 && device < DIP_MAX_DEVICES;
    if (tracked && once.done[device].load(std::memory_order_acquire)) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && tracked) once.done[device].store(1, std::memory_order_release);
    return e;
}

// ---- launchers implemented in the kernel files (host functions) -----------------

// topk.cu: mask of each row: k largest rank keys (|x|, or |x| * (resident ? 1 : gamma) when stamp
// is given).  xb != nullptr: the row is first formed as (xa + xb) / rms(xa + xb), written to x_out.
// coarse != nullptr (no xb, d % 32 == 0; several rows only without stamps): the producer of xa has left the top 16 bits of
// every column's rank key there (dip_gemv_keys), and the launch reads those instead of all of
// xa and stamp.
dip_status dip_launch_select(dip_ctx *ctx, const float *xa, const float *xb, float *x_out, int batch, int d, int k,
                             float gamma, const int32_t *stamp, uint32_t *mask_bits, cudaStream_t stream,
                             const uint16_t *coarse = nullptr);

// topk.cu: LRU cache update from (mask, state).
// count != nullptr: LFU (use counters), else LRU.
dip_status dip_launch_cache_update(dip_ctx *ctx, const uint32_t *mask_bits, int d, int32_t *stamp, int32_t *count,
                                   int32_t *meta, int capacity, cudaStream_t stream);

// topk.cu: per-device set-up of the mask kernels (dynamic shared memory limit).
dip_status dip_init_mask_kernels(dip_ctx *ctx);

// topk.cu: `rows` index lists, each from the OR of `nb` consecutive masks; lengths to count_out.
dip_status dip_launch_mask_to_idx(dip_ctx *ctx, const uint32_t *mask_bits, int rows, int nb, int d,
                                  int32_t *idx_out, int out_stride, int32_t *count_out, cudaStream_t stream);

// topk.cu: x_next = (x + y) / rms(x + y) per row.
dip_status dip_launch_residual_rmsnorm(dip_ctx *ctx, const float *x, const float *y, int batch, int d,
                                       float *x_next, cudaStream_t stream);

// gemv.cu: gather GEMV over the rows named by the mask bits (OR over the batch; token b uses a
// row only if its own bit is set).
//   which = 0: gate/up bundle with the silu*up epilogue, out = h[batch][d_ff]
//   which = 1: down, out = y[batch][d_model]
// n_kept_max bounds the number of rows (sizes the row parts).
// rows != nullptr (two-tier execution, one token): the packed row of column i is
// base + loc[i] * row_bytes instead of row i of the weights; mode 1 leaves this launch's row parts
// in the workspace, mode 2 adds its own behind them and then sums both launches' parts into out
// (so that the first launch can run while the second one's rows are still being fetched).
struct dip_gemv_rows {
    const void *base;
    const int32_t *loc;
    int mode;            // 0 = a launch of its own
};
// keys != nullptr (which = 0): the caller ranks h next and wants the top 16 bits of every rank key
// |h_j| * (stamp[j] >= 0 ? 1 : gamma) (stamp == nullptr: |h_j|) in keys->coarse[j].  Only the
// single-token F32 / BF16 launch writes them; keys->written says whether it did.  The stamps are
// read while the product runs, so nothing may change them between this launch and the ranking.
struct dip_gemv_keys {
    uint16_t *coarse;        // [d_ff]
    const int32_t *stamp;    // cache state of the down input, or nullptr
    float gamma;
    int written;             // out
};
dip_status dip_launch_gemv(dip_ctx *ctx, const dip_mlp_weights *w, int which,
                           const float *v, int batch, const uint32_t *mask_bits, int n_kept_max,
                           float *out, cudaStream_t stream, const dip_gemv_rows *rows = nullptr,
                           dip_gemv_keys *keys = nullptr);

// gemv_fused.cu: the product `which` of a single-token step together with the select of its input.
struct dip_fused_select {
    const float *xa;         // gate/up: x, or the previous layer's x when xb is given; down: h
    const float *xb;         // gate/up, chained layers: the previous layer's y (else nullptr)
    float *x_out;            // gate/up with xb: receives x = (xa + xb) / rms(xa + xb)
    const uint16_t *coarse;  // down: the 16-bit rank keys that the gate/up product left
    int k;
    float gamma;
    const int32_t *stamp;    // cache state of the input (cache-aware ranking) or nullptr
    uint32_t *mask_out;      // receives the mask
};
bool dip_gemv_fused_supported(const dip_ctx *ctx, const dip_mlp_weights *w, int which, bool norm);
dip_status dip_launch_gemv_fused(dip_ctx *ctx, const dip_mlp_weights *w, int which, const dip_fused_select *sel,
                                 float *out, cudaStream_t stream, dip_gemv_keys *keys);

// gemv.cu: one tiny kernel whose bounded wait runs out (sets the status word to 1).
dip_status dip_launch_bounded_wait_selftest(dip_ctx *ctx, unsigned long long limit_ns, unsigned long long *waited_ns,
                                            cudaStream_t stream);

// gemv.cu: bit set from an ascending index list.
dip_status dip_launch_idx_to_mask(dip_ctx *ctx, const int32_t *idx, int n, int d, uint32_t *mask, cudaStream_t stream);

// tier.cu: before the cache update of a mask: its hits (resident columns, with their arena rows)
// and its misses.
dip_status dip_launch_tier_split(dip_ctx *ctx, const dip_tier *t, const uint32_t *mask_bits, cudaStream_t stream);
// tier.cu: after the cache update: evicted columns free their slots, inserted columns get slots,
// and the install list says which staging rows move where.
dip_status dip_launch_tier_assign(dip_ctx *ctx, const dip_tier *t, const uint32_t *mask_bits, const int32_t *stamp,
                                  cudaStream_t stream);
// tier.cu: copy the rows of the miss list (fetch[0] columns at fetch + 4) from the slow tier into
// the staging rows of the arena, in list order, and point loc at them.
dip_status dip_launch_tier_fetch(dip_ctx *ctx, const dip_tier *t, cudaStream_t stream);
// tier.cu: move the staged rows of the inserted columns into their cache slots (install list).
dip_status dip_launch_tier_install(dip_ctx *ctx, const dip_tier *t, cudaStream_t stream);

// rowdot.cu: out_j = [silu](W[j, :] . x) [* mul_j] for the listed rows (rows == nullptr: rows
// 0 .. n_rows-1) of a row-major [d_ff][d_model] matrix; F32 or BF16.
dip_status dip_launch_rowdot(dip_ctx *ctx, int wtype, const void *W, int d_model, int d_ff, const float *x,
                             const int32_t *rows, int n_rows, int silu, const float *mul, float *out,
                             cudaStream_t stream);

// pack.cu
dip_status dip_launch_pack(dip_ctx *ctx, int wtype, int d_model, int d_ff,
                           const void *Wg, const void *Wu, const void *Wd,
                           const void *Sg, const void *Su, const void *Sd,
                           const dip_mlp_weights *out, cudaStream_t stream);
