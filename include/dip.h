/*
 * dip.h — C ABI of the B200 (sm_100a) sparse SwiGLU decode-MLP library for
 * Dynamic Input Pruning (DIP) and its cache-aware variant (DIP-CA),
 * arxiv 2412.01380.
 *
 * The library computes, per decode token and per MLP block, the sparse MLP of
 * Eq. 3 with the input-pruning masks of Eq. 7-8:
 *
 *     m_x = topK(score(x))            keep k_x of the d_model input columns
 *     h   = (W~u x) * silu(W~g x)     gate/up read only the kept columns of W^g, W^u
 *     m_h = topK(score(h))            keep k_h of the d_ff columns of W^d
 *     y   = W~d h                     down reads only the kept columns of W^d
 *
 * where score is |.| (DIP) or the cache-aware re-weighting of Eq. 10 with the
 * column-cache update of Algorithm 1 (DIP-CA).
 *
 * Conventions
 *  - Every data pointer is DEVICE memory owned by the caller unless a comment
 *    says "host".  Structs and the context handle are host memory.
 *  - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and
 *    return without synchronising.  Results are valid once the stream reaches
 *    the end of the enqueued work.
 *  - Calls on the same context must not overlap on the GPU (they share the
 *    context's scratch workspace): use one context per concurrently running
 *    stream.  With a column cache the state update of Algorithm 1 runs on a
 *    stream of the context's own, beside the products that do not depend on
 *    it, and is joined back into `stream` before the call's work ends.
 *  - Arguments are validated on the host before anything is launched; a failed
 *    validation returns an error code and launches nothing.
 *  - Data pointers (vectors, masks, cache state, weights) must be 16-byte
 *    aligned; a misaligned one is DIP_ERR_INVALID_ARG.
 *  - Float vectors are binary32.  Masks are bit sets: bit (i & 31) of word
 *    (i >> 5) is column i.  Kept-index lists are int32 in ascending order.
 *  - Top-k ties are resolved in favour of the lower column index, so every
 *    result is unique; the paper does not fix a tie rule.
 *  - Floating-point sums run in a fixed order: results are bit-reproducible
 *    from run to run on the same device and library build.
 */
#ifndef DIP_H
#define DIP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DIP_OK = 0,
    DIP_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, k or capacity out of range, bad size   */
    DIP_ERR_UNSUPPORTED = 2,   /* valid request the library does not implement (see each call)      */
    DIP_ERR_CUDA = 3,          /* a CUDA runtime call failed; see dip_last_error                     */
    DIP_ERR_WORKSPACE = 4      /* problem larger than the context's scratch workspace allows         */
} dip_status;

typedef enum {
    DIP_W_F32 = 0,             /* binary32 weights                                                   */
    DIP_W_BF16 = 1,            /* bfloat16 weights                                                   */
    DIP_W_INT4_G128 = 2        /* 4-bit symmetric codes, one binary16 scale per 128 input indices    */
} dip_wtype;

enum {
    DIP_MAX_D = 32768,         /* largest masked dimension (d_model or d_ff)                         */
    DIP_MAX_BATCH = 16,
    DIP_INT4_GROUP = 128,
    DIP_CACHE_META_INTS = 8    /* length of dip_cache_state.meta                                     */
};

typedef struct dip_ctx dip_ctx;   /* opaque; owns scratch workspace on one device */

/* Options of a context.  A zeroed struct gives the defaults; the library reads no
 * environment variable and has no other global switch.
 *   max_d, max_batch   size the workspace: the largest d_model / d_ff and the most tokens per
 *                      call that this context will see (0 = DIP_MAX_D / DIP_MAX_BATCH).  A call
 *                      beyond them returns DIP_ERR_WORKSPACE.
 *   gemv_segment_bytes 0 = chosen per launch; 512, 1024 or 2048 force the segment of a packed
 *                      row that one thread block of the copy-ring product kernel handles.
 *   gemv_copy_ring     non-zero: single-token F32 / BF16 products also go through the
 *                      copy-ring kernel (by default they use the plain-load kernel).
 *   coarse_min_d       smallest d_ff for which a step that runs a select kernel in front of the
 *                      down product (INT4 weights, several tokens, select_in_product < 0) ranks
 *                      h from the 16-bit keys that the gate/up product leaves behind: 0 = default
 *                      (4096), negative = every size.  Either way the masks are the same bits.
 *   wait_limit_us      bound of every in-kernel wait (on an asynchronous copy, on another thread
 *                      block's flag), in microseconds (0 = one second); see dip_device_status.
 *   select_in_product  0 = default: in a single-token step with F32 / BF16 weights each product
 *                      kernel builds the mask of its own input (every thread block finds the
 *                      columns that are certainly kept and streams them at once, one extra block
 *                      completes the mask meanwhile); negative: a select kernel runs in front of
 *                      each product instead.  The masks are the same bits either way; the
 *                      products add the same rows in a different order. */
typedef struct {
    int32_t max_d;
    int32_t max_batch;
    int32_t gemv_segment_bytes;
    int32_t gemv_copy_ring;
    int32_t coarse_min_d;
    int32_t wait_limit_us;
    int32_t select_in_product;
    int32_t reserved[3];          /* keep zero */
} dip_options;

/* Create a context on `device` (a CUDA ordinal).  Allocates the scratch
 * workspace (about 50 MB at the default sizes) with cudaMalloc; no other call
 * allocates.  *out is NULL on failure.  The calling thread's current device is
 * left as it was.  Every later call on the context must be made with `device`
 * current (DIP_ERR_INVALID_ARG otherwise). */
dip_status dip_create(dip_ctx **out, int device);
/* The same with options (NULL = defaults). */
dip_status dip_create_ex(dip_ctx **out, int device, const dip_options *options);
/* Frees the workspace.  The caller makes sure no work of this context is in flight. */
dip_status dip_destroy(dip_ctx *ctx);
/* Static description of a status code (host string, never NULL). */
const char *dip_status_string(dip_status s);
/* Text of the last CUDA failure seen by this context (host string owned by the
 * context; empty if none). */
const char *dip_last_error(const dip_ctx *ctx);
/* Number of streaming multiprocessors of the context's device. */
int dip_sm_count(const dip_ctx *ctx);
/* Every wait inside a kernel (on the arrival of an asynchronous copy) is bounded.  If one runs
 * out, the kernel stops early, its outputs are invalid and a sticky status word on the device
 * becomes non-zero.  This call waits for `stream`, then copies the word to *status_out (host). */
typedef enum {
    DIP_DEVICE_OK = 0,
    DIP_DEVICE_WAIT_TIMEOUT = 1,        /* a kernel gave up a bounded wait                          */
    DIP_DEVICE_TIER_INCONSISTENT = 2    /* two-tier step: slot table and cache state disagree       */
} dip_device_status_word;
dip_status dip_device_status(dip_ctx *ctx, int *status_out, void *stream);
/* Clears the sticky word (enqueued on `stream`). */
dip_status dip_reset_device_status(dip_ctx *ctx, void *stream);
/* Self-test of the bounded wait (diagnostics): enqueues one tiny kernel that waits, with the
 * given limit, for a copy that is never issued.  The wait runs out, the kernel returns, and the
 * status word becomes DIP_DEVICE_WAIT_TIMEOUT; nothing else is touched and the context stays
 * usable.  waited_ns (device uint64, may be NULL) receives how long the kernel waited.
 * 1 <= limit_us <= 1000000. */
dip_status dip_selftest_bounded_wait(dip_ctx *ctx, int limit_us, unsigned long long *waited_ns, void *stream);

/* ------------------------------------------------------------------------
 * Timeline of the library's own kernels (diagnostics; off by default).  Between
 * dip_trace_begin and dip_trace_end every kernel the context launches (up to
 * 1024 launches) gets a slot in which it stamps, with the device's nanosecond
 * timer: the first CTA's entry, the first return from the wait on the previous
 * kernel in the stream, the last CTA's exit and, for the GEMVs, the end of the
 * weight streaming.  A CUDA graph captured while tracing is on keeps its slots:
 * dip_trace_reset clears the stamps (not the slots) before a replay, and
 * dip_trace_read returns the records of the launches that ran since.  These
 * calls synchronise the device; the stamps cost one atomic per CTA.
 *   kind: 1 select (DIP), 2 select (cache-aware), 3 cache update, 4 gate/up GEMV,
 *         5 down GEMV, 6 slot assignment, 7 fetch, 8 hit/miss split, 10 install (two-tier
 *         step), 9 neuron-major product (Gate / Up pruning).
 * ------------------------------------------------------------------------ */
typedef struct {
    int32_t kind;
    int32_t reserved;
    uint64_t t_start_ns, t_ready_ns, t_end_ns, t_aux_ns;
} dip_trace_record;
dip_status dip_trace_begin(dip_ctx *ctx);
dip_status dip_trace_reset(dip_ctx *ctx);
dip_status dip_trace_read(dip_ctx *ctx, dip_trace_record *out /* host */, int max_records, int *n_out /* host */);
dip_status dip_trace_end(dip_ctx *ctx);

/* ------------------------------------------------------------------------
 * Weights.  The paper's unit of selection is a column W[:, i] of a matrix
 * W in R^{d_out x d_in} (Eq. 4, 7, 8), so the library stores each matrix
 * column-contiguous: row i of the packed array holds column i.  Gate and up
 * always share one mask (Eq. 7), so their columns are bundled in one packed row.
 *
 *   gate_up        [d_model][2 * d_ff] elements
 *   down           [d_ff][d_model]     elements
 * F32 / BF16: a gate_up row interleaves gate and up in chunks of C outputs (piece
 * 2c = gate outputs of chunk c, piece 2c+1 = up outputs of chunk c), C = 4 for
 * F32 and 8 for BF16 (16-byte pieces); a down row is the column as it is.
 * INT4: value = (code - 8) * scale.  A packed row is a sequence of chunks of 128
 * codes = 64 bytes = 16 little-endian 32-bit words.  Local element e of a chunk is
 * nibble (e >> 4) of word (e & 15) (nibble n = bits 4n .. 4n+3), and the words are
 * stored in the order 0, 8, 1, 9, ..., 7, 15.  Chunk c of a down row holds outputs
 * 128 c + e; chunk c of a gate_up row holds gate output 64 c + e for e < 64 and up
 * output 64 c + (e - 64) for e >= 64.  (In this order the eight bytes at offset 8 g
 * of a chunk are one thread's operand share of eight 16 x 16 tensor-core tiles.)
 *   gate_up_scales [d_model/128][2 * d_ff] binary16, chunk for chunk like a
 *                  gate_up row, local element e at position (e & 15) * 8 + (e >> 4)
 *   down_scales    [d_ff/128][d_model] binary16, likewise
 *
 * Requirements: d_model % 32 == 0, d_ff % 32 == 0 (all formats); INT4 also
 * needs d_model % 128 == 0 and d_ff % 128 == 0.
 * ------------------------------------------------------------------------ */
typedef struct {
    int32_t wtype;               /* dip_wtype */
    int32_t d_model;
    int32_t d_ff;
    int32_t reserved;
    const void *gate_up;
    const void *gate_up_scales;  /* NULL unless INT4 */
    const void *down;
    const void *down_scales;     /* NULL unless INT4 */
} dip_mlp_weights;

/* Bytes of a packed array: which = 0 gate_up, 1 down, 2 gate_up_scales,
 * 3 down_scales.  Returns 0 for scales of non-INT4 types and for invalid
 * arguments. */
size_t dip_packed_bytes(int wtype, int d_model, int d_ff, int which);

/* Repack canonical matrices (row-major [d_out][d_in]: Wg, Wu are
 * [d_ff][d_model], Wd is [d_model][d_ff]; INT4 codes two per byte along d_in
 * with the even index in the low nibble; INT4 scales Sg, Su [d_model/128][d_ff],
 * Sd [d_ff/128][d_model]) into the packed layout above.  `out` names
 * caller-allocated device buffers of dip_packed_bytes() bytes each.  A one-off
 * set-up step; values are copied bit for bit. */
dip_status dip_pack_weights(dip_ctx *ctx, int wtype, int d_model, int d_ff,
                            const void *Wg, const void *Wu, const void *Wd,
                            const void *Sg, const void *Su, const void *Sd,
                            const dip_mlp_weights *out, void *stream);

/* ------------------------------------------------------------------------
 * Column-cache state of ONE masked linear-layer input (Algorithm 1's c):
 * gate and up share one cache over the d_model input columns, down has one
 * over its d_ff input columns.  Eviction policy: LRU (Sec. 5.1: the column
 * whose last use lies farthest in the past is evicted).
 *
 *   stamp[i]  -1 if column i is not resident, else the update number at which
 *             it was last used while resident
 *   meta[0]   number of resident columns        meta[1]  updates so far
 *   meta[2..5] accumulated hits, misses, evictions, bypassed columns
 *   meta[6..7] reserved (kept zero)
 * A cold cache is stamp = -1 everywhere and meta = 0.  The state is updated
 * in place; saving and restoring it is a copy of the two buffers.
 *
 * One update with mask m (k ones): hits are counted against the state the
 * score used; columns of m are never evicted by the same update; the number
 * of evictions is max(0, misses - free slots), limited by the resident columns
 * outside m, taking the smallest (stamp, index) first; missed columns become
 * resident in ascending index while room remains, the rest are used without
 * being cached ("bypassed", the case of Sec. 6.3 where the active set exceeds
 * the cache).
 *
 * LFU (Sec. 5.1, the policy of the paper's experiments): count[i] is the number
 * of updates whose mask contained column i since the state was created (kept
 * whether or not the column is resident); victims are the smallest
 * (count, index) instead of the smallest (stamp, index); everything else is
 * the same.
 * ------------------------------------------------------------------------ */
typedef enum { DIP_CACHE_LRU = 0, DIP_CACHE_LFU = 1 } dip_cache_policy;

typedef struct {
    int32_t d;          /* number of columns (input dimension of the layer) */
    int32_t capacity;   /* cache size in columns, 0 <= capacity <= d        */
    int32_t *stamp;     /* device int32[d]                                  */
    int32_t *meta;      /* device int32[DIP_CACHE_META_INTS]                */
    int32_t *count;     /* LFU only: device int32[d] use counters, 0 when cold; NULL for LRU */
    int32_t policy;     /* dip_cache_policy                                 */
    int32_t reserved;
} dip_cache_state;

/* ------------------------------------------------------------------------
 * dip_mask_topk — per-token magnitude top-k (Sec. 3.1; the masks of Eq. 7-8).
 * For each of `batch` rows of x[batch][d]: keep the k columns of largest |x|.
 *   mask_bits [batch][ceil(d/32)] out (may be NULL)
 *   kept_idx  [batch][k]          out, ascending (may be NULL)
 * 1 <= k <= d <= DIP_MAX_D, 1 <= batch <= DIP_MAX_BATCH.
 * ------------------------------------------------------------------------ */
dip_status dip_mask_topk(dip_ctx *ctx, const float *x, int batch, int d, int k,
                         uint32_t *mask_bits, int32_t *kept_idx, void *stream);

/* ------------------------------------------------------------------------
 * dip_ca_mask — Algorithm 1 for one linear-layer input and one token:
 *     s = |x| (c + gamma (1 - c)) / ||x||_inf      (Eq. 10)
 *     m = topK(s, k);   c' = cache_update(c, m)    (LRU, see dip_cache_state)
 * The ranking uses the numerator of Eq. 10 evaluated as ONE binary32
 * round-to-nearest product |x_i| * (c_i ? 1 : gamma); the positive constant
 * 1/||x||_inf cannot change the order and is not applied.  gamma == 1 gives
 * the DIP mask while still tracking the cache.
 *   st        cache state, updated in place (required)
 *   mask_bits [ceil(d/32)] out (may be NULL);  kept_idx [k] out (may be NULL)
 * 1 <= k <= d <= DIP_MAX_D, gamma finite and >= 0, st->d == d.
 * ------------------------------------------------------------------------ */
dip_status dip_ca_mask(dip_ctx *ctx, const float *x, int d, int k, float gamma,
                       const dip_cache_state *st,
                       uint32_t *mask_bits, int32_t *kept_idx, void *stream);

/* ------------------------------------------------------------------------
 * dip_sparse_gemv_gate_up — h = (W~u x) * silu(W~g x) over the kept columns
 * (Eq. 2 inside Eq. 3 with the mask of Eq. 7), binary32 accumulation.
 *   x        [batch][d_model]
 *   kept_idx [n_kept] ascending columns to read.  batch == 1: the token's mask.
 *            batch > 1: the union of the tokens' masks, each row read once.
 *   mask_bits [batch][ceil(d_model/32)] per-token masks; token b uses column i
 *            only if its bit is set.  Required for batch > 1, where the rows read
 *            are the union of the masks.  For batch == 1 it may be NULL (the list
 *            is used), or given with kept_idx == NULL (the bit set is used and
 *            n_kept is an upper bound on its size).
 *   h        [batch][d_ff] out
 * 1 <= n_kept <= d_model.
 * ------------------------------------------------------------------------ */
dip_status dip_sparse_gemv_gate_up(dip_ctx *ctx, const dip_mlp_weights *w,
                                   const float *x, int batch,
                                   const int32_t *kept_idx, int n_kept,
                                   const uint32_t *mask_bits,
                                   float *h, void *stream);

/* ------------------------------------------------------------------------
 * dip_sparse_gemv_down — y = W~d h over the kept columns of W^d (Eq. 1 inside
 * Eq. 3 with the mask of Eq. 8).  Arguments as above with h [batch][d_ff] in,
 * y [batch][d_model] out, kept_idx over the d_ff columns, 1 <= n_kept <= d_ff.
 * ------------------------------------------------------------------------ */
dip_status dip_sparse_gemv_down(dip_ctx *ctx, const dip_mlp_weights *w,
                                const float *h, int batch,
                                const int32_t *kept_idx, int n_kept,
                                const uint32_t *mask_bits,
                                float *y, void *stream);

/* ------------------------------------------------------------------------
 * dip_select_gemv_gate_up / dip_select_gemv_down — a mask and its product in
 * ONE launch, for one token and F32 / BF16 weights: the two halves of
 * dip_mlp_step as that step itself runs them (Eq. 7 + Eq. 2 in Eq. 3, then
 * Eq. 8 + Eq. 1 in Eq. 3).  Every thread block of the product selects for
 * itself and goes straight on to its rows, so nothing waits for a select kernel.
 *   gate_up: x [d_model] in;  mask_x [ceil(d_model/32)] out;  h [d_ff] out.
 *   down:    h [d_ff] in;     mask_h [ceil(d_ff/32)] out;     y [d_model] out.
 *   cache    optional state of that input: the ranking of Algorithm 1 with
 *            gamma; the state is only READ (no cache_update here).  NULL: plain
 *            magnitude top-k, gamma ignored.
 * The paper names no such operation: it is a fusion of dip_mask_topk /
 * dip_ca_mask's ranking with dip_sparse_gemv_*, and gives their results (the
 * mask bit for bit, the product up to the order of the binary32 sums).
 * dip_select_gemv_down ranks h from 16-bit keys that dip_select_gemv_gate_up
 * left in the context: call it right after dip_select_gemv_gate_up on the same
 * context and stream, with that call's h, and pass the SAME cache_d and gamma to
 * both (gate_up needs them to form the keys; NULL there means NULL here).
 * DIP_ERR_UNSUPPORTED for INT4 weights, for shapes whose working set does not
 * fit a thread block's shared memory, and when the context was created with
 * select_in_product < 0.
 * ------------------------------------------------------------------------ */
dip_status dip_select_gemv_gate_up(dip_ctx *ctx, const dip_mlp_weights *w, const float *x,
                                   int k_x, float gamma, const dip_cache_state *cache_gu,
                                   const dip_cache_state *cache_d,
                                   uint32_t *mask_x, float *h, void *stream);
dip_status dip_select_gemv_down(dip_ctx *ctx, const dip_mlp_weights *w, const float *h,
                                int k_h, float gamma, const dip_cache_state *cache_d,
                                uint32_t *mask_h, float *y, void *stream);

/* Optional outputs of a step; any pointer may be NULL (the step then keeps the
 * intermediate in its own workspace). */
typedef struct {
    uint32_t *mask_x;   /* [batch][ceil(d_model/32)] */
    int32_t *idx_x;     /* [batch][k_x]              */
    float *h;           /* [batch][d_ff]             */
    uint32_t *mask_h;   /* [batch][ceil(d_ff/32)]    */
    int32_t *idx_h;     /* [batch][k_h]              */
    int32_t *union_counts; /* batch > 1: int32[2] = |union of m_x|, |union of m_h| */
} dip_step_outputs;

/* ------------------------------------------------------------------------
 * dip_mlp_step — the whole sparse MLP step of Eq. 3 / 7 / 8 for one block:
 * mask x, gate/up + silu*up, mask h, down.  h stays binary32 between the
 * halves.  cache_gu / cache_d NULL = DIP (|.| ranking, no cache); non-NULL =
 * DIP-CA (Algorithm 1) on that input, batch must then be 1.
 *   x [batch][d_model] in;  y [batch][d_model] out;  out may be NULL.
 * batch > 1 computes one mask per token and reads the union of the kept
 * columns once.
 * ------------------------------------------------------------------------ */
dip_status dip_mlp_step(dip_ctx *ctx, const dip_mlp_weights *w,
                        const float *x, int batch, int k_x, int k_h, float gamma,
                        const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                        float *y, const dip_step_outputs *out, void *stream);

/* ------------------------------------------------------------------------
 * Layer chaining for multi-layer workloads (not part of the paper's method):
 * x_next = (x + y) / rms(x + y), per row, binary32 out.  x, y, x_next are
 * [batch][d]; x_next may alias x.
 * ------------------------------------------------------------------------ */
dip_status dip_residual_rmsnorm(dip_ctx *ctx, const float *x, const float *y,
                                int batch, int d, float *x_next, void *stream);

/* ------------------------------------------------------------------------
 * dip_stack_step — one decode token (or batch) through n_layers blocks:
 * for each layer l: y = dip_mlp_step(layer l, x_l); x_{l+1} = residual_rmsnorm(x_l, y).
 *   layers    host array [n_layers] of weights (all with the same shapes)
 *   cache_gu, cache_d  host arrays [n_layers] or NULL (DIP)
 *   x_in  [batch][d_model] in;  x_out [batch][d_model] out = x_{n_layers}
 *   y_last [batch][d_model] out, the last layer's MLP output (may be NULL)
 * ------------------------------------------------------------------------ */
dip_status dip_stack_step(dip_ctx *ctx, int n_layers, const dip_mlp_weights *layers,
                          const float *x_in, int batch, int k_x, int k_h, float gamma,
                          const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                          float *x_out, float *y_last, void *stream);

/* dip_stack_step that also keeps every layer's intermediates (for checking a stack layer by
 * layer against Eq. 7-8 and Algorithm 1): the same kernels in the same order, writing into the
 * caller's arrays instead of the context's workspace.  All arrays are required, device memory,
 * 16-byte aligned:
 *   x      [n_layers][batch][d_model]   x_l, the input of layer l (x_0 = x_in)
 *   mask_x [n_layers][batch][d_model/32]
 *   h      [n_layers][batch][d_ff]
 *   mask_h [n_layers][batch][d_ff/32]
 *   y      [n_layers][batch][d_model]   the MLP output of layer l */
typedef struct {
    float *x;
    uint32_t *mask_x;
    float *h;
    uint32_t *mask_h;
    float *y;
} dip_stack_probe;
dip_status dip_stack_step_probed(dip_ctx *ctx, int n_layers, const dip_mlp_weights *layers,
                                 const float *x_in, int batch, int k_x, int k_h, float gamma,
                                 const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                                 float *x_out, const dip_stack_probe *probe, void *stream);

/* ------------------------------------------------------------------------
 * Gate pruning and Up pruning (Sec. 3.2, Eq. 5), the neuron-wise schedules the
 * paper compares DIP with: one of the two first-layer products is computed
 * densely and ranks the d_ff neurons, p = silu(W^g x) (Gate pruning) or
 * p = W^u x (Up pruning); only the k neurons of largest |p| (ties to the lower
 * index) are evaluated in the other first-layer matrix and in W^d:
 *   h_j = p_j * (W^u x)_j   resp.   p_j * silu((W^g x)_j)   for kept j, else 0
 *   y   = sum over kept j of W^d[:, j] h_j
 * A neuron is a ROW of W^g / W^u and a COLUMN of W^d, so the layout differs
 * from dip_mlp_weights: gate and up are the matrices' own row-major
 * [d_ff][d_model] arrays (row j = neuron j), down is [d_ff][d_model] with row
 * j = W^d[:, j] (the `down` array of dip_pack_weights).  F32 or BF16; INT4
 * returns DIP_ERR_UNSUPPORTED.  One token per call.
 *   x [d_model] in, y [d_model] out; optional outputs (device, may be NULL):
 *   p_out [d_ff] the ranking activation, mask_out [ceil(d_ff/32)], idx_out [k]
 *   ascending, h_out [d_ff].  p and h are binary32, sums binary32.
 * ------------------------------------------------------------------------ */
typedef struct {
    int32_t wtype;
    int32_t d_model;
    int32_t d_ff;
    int32_t reserved;
    const void *gate;
    const void *up;
    const void *down;
} dip_neuron_weights;
enum { DIP_PRUNE_BY_GATE = 0, DIP_PRUNE_BY_UP = 1 };
dip_status dip_mlp_step_neuron_pruned(dip_ctx *ctx, const dip_neuron_weights *w, int prune_by,
                                      const float *x, int k, float *y,
                                      float *p_out, uint32_t *mask_out, int32_t *idx_out, float *h_out,
                                      void *stream);

/* ------------------------------------------------------------------------
 * Two-tier execution (Sec. 5 and its diagram of a single linear layer; the
 * memory model of the evaluation in Sec. 6): the weights of a masked input
 * live in a large slow tier, the columns the cache holds live in a small fast
 * tier, a step reads the missing columns of its mask from the slow tier,
 * evicts what the policy names when the fast tier is full, and multiplies with
 * the fast tier's copy.  Here the fast tier is an arena in device memory and
 * the slow tier is any memory the device can read: pinned, mapped host memory
 * (reads cross the host link) or another device allocation.
 *
 * A dip_tier belongs to one dip_cache_state (same d, same capacity): the cache
 * state says WHICH columns are resident, the tier says WHERE.  All buffers are
 * the caller's.
 *   backing  slow tier: the d packed rows of the matrix ([d][row_bytes], the
 *            layout of dip_pack_weights: gate_up or down), device-accessible
 *   arena    fast tier, device: (capacity + staging) rows of row_bytes; rows
 *            0 .. capacity-1 are cache slots; the rest are staging rows: a
 *            step's misses land there (the j-th miss in ascending column order
 *            in row capacity + j) and are multiplied from there; those that the
 *            cache keeps are then moved into their slots
 *   slot     device int32[d]: cache slot of column i, -1 = not resident.  Must
 *            agree with the cache state: slot[i] >= 0 exactly where
 *            stamp[i] >= 0; start both cold (all -1)
 *   loc      device int32[d]: scratch; arena row of each column of the current mask
 *   fetch    device int32[4 + 2 * staging]: scratch; [0] = misses of the step,
 *            [1] = rows moved into slots, then the misses' columns, then the moves
 *   split    device uint32[2][ceil(d/32)]: scratch; the mask's hits and its misses
 *   counters device uint64[2], accumulated: rows fetched, bytes fetched
 * Which slot a new column gets is the library's choice (the lowest free slots,
 * in ascending column order); every choice gives the same products.
 * INT4: the scales stay whole in device memory (dip_mlp_weights.*_scales);
 * only the codes are tiered.
 * ------------------------------------------------------------------------ */
typedef struct {
    int32_t d;
    int32_t capacity;       /* cache slots = capacity of the matching dip_cache_state */
    int32_t staging;        /* rows after the slots; >= the largest k used with this tier */
    int32_t reserved;
    uint64_t row_bytes;     /* bytes of one packed row; a multiple of 16 */
    const void *backing;
    void *arena;
    int32_t *slot;
    int32_t *loc;
    int32_t *fetch;
    uint32_t *split;
    unsigned long long *counters;
} dip_tier;

/* ------------------------------------------------------------------------
 * dip_mlp_step_tiered — dip_mlp_step for one token with both masked inputs
 * cache-aware and their weights two-tiered.  Per input: mask (Algorithm 1's
 * ranking); the mask's hits are multiplied out of the arena at once while one
 * stream of the context copies its misses from the slow tier into the staging
 * rows and another keeps the books (cache update, slot assignment, the move of
 * the staged rows that the cache keeps into their slots); the misses' product
 * follows the copy and the two partial results are added (hits first).  The
 * book-keeping is joined into `stream` before the call's work ends.  w gives
 * the format and shapes (and the INT4 scales); w->gate_up and w->down are not
 * read and may be NULL.  Results equal dip_mlp_step's on the same cache states
 * up to the order of the binary32 sums.  k_x <= tier_gu->staging and
 * k_h <= tier_d->staging.  A slot table that disagrees with the cache state
 * (fewer free slots than columns to insert, a resident column the table does
 * not know) sets the sticky device status to 2 and installs nothing.
 * ------------------------------------------------------------------------ */
dip_status dip_mlp_step_tiered(dip_ctx *ctx, const dip_mlp_weights *w,
                               const dip_tier *tier_gu, const dip_tier *tier_d,
                               const float *x, int k_x, int k_h, float gamma,
                               const dip_cache_state *cache_gu, const dip_cache_state *cache_d,
                               float *y, const dip_step_outputs *out, void *stream);

/* ------------------------------------------------------------------------
 * dip_sparse_gemv_down_noalloc — the down product y = W~d h of
 * dip_sparse_gemv_down (batch 1, F32 or BF16 weights) for callers that are not
 * allowed to allocate device memory.  The paper has no counterpart of this
 * call; it exists for integration only.
 *
 * Who needs it: code that runs where cudaMalloc is off limits — inside a
 * framework that owns the whole memory pool and forbids foreign allocations,
 * in a latency-critical serving loop where an allocation (an implicit device
 * synchronisation) is not acceptable, or in a process that has handed all of
 * the device's free memory to its own allocator, so that creating a dip_ctx
 * (which allocates its workspace) would fail.  This call takes no context:
 * the split-row partial sums and arrival counters that the context-based call
 * keeps in its workspace live in a fixed array of about 4 MB inside the
 * library image instead.  Every GPU that loads the library holds that array
 * until the process exits, whether or not this call is used.
 *
 * It calls no cudaMalloc / cudaFree and no allocating library routine.  The
 * first call on a device looks up the array's device address and the device's
 * SM count (once per device, with that device current); make that first call
 * before any stream capture.  The device used is the calling thread's current
 * device; w, h, kept_idx and y must live there.
 *
 * Limits: d_model <= 16384 (DIP_ERR_WORKSPACE beyond it: the fixed array
 * cannot hold the partial sums), d_model % 32 == 0, 1 <= n_kept <= d_ff <=
 * DIP_MAX_D; INT4 weights return DIP_ERR_UNSUPPORTED.  Only w->wtype,
 * w->d_model, w->d_ff and w->down are read.  kept_idx lists each kept column
 * once (ascending, as dip_mask_topk writes it); an entry outside [0, d_ff) is
 * skipped, a repeated entry is counted as often as it appears.
 *
 * All calls on a device share the one array, which keeps the previous call's
 * contents (each call clears the counters it needs on `stream` first).  Two
 * calls that overlap on the GPU — different streams, or different host
 * threads without ordering — race on it and give wrong results: serialise them.
 * The result equals dip_sparse_gemv_down's up to the order of the binary32
 * sums (the split into row parts may differ).
 * ------------------------------------------------------------------------ */
dip_status dip_sparse_gemv_down_noalloc(const dip_mlp_weights *w, const float *h,
                                        const int32_t *kept_idx, int n_kept,
                                        float *y, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* DIP_H */
