// Masking kernels: magnitude top-k (Sec. 3.1, Eq. 7-8), the cache-aware ranking of Eq. 10
// with the LRU column-cache update of Algorithm 1, the union of per-token masks for batched
// decode, and the residual + RMS re-normalisation that chains layers.
//
// One CTA of 1024 threads handles one input row.  The row's rank keys live in shared memory;
// the k-th largest key is found by an 11-bit-per-pass radix select, then one ordered sweep
// (warp ballots over 32 consecutive columns = one mask word) emits the bit mask and the
// ascending index list.  Everything here is integer work on bit patterns, so results are
// exact and unique (ties go to the lower column index).
#include "common.cuh"

namespace {

constexpr int TK_THREADS = 1024;
constexpr int TK_WARPS = TK_THREADS / 32;
constexpr int RADIX_BITS = 11;
constexpr int RADIX_BINS = 1 << RADIX_BITS;   // two bins per thread

struct TkShared {
    unsigned int hist[RADIX_BINS];
    int bcast[4];
    int wa[TK_WARPS];   // per-warp counts for ordered prefix sums
    int wb[TK_WARPS];
    int wc[TK_WARPS];
    float wf[TK_WARPS];
    float scale;
};

__device__ __forceinline__ unsigned lanemask_lt()
{
    unsigned m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// Exclusive prefix of a per-warp count array (TK_WARPS == 32 entries) for warp `warp`, plus the total.
__device__ __forceinline__ int warp_array_prefix(const int *arr, int warp, int lane, int &total)
{
    int v = arr[lane];
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    total = __shfl_sync(0xffffffffu, incl, 31);
    int excl = incl - v;
    return __shfl_sync(0xffffffffu, excl, warp);
}

// k-th largest of (keys[e] & keymask), e in [0, d).  All threads of the CTA take part and get
// the same answer: keep every key > T and the first `quota` columns (by index) with key == T.
// Requires 1 <= k <= d and every masked key < 2^top_bit.  A caller that wants to exclude a
// column gives it key 0 and makes sure k does not reach the zeros.
//
// Radix select from the top bit down, up to 11 bits per pass: a shared-memory histogram of the
// current digit over the keys that match the prefix found so far, then a suffix scan over the
// bins (two per thread) to find the bin holding the k-th key.  The four smallest digits, which
// are by far the most frequent ones when the keys are ages of cache lines, are counted in
// registers instead of with contended atomics.
__device__ void block_radix_select(const uint32_t *keys, int d, uint32_t keymask, int top_bit, int k,
                                   TkShared &s, uint32_t &T, int &quota)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t prefix = 0, prefmask = 0;
    int krem = k;
    int hi = top_bit;
    while (hi > 0) {
        const int w = hi < RADIX_BITS ? hi : RADIX_BITS;
        const int shift = hi - w;
        const uint32_t dmask = (1u << w) - 1u;
        s.hist[2 * tid] = 0;
        s.hist[2 * tid + 1] = 0;
        __syncthreads();
        int c0 = 0, c1 = 0, c2 = 0, c3 = 0;
        for (int e = tid; e < d; e += TK_THREADS) {
            const uint32_t key = keys[e] & keymask;
            if ((key & prefmask) == prefix) {
                const uint32_t dg = (key >> shift) & dmask;
                if (dg >= 4u) atomicAdd(&s.hist[dg], 1u);
                c0 += dg == 0u;
                c1 += dg == 1u;
                c2 += dg == 2u;
                c3 += dg == 3u;
            }
        }
        c0 = __reduce_add_sync(0xffffffffu, c0);
        c1 = __reduce_add_sync(0xffffffffu, c1);
        c2 = __reduce_add_sync(0xffffffffu, c2);
        c3 = __reduce_add_sync(0xffffffffu, c3);
        if (lane == 0) {
            if (c0) atomicAdd(&s.hist[0], (unsigned)c0);
            if (c1) atomicAdd(&s.hist[1], (unsigned)c1);
            if (c2) atomicAdd(&s.hist[2], (unsigned)c2);
            if (c3) atomicAdd(&s.hist[3], (unsigned)c3);
        }
        __syncthreads();
        // suffix scan: thread t owns bins 2t and 2t+1
        const unsigned h0 = s.hist[2 * tid], h1 = s.hist[2 * tid + 1];
        const int own = (int)(h0 + h1);
        int suf = own;   // inclusive suffix within the warp
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_down_sync(0xffffffffu, suf, o);
            if (lane + o < 32) suf += n;
        }
        if (lane == 0) s.wa[warp] = suf;
        __syncthreads();
        int wv = s.wa[lane];
        int wsuf = wv;   // inclusive suffix over warps
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_down_sync(0xffffffffu, wsuf, o);
            if (lane + o < 32) wsuf += n;
        }
        const int above_warp = __shfl_sync(0xffffffffu, wsuf - wv, warp);
        int cum = above_warp + suf - own;             // keys in bins above 2t+1
        if (cum < krem && krem <= cum + (int)h1) {
            s.bcast[0] = 2 * tid + 1;
            s.bcast[1] = krem - cum;
        }
        cum += (int)h1;
        if (cum < krem && krem <= cum + (int)h0) {
            s.bcast[0] = 2 * tid;
            s.bcast[1] = krem - cum;
        }
        __syncthreads();
        prefix |= (uint32_t)s.bcast[0] << shift;
        prefmask |= dmask << shift;
        krem = s.bcast[1];
        hi = shift;
    }
    T = prefix;
    quota = krem;
}

// ---------------------------------------------------------------------------------------
// mask_kernel: Algorithm 1 for one row.
//   CA == false: key = bits(|x|)                              (DIP, Eq. 7-8)
//   CA == true : key = bits(|x| * (resident ? 1 : gamma))     (numerator of Eq. 10), then the
//                LRU cache update c' = cache_update(c, m).
//   NORM == true: the row is first formed as x = (xa + xb) / rms(xa + xb) (the layer chaining
//                of a stack) and written to x_out; the summation order is that of
//                residual_rmsnorm_kernel, so both give the same bits.
// keys[] is dynamic shared memory: d words.
// ---------------------------------------------------------------------------------------
template <bool CA, bool NORM>
__global__ void __launch_bounds__(TK_THREADS, 1)
mask_kernel(const float *__restrict__ xa, const float *__restrict__ xb, float *__restrict__ x_out,
            int d, int k, float gamma, int32_t *stamp, int32_t *meta, int capacity,
            uint32_t *__restrict__ mask_bits, int32_t *__restrict__ kept_idx)
{
    extern __shared__ uint32_t keys[];
    __shared__ TkShared s;
    __shared__ unsigned int s_mask[DIP_MAX_D / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = blockIdx.x;
    const int n_words = (d + 31) >> 5;
    xa += (size_t)row * d;
    if (NORM) {
        xb += (size_t)row * d;
        x_out += (size_t)row * d;
    }
    if (mask_bits) mask_bits += (size_t)row * n_words;
    if (kept_idx) kept_idx += (size_t)row * k;

    int n_res = 0, t_now = 0;
    if (CA) {
        n_res = meta[0];
        t_now = meta[1] + 1;
    }

    if (NORM) {
        float ss = 0.f;
        for (int e = tid; e < d; e += TK_THREADS) {
            float r = xa[e] + xb[e];
            keys[e] = __float_as_uint(r);
            ss = fmaf(r, r, ss);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) s.wf[warp] = ss;
        __syncthreads();
        if (warp == 0) {
            float v = s.wf[lane];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) {
                float rms = sqrtf(v / (float)d);
                s.scale = rms > 0.f ? 1.0f / rms : 1.0f;
            }
        }
        __syncthreads();
    }
    for (int e = tid; e < d; e += TK_THREADS) {
        float v;
        if (NORM) {
            v = __uint_as_float(keys[e]) * s.scale;
            x_out[e] = v;
        } else {
            v = xa[e];
        }
        float a = fabsf(v);
        if (CA) a = __fmul_rn(a, stamp[e] >= 0 ? 1.0f : gamma);
        keys[e] = __float_as_uint(a) & 0x7fffffffu;
    }
    __syncthreads();

    uint32_t T;
    int quota;
    block_radix_select(keys, d, 0x7fffffffu, 31, k, s, T, quota);

    // ordered sweeps: warp w owns columns [w*span, (w+1)*span), span a multiple of 32
    const int span = ((d + TK_THREADS - 1) / TK_THREADS) * 32;
    const int base = warp * span;
    const unsigned lt = lanemask_lt();

    int gt = 0, eq = 0;
    for (int it = 0; it < span; it += 32) {
        int e = base + it + lane;
        uint32_t key = e < d ? keys[e] : 0u;
        bool valid = e < d;
        gt += __popc(__ballot_sync(0xffffffffu, valid && key > T));
        eq += __popc(__ballot_sync(0xffffffffu, valid && key == T));
    }
    if (lane == 0) {
        s.wa[warp] = gt;
        s.wb[warp] = eq;
    }
    __syncthreads();
    int tot;
    int gt_before = warp_array_prefix(s.wa, warp, lane, tot);
    int eq_before = warp_array_prefix(s.wb, warp, lane, tot);
    __syncthreads();   // wa/wb are reused below

    // second sweep: emit the mask and the index list; for CA also turn keys[] into
    // (resident flag << 31) | eviction key and count hits and misses
    int hits = 0, misses = 0;
    for (int it = 0; it < span; it += 32) {
        int e = base + it + lane;
        bool valid = e < d;
        uint32_t key = valid ? keys[e] : 0u;
        bool g = valid && key > T;
        bool q = valid && key == T;
        unsigned bg = __ballot_sync(0xffffffffu, g);
        unsigned bq = __ballot_sync(0xffffffffu, q);
        bool keep = g || (q && (eq_before + __popc(bq & lt)) < quota);
        unsigned bk = __ballot_sync(0xffffffffu, keep);
        if (base + it < d) {
            if (lane == 0) {
                if (CA) s_mask[(base + it) >> 5] = bk;
                if (mask_bits) mask_bits[(base + it) >> 5] = bk;
            }
            if (kept_idx && keep) {
                int pos = gt_before + min(eq_before, quota) + __popc(bk & lt);
                kept_idx[pos] = e;
            }
        }
        if (CA) {
            int st = valid ? stamp[e] : -1;
            bool res = st >= 0;
            // eviction key = age of the last use: an older column has a larger key; columns
            // that cannot be evicted (not resident, or in the current mask) get 0
            if (valid) keys[e] = (res ? 0x80000000u : 0u) | ((res && !keep) ? (uint32_t)(t_now - st) : 0u);
            hits += __popc(__ballot_sync(0xffffffffu, keep && res));
            misses += __popc(__ballot_sync(0xffffffffu, keep && !res));
        }
        gt_before += __popc(bg);
        eq_before += __popc(bq);
    }
    if (!CA) return;

    // ---------------- cache update (LRU, Sec. 5.1; Algorithm 1's cache_update) ----------------
    if (lane == 0) {
        s.wa[warp] = hits;
        s.wc[warp] = misses;
    }
    __syncthreads();
    int total_hits, total_misses;
    (void)warp_array_prefix(s.wa, warp, lane, total_hits);
    int miss_before = warp_array_prefix(s.wc, warp, lane, total_misses);
    const int free_slots = capacity - n_res;
    const int evictable = n_res - total_hits;
    const int n_evict = min(max(0, total_misses - free_slots), evictable);
    const int room = free_slots + n_evict;
    __syncthreads();   // the warp arrays are reused by the select

    // victims: the n_evict largest eviction keys (oldest stamps), lower index first among equals
    uint32_t T2 = 0x7fffffffu;   // no key exceeds it: no victim
    int quota2 = 0;
    if (n_evict > 0) {
        if (n_evict == evictable)
            T2 = 0u;             // every evictable column (key > 0) goes
        else
            block_radix_select(keys, d, 0x7fffffffu, 32 - __clz(t_now), n_evict, s, T2, quota2);
    }

    // ordered rank of the eviction-key ties
    int veq_before = 0;
    if (quota2 > 0) {
        int veq = 0;
        for (int it = 0; it < span; it += 32) {
            int e = base + it + lane;
            veq += __popc(__ballot_sync(0xffffffffu, e < d && (keys[e] & 0x7fffffffu) == T2));
        }
        if (lane == 0) s.wb[warp] = veq;
        __syncthreads();
        veq_before = warp_array_prefix(s.wb, warp, lane, tot);
    }

    for (int it = 0; it < span; it += 32) {
        int e = base + it + lane;
        bool valid = e < d;
        uint32_t kv = valid ? keys[e] : 0u;
        uint32_t vkey = kv & 0x7fffffffu;
        bool res = (kv >> 31) != 0u;
        bool keep = valid && ((s_mask[e >> 5] >> lane) & 1u);
        bool vq = valid && quota2 > 0 && vkey == T2;
        unsigned bvq = __ballot_sync(0xffffffffu, vq);
        bool evict = valid && (vkey > T2 || (vq && (veq_before + __popc(bvq & lt)) < quota2));
        bool miss = keep && !res;
        unsigned bm = __ballot_sync(0xffffffffu, miss);
        if (valid) {
            if (evict) {
                stamp[e] = -1;
            } else if (keep) {
                // a hit, or a miss that still finds room (ascending index order)
                if (!miss || (miss_before + __popc(bm & lt)) < room) stamp[e] = t_now;
            }
        }
        veq_before += __popc(bvq);
        miss_before += __popc(bm);
    }
    if (tid == 0) {
        const int inserted = min(total_misses, room);
        meta[0] = n_res - n_evict + inserted;
        meta[1] = t_now;
        meta[2] += total_hits;
        meta[3] += total_misses;
        meta[4] += n_evict;
        meta[5] += total_misses - inserted;
    }
}

// ---------------------------------------------------------------------------------------
// union_kernel: U = OR_b m_b as an ascending index list plus |U| (batched decode: the set of
// weight columns a step reads once).  One CTA; thread t owns mask word t.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(TK_THREADS, 1)
union_kernel(const uint32_t *__restrict__ mask_bits, int batch, int d,
             int32_t *__restrict__ union_idx, int32_t *__restrict__ union_count)
{
    __shared__ int wsum[TK_WARPS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_words = (d + 31) >> 5;
    uint32_t u = 0;
    if (tid < n_words)
        for (int b = 0; b < batch; ++b) u |= mask_bits[(size_t)b * n_words + tid];
    int c = __popc(u);
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    int total;
    int before = warp_array_prefix(wsum, warp, lane, total) + incl - c;
    while (u) {
        int bit = __ffs(u) - 1;
        u &= u - 1;
        union_idx[before++] = tid * 32 + bit;
    }
    if (tid == 0) *union_count = total;
}

// ---------------------------------------------------------------------------------------
// residual_rmsnorm_kernel: x_next = (x + y) / rms(x + y), one CTA per row, fixed summation
// order (per-thread strided partial sums, then a shuffle tree).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(TK_THREADS, 1)
residual_rmsnorm_kernel(const float *x, const float *__restrict__ y, int d, float *x_next)
{
    __shared__ float wsum[TK_WARPS];
    __shared__ float s_scale;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t off = (size_t)blockIdx.x * d;
    float ss = 0.f;
    for (int e = tid; e < d; e += TK_THREADS) {
        float r = x[off + e] + y[off + e];
        ss = fmaf(r, r, ss);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) wsum[warp] = ss;
    __syncthreads();
    if (warp == 0) {
        float v = wsum[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) {
            float rms = sqrtf(v / (float)d);
            s_scale = rms > 0.f ? 1.0f / rms : 1.0f;
        }
    }
    __syncthreads();
    const float sc = s_scale;
    for (int e = tid; e < d; e += TK_THREADS) x_next[off + e] = (x[off + e] + y[off + e]) * sc;
}

}  // namespace

// ---------------------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------------------
dip_status dip_launch_mask(dip_ctx *ctx, const float *x, int batch, int d, int k, float gamma,
                           int32_t *stamp, int32_t *meta, int capacity,
                           uint32_t *mask_bits, int32_t *kept_idx, cudaStream_t stream)
{
    const size_t smem = (size_t)d * sizeof(uint32_t);
    if (stamp)
        mask_kernel<true, false><<<batch, TK_THREADS, smem, stream>>>(x, nullptr, nullptr, d, k, gamma, stamp, meta,
                                                                      capacity, mask_bits, kept_idx);
    else
        mask_kernel<false, false><<<batch, TK_THREADS, smem, stream>>>(x, nullptr, nullptr, d, k, 1.0f, nullptr,
                                                                       nullptr, 0, mask_bits, kept_idx);
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}

// x_out = (xa + xb) / rms(xa + xb), then the mask of x_out: one launch for the layer chaining
// and the first mask of the next layer.
dip_status dip_launch_norm_mask(dip_ctx *ctx, const float *xa, const float *xb, float *x_out, int batch, int d,
                                int k, float gamma, int32_t *stamp, int32_t *meta, int capacity,
                                uint32_t *mask_bits, int32_t *kept_idx, cudaStream_t stream)
{
    const size_t smem = (size_t)d * sizeof(uint32_t);
    if (stamp)
        mask_kernel<true, true><<<batch, TK_THREADS, smem, stream>>>(xa, xb, x_out, d, k, gamma, stamp, meta,
                                                                     capacity, mask_bits, kept_idx);
    else
        mask_kernel<false, true><<<batch, TK_THREADS, smem, stream>>>(xa, xb, x_out, d, k, 1.0f, nullptr, nullptr,
                                                                      0, mask_bits, kept_idx);
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}

// Per-device set-up: the mask kernels keep up to DIP_MAX_D rank keys in dynamic shared memory.
dip_status dip_init_mask_kernels(dip_ctx *ctx)
{
    const int bytes = DIP_MAX_D * (int)sizeof(uint32_t);
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(mask_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(mask_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(mask_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(mask_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    return DIP_OK;
}

dip_status dip_launch_union(dip_ctx *ctx, const uint32_t *mask_bits, int batch, int d,
                            int32_t *union_idx, int32_t *union_count, cudaStream_t stream)
{
    union_kernel<<<1, TK_THREADS, 0, stream>>>(mask_bits, batch, d, union_idx, union_count);
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}

dip_status dip_launch_residual_rmsnorm(dip_ctx *ctx, const float *x, const float *y, int batch, int d,
                                       float *x_next, cudaStream_t stream)
{
    residual_rmsnorm_kernel<<<batch, TK_THREADS, 0, stream>>>(x, y, d, x_next);
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}
