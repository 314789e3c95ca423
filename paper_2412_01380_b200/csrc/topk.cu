// Masking kernels: magnitude top-k (Sec. 3.1, Eq. 7-8), the cache-aware ranking of Eq. 10, the
// LRU column-cache update of Algorithm 1, index lists / unions from bit masks, and the residual
// + RMS re-normalisation that chains layers.
//
// The step's critical path only needs the mask, so the work is split in two kernels:
//   select_kernel        rank keys -> k-th largest key by radix select -> bit mask.  One CTA of
//                        1024 threads per row; the keys live in shared memory.
//   cache_update_kernel  hits, misses, LRU victims and the new stamps from (mask, state).  It
//                        does not feed the GEMVs and runs beside them on another stream.
// Everything here is integer work on bit patterns, so results are exact and unique (ties go
// to the lower column index).
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
    int n_cand2;
    uint32_t last_key[32];
    int last_idx[32];
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

// Find the histogram bin holding the krem-th largest key: suffix scan over the RADIX_BINS bins,
// two per thread.  Leaves bcast[0] = bin, bcast[1] = rank of the wanted key inside the bin
// (1-based, from the top), bcast[2] = keys in the bin.  All threads call it; ends with a barrier.
__device__ __forceinline__ void find_bin(TkShared &s, int krem)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
    int cum = above_warp + suf - own;         // keys in bins above 2t+1
    if (cum < krem && krem <= cum + (int)h1) {
        s.bcast[0] = 2 * tid + 1;
        s.bcast[1] = krem - cum;
        s.bcast[2] = (int)h1;
    }
    cum += (int)h1;
    if (cum < krem && krem <= cum + (int)h0) {
        s.bcast[0] = 2 * tid;
        s.bcast[1] = krem - cum;
        s.bcast[2] = (int)h0;
    }
    __syncthreads();
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
                                   TkShared &s, uint32_t &T, int &quota, int &n_eq)
{
    const int tid = threadIdx.x, lane = tid & 31;
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
        find_bin(s, krem);
        prefix |= (uint32_t)s.bcast[0] << shift;
        prefmask |= dmask << shift;
        krem = s.bcast[1];
        n_eq = s.bcast[2];        // after the last pass: the number of keys equal to T
        hi = shift;
    }
    T = prefix;
    quota = krem;
}


constexpr int TK_VEC_ITERS = DIP_MAX_D / 4 / TK_THREADS;   // float4 loads per thread at the largest d
constexpr int TK_VEC_BATCH = 5;                            // of which this many are in flight together

// scale = 1 / rms(xa + xb) over d elements, the same bits on every thread of the CTA.  The sums
// r = xa + xb are optionally parked in stash[] (as bit patterns).  Summation order: each thread
// adds its elements in index order (16-byte groups tid, tid + 1024, ... when d % 4 == 0, single
// elements otherwise), then a shuffle tree per warp, then one over the warps.  Both users of this
// function (the fused select and the stand-alone chaining kernel) therefore agree bit for bit.
__device__ float block_residual_scale(const float *__restrict__ xa, const float *__restrict__ xb, int d,
                                      uint32_t *stash, float *wf, float *scale_slot)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float ss = 0.f;
    if ((d & 3) == 0) {
        const float4 *a4 = reinterpret_cast<const float4 *>(xa), *b4 = reinterpret_cast<const float4 *>(xb);
        const int n4 = d >> 2;
        for (int j0 = 0; j0 < TK_VEC_ITERS && tid + j0 * TK_THREADS < n4; j0 += TK_VEC_BATCH) {
        float4 va[TK_VEC_BATCH], vb[TK_VEC_BATCH];
#pragma unroll
        for (int j = 0; j < TK_VEC_BATCH; ++j) {
            const int q = tid + (j0 + j) * TK_THREADS;
            if (q < n4) {
                va[j] = a4[q];
                vb[j] = b4[q];
            }
        }
#pragma unroll
        for (int j = 0; j < TK_VEC_BATCH; ++j) {
            const int q = tid + (j0 + j) * TK_THREADS;
            if (q < n4) {
                const float r0 = va[j].x + vb[j].x, r1 = va[j].y + vb[j].y, r2 = va[j].z + vb[j].z, r3 = va[j].w + vb[j].w;
                if (stash)
                    *reinterpret_cast<uint4 *>(stash + 4 * q) =
                        make_uint4(__float_as_uint(r0), __float_as_uint(r1), __float_as_uint(r2), __float_as_uint(r3));
                ss = fmaf(r0, r0, ss);
                ss = fmaf(r1, r1, ss);
                ss = fmaf(r2, r2, ss);
                ss = fmaf(r3, r3, ss);
            }
        }
        }
    } else {
        for (int e = tid; e < d; e += TK_THREADS) {
            const float r = xa[e] + xb[e];
            if (stash) stash[e] = __float_as_uint(r);
            ss = fmaf(r, r, ss);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) wf[warp] = ss;
    __syncthreads();
    if (warp == 0) {
        float v = wf[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) {
            const float rms = sqrtf(v / (float)d);
            *scale_slot = rms > 0.f ? 1.0f / rms : 1.0f;
        }
    }
    __syncthreads();
    return *scale_slot;
}

// Second half of the fast path.  s_maskw holds the columns whose key lies in a bin above the
// threshold's, s_candw those in the threshold's bin (both in the mask's layout, complete and
// visible), keys[] the rank key of every candidate column at least, s.hist is zero.  The krem1
// largest candidates (lower column first among equals) complete the mask.  Returns false when
// more than 32 candidates share the threshold's top 22 bits; nothing has been written then.
__device__ bool refine_candidates(const uint32_t *keys, TkShared &s, unsigned int *s_maskw, const unsigned int *s_candw,
                                  int n_words, int krem1, uint32_t *__restrict__ mask_bits)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // second digit (bits 19..9) of the candidates; a thread walks the candidate bits of a word
    for (int w = tid; w < n_words; w += TK_THREADS) {
        unsigned u = s_candw[w];
        while (u) {
            const int col = w * 32 + __ffs(u) - 1;
            u &= u - 1;
            atomicAdd(&s.hist[(keys[col] & 0xfffffu) >> 9], 1u);
        }
    }
    __syncthreads();
    find_bin(s, krem1);
    const uint32_t b2 = (uint32_t)s.bcast[0];
    const int krem2 = s.bcast[1], cnt2 = s.bcast[2];
    if (cnt2 > 32) return false;
    for (int w = tid; w < n_words; w += TK_THREADS) {
        unsigned u = s_candw[w], keep = 0u;
        while (u) {
            const int bit = __ffs(u) - 1;
            u &= u - 1;
            const uint32_t low = keys[w * 32 + bit] & 0xfffffu;
            const uint32_t dg = low >> 9;
            if (dg > b2) {
                keep |= 1u << bit;
            } else if (dg == b2) {
                const int pos = atomicAdd(&s.n_cand2, 1);
                s.last_key[pos] = low & 0x1ffu;
                s.last_idx[pos] = w * 32 + bit;
            }
        }
        if (keep) s_maskw[w] |= keep;                  // the word is this thread's
    }
    __syncthreads();
    if (warp == 0) {
        // at most 32 keys share the threshold's top 22 bits: rank them by (key descending,
        // column ascending) and keep the first krem2
        const uint32_t kv = lane < cnt2 ? s.last_key[lane] : 0u;
        const int iv = lane < cnt2 ? s.last_idx[lane] : 0x7fffffff;
        int rank = 0;
        for (int j = 0; j < cnt2; ++j) {
            const uint32_t kj = __shfl_sync(0xffffffffu, kv, j);
            const int ij = __shfl_sync(0xffffffffu, iv, j);
            rank += (kj > kv) || (kj == kv && ij < iv);
        }
        if (lane < cnt2 && rank < krem2) atomicOr(&s_maskw[iv >> 5], 1u << (iv & 31));
    }
    __syncthreads();
    for (int w = tid; w < n_words; w += TK_THREADS) mask_bits[w] = s_maskw[w];
    return true;
}

// General path (very many keys tied around the threshold): full radix select on all d keys in
// keys[], then an ordered sweep that ranks the ties by column.
__device__ void general_select(const uint32_t *keys, int d, int k, TkShared &s, uint32_t *__restrict__ mask_bits)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // warp w owns columns [w*span, (w+1)*span), span a multiple of 32: one ballot = one mask word
    const int span = ((d + TK_THREADS - 1) / TK_THREADS) * 32;
    const int base = warp * span;
    uint32_t T;
    int quota, n_eq;
    block_radix_select(keys, d, 0x7fffffffu, 31, k, s, T, quota, n_eq);
    if (quota == n_eq) {
        // every column tied with the threshold is kept: the mask is key >= T
        for (int it = 0; it < span && base + it < d; it += 32) {
            const int e = base + it + lane;
            const unsigned bk = __ballot_sync(0xffffffffu, e < d && keys[e] >= T);
            if (lane == 0) mask_bits[(base + it) >> 5] = bk;
        }
        return;
    }
    // only the first `quota` tied columns (by index) are kept: rank the ties in order
    const unsigned lt = lanemask_lt();
    int eq = 0;
    for (int it = 0; it < span; it += 32) {
        const int e = base + it + lane;
        eq += __popc(__ballot_sync(0xffffffffu, e < d && keys[e] == T));
    }
    if (lane == 0) s.wb[warp] = eq;
    __syncthreads();
    int tot;
    int eq_before = warp_array_prefix(s.wb, warp, lane, tot);
    for (int it = 0; it < span && base + it < d; it += 32) {
        const int e = base + it + lane;
        const uint32_t key = e < d ? keys[e] : 0u;
        const bool q = e < d && key == T;
        const unsigned bq = __ballot_sync(0xffffffffu, q);
        const bool keep = (e < d && key > T) || (q && (eq_before + __popc(bq & lt)) < quota);
        const unsigned bk = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) mask_bits[(base + it) >> 5] = bk;
        eq_before += __popc(bq);
    }
}

// ---------------------------------------------------------------------------------------
// select_kernel: the mask of one row.
//   CA == false: key = bits(|x|)                              (DIP, Eq. 7-8)
//   CA == true : key = bits(|x| * (resident ? 1 : gamma))     (numerator of Eq. 10); the cache
//                state is only read.
//   NORM == true: the row is first formed as x = (xa + xb) / rms(xa + xb) (the layer chaining
//                of a stack) and written to x_out; the summation order is that of
//                residual_rmsnorm_kernel, so both give the same bits.
// keys[] is dynamic shared memory: d words rounded up to a multiple of four.
// ---------------------------------------------------------------------------------------
template <bool CA, bool NORM>
__global__ void __launch_bounds__(TK_THREADS, 1)
select_kernel(const float *__restrict__ xa, const float *__restrict__ xb, float *__restrict__ x_out,
              int d, int k, float gamma, const int32_t *__restrict__ stamp,
              uint32_t *__restrict__ mask_bits, unsigned long long *tr)
{
    DIP_TRACE_MIN(tr, 0);
    extern __shared__ uint32_t keys[];
    __shared__ TkShared s;
    __shared__ unsigned int s_maskw[DIP_MAX_D / 32];   // the mask being built
    __shared__ unsigned int s_candw[DIP_MAX_D / 32];   // columns whose key falls in the threshold's bin
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = blockIdx.x;
    const int n_words = (d + 31) >> 5;
    xa += (size_t)row * d;
    if (NORM) {
        xb += (size_t)row * d;
        x_out += (size_t)row * d;
    }
    mask_bits += (size_t)row * n_words;

    s.hist[2 * tid] = 0;
    s.hist[2 * tid + 1] = 0;
    if (tid == 0) {
        s.n_cand2 = 0;
    }
    dip_grid_dependency_wait();        // the inputs come from the previous kernel in the stream
    DIP_TRACE_MIN(tr, 1);
    dip_launch_dependents();

    float scale = 1.0f;
    if (NORM)
        scale = block_residual_scale(xa, xb, d, keys, s.wf, &s.scale);   // ends with a barrier
    else
        __syncthreads();                                                  // histogram zeroed
    // rank keys, and the histogram of their top 11 bits (first radix pass) in the same sweep
    if ((d & 3) == 0) {
        const int n4 = d >> 2;
        for (int j0 = 0; j0 < TK_VEC_ITERS && tid + j0 * TK_THREADS < n4; j0 += TK_VEC_BATCH) {
        float4 v4[TK_VEC_BATCH];
        int4 st4[TK_VEC_BATCH];
#pragma unroll
        for (int j = 0; j < TK_VEC_BATCH; ++j) {
            const int q = tid + (j0 + j) * TK_THREADS;
            if (q < n4) {
                if (NORM) {
                    const uint4 r = *reinterpret_cast<const uint4 *>(keys + 4 * q);
                    v4[j] = make_float4(__uint_as_float(r.x) * scale, __uint_as_float(r.y) * scale,
                                        __uint_as_float(r.z) * scale, __uint_as_float(r.w) * scale);
                } else {
                    v4[j] = reinterpret_cast<const float4 *>(xa)[q];
                }
                if (CA) st4[j] = reinterpret_cast<const int4 *>(stamp)[q];
            }
        }
#pragma unroll
        for (int j = 0; j < TK_VEC_BATCH; ++j) {
            const int q = tid + (j0 + j) * TK_THREADS;
            if (q < n4) {
                if (NORM) reinterpret_cast<float4 *>(x_out)[q] = v4[j];
                const float vv[4] = {v4[j].x, v4[j].y, v4[j].z, v4[j].w};
                const int sv[4] = {CA ? st4[j].x : 0, CA ? st4[j].y : 0, CA ? st4[j].z : 0, CA ? st4[j].w : 0};
                uint32_t kk[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    float a = fabsf(vv[t]);
                    if (CA) a = __fmul_rn(a, sv[t] >= 0 ? 1.0f : gamma);
                    kk[t] = __float_as_uint(a) & 0x7fffffffu;
                    atomicAdd(&s.hist[kk[t] >> 20], 1u);
                }
                *reinterpret_cast<uint4 *>(keys + 4 * q) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
            }
        }
        }
    } else {
        for (int e = tid; e < d; e += TK_THREADS) {
            float v;
            if (NORM) {
                v = __uint_as_float(keys[e]) * scale;
                x_out[e] = v;
            } else {
                v = xa[e];
            }
            float a = fabsf(v);
            if (CA) a = __fmul_rn(a, stamp[e] >= 0 ? 1.0f : gamma);
            const uint32_t key = __float_as_uint(a) & 0x7fffffffu;
            keys[e] = key;
            atomicAdd(&s.hist[key >> 20], 1u);
        }
    }
    __syncthreads();
    find_bin(s, k);
    const uint32_t b1 = (uint32_t)s.bcast[0];
    const int krem1 = s.bcast[1];

    // Every key in a bin above b1 is kept, every key below is dropped; the krem1 largest of the
    // keys in bin b1 (lower index first among equals) complete the mask.  One sweep, four keys
    // per lane, builds two bit sets in the mask's layout: the certain columns and the columns of
    // bin b1.  A lane's four flags are a nibble; eight neighbouring lanes OR theirs into a word.
    s.hist[2 * tid] = 0;          // free again: refilled below with the candidates' next digit
    s.hist[2 * tid + 1] = 0;
    {
        const int n4 = (d + 3) >> 2;
        const int sh = (lane & 7) * 4;
        for (int q0 = warp * 32; q0 < n4; q0 += TK_THREADS) {
            const int q = q0 + lane;
            uint4 kk = make_uint4(0u, 0u, 0u, 0u);
            unsigned live = 0u;                                // which of the four columns exist
            if (q < n4) {
                kk = *reinterpret_cast<const uint4 *>(keys + 4 * q);
                live = 4 * q + 4 <= d ? 0xfu : (1u << (d - 4 * q)) - 1u;
            }
            const uint32_t d0 = kk.x >> 20, d1 = kk.y >> 20, d2 = kk.z >> 20, d3 = kk.w >> 20;
            unsigned gt = (d0 > b1 ? 1u : 0u) | (d1 > b1 ? 2u : 0u) | (d2 > b1 ? 4u : 0u) | (d3 > b1 ? 8u : 0u);
            unsigned eq = (d0 == b1 ? 1u : 0u) | (d1 == b1 ? 2u : 0u) | (d2 == b1 ? 4u : 0u) | (d3 == b1 ? 8u : 0u);
            gt = (gt & live) << sh;
            eq = (eq & live) << sh;
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) {
                gt |= __shfl_xor_sync(0xffffffffu, gt, o);
                eq |= __shfl_xor_sync(0xffffffffu, eq, o);
            }
            if ((lane & 7) == 0 && q < n4) {
                s_maskw[q >> 3] = gt;
                s_candw[q >> 3] = eq;
            }
        }
    }
    __syncthreads();
    if (refine_candidates(keys, s, s_maskw, s_candw, n_words, krem1, mask_bits)) {
        DIP_TRACE_MAX(tr, 2);
        return;
    }
    general_select(keys, d, k, s, mask_bits);
    DIP_TRACE_MAX(tr, 2);
}

// ---------------------------------------------------------------------------------------
// select_coarse_kernel: the same mask as select_kernel<CA, false> for one row whose producer has
// already left the top 16 bits of every rank key in coarse[] (the gate/up GEMV does, in its
// epilogue).  One SM reads global memory at a fraction of the device's rate, so the bytes this CTA
// has to pull in are its floor: two bytes per column here instead of the eight of value + stamp.
// The first radix digit (top 11 bits) and the classification sweep work on the coarse keys, eight
// per lane, held in registers; the full key is formed only for the few hundred columns of the
// threshold's bin.  Needs d % 8 == 0 and d <= 8 * TK_COARSE_ITERS * TK_THREADS.
// ---------------------------------------------------------------------------------------
constexpr int TK_COARSE_ITERS = DIP_MAX_D / 8 / TK_THREADS;    // 16-byte loads per thread at the largest d

template <bool CA>
__device__ __forceinline__ uint32_t rank_key(float v, int stamp, float gamma)
{
    float a = fabsf(v);
    if (CA) a = __fmul_rn(a, stamp >= 0 ? 1.0f : gamma);
    return __float_as_uint(a) & 0x7fffffffu;
}

template <bool CA>
__global__ void __launch_bounds__(TK_THREADS, 1)
select_coarse_kernel(const float *__restrict__ x, const uint16_t *__restrict__ coarse, int d, int k, float gamma,
                     const int32_t *__restrict__ stamp, uint32_t *__restrict__ mask_bits, unsigned long long *tr)
{
    DIP_TRACE_MIN(tr, 0);
    extern __shared__ uint32_t keys[];
    __shared__ TkShared s;
    __shared__ unsigned int s_maskw[DIP_MAX_D / 32];
    __shared__ unsigned int s_candw[DIP_MAX_D / 32];
    const int tid = threadIdx.x, lane = tid & 31;
    const int n_words = d >> 5;
    const int n8 = d >> 3;

    s.hist[2 * tid] = 0;
    s.hist[2 * tid + 1] = 0;
    if (tid == 0) s.n_cand2 = 0;
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(tr, 1);
    dip_launch_dependents();

    // coarse keys to registers (all loads in flight together)
    uint4 ck[TK_COARSE_ITERS];
#pragma unroll
    for (int j = 0; j < TK_COARSE_ITERS; ++j) {
        const int q = tid + j * TK_THREADS;
        ck[j] = make_uint4(0u, 0u, 0u, 0u);
        if (q < n8) ck[j] = __ldcg(reinterpret_cast<const uint4 *>(coarse) + q);
    }
    __syncthreads();                                               // histogram zeroed
#pragma unroll
    for (int j = 0; j < TK_COARSE_ITERS; ++j) {
        if (tid + j * TK_THREADS < n8) {
            const uint32_t wv[4] = {ck[j].x, ck[j].y, ck[j].z, ck[j].w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                atomicAdd(&s.hist[(wv[t] & 0xffffu) >> 4], 1u);
                atomicAdd(&s.hist[wv[t] >> 20], 1u);
            }
        }
    }
    __syncthreads();
    find_bin(s, k);
    const uint32_t b1 = (uint32_t)s.bcast[0];
    const int krem1 = s.bcast[1];

    // classification: a lane's eight flags are a byte, four neighbouring lanes make a mask word
    s.hist[2 * tid] = 0;
    s.hist[2 * tid + 1] = 0;
    {
        const int sh = (lane & 3) * 8;
#pragma unroll
        for (int j = 0; j < TK_COARSE_ITERS; ++j) {
            const int q = tid + j * TK_THREADS;
            if ((tid & ~31) + j * TK_THREADS < n8) {                  // the whole warp or none of it
                const uint32_t wv[4] = {ck[j].x, ck[j].y, ck[j].z, ck[j].w};
                unsigned gt = 0u, eq = 0u;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const uint32_t lo = (wv[t] & 0xffffu) >> 4, hi = wv[t] >> 20;
                    gt |= (lo > b1 ? 1u : 0u) << (2 * t) | (hi > b1 ? 2u : 0u) << (2 * t);
                    eq |= (lo == b1 ? 1u : 0u) << (2 * t) | (hi == b1 ? 2u : 0u) << (2 * t);
                }
                if (q >= n8) gt = eq = 0u;
                gt <<= sh;
                eq <<= sh;
                gt |= __shfl_xor_sync(0xffffffffu, gt, 1);
                eq |= __shfl_xor_sync(0xffffffffu, eq, 1);
                gt |= __shfl_xor_sync(0xffffffffu, gt, 2);
                eq |= __shfl_xor_sync(0xffffffffu, eq, 2);
                if ((lane & 3) == 0 && q < n8) {
                    s_maskw[q >> 2] = gt;
                    s_candw[q >> 2] = eq;
                }
            }
        }
    }
    __syncthreads();
    // the full rank keys of the candidates (a word's candidates belong to one thread, here and in
    // the refinement)
    for (int w = tid; w < n_words; w += TK_THREADS) {
        unsigned u = s_candw[w];
        while (u) {
            // four columns at a time, their loads in flight together
            int col[4], sv[4];
            float xv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                col[i] = -1;
                if (u) {
                    col[i] = w * 32 + __ffs(u) - 1;
                    u &= u - 1;
                    xv[i] = __ldcg(x + col[i]);
                    sv[i] = CA ? __ldcg(stamp + col[i]) : 0;
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (col[i] >= 0) keys[col[i]] = rank_key<CA>(xv[i], sv[i], gamma);
        }
    }
    if (refine_candidates(keys, s, s_maskw, s_candw, n_words, krem1, mask_bits)) {
        DIP_TRACE_MAX(tr, 2);
        return;
    }
    // heavy ties: all keys in full, then the general path
    for (int e = tid; e < d; e += TK_THREADS) keys[e] = rank_key<CA>(x[e], CA ? stamp[e] : 0, gamma);
    __syncthreads();
    general_select(keys, d, k, s, mask_bits);
    DIP_TRACE_MAX(tr, 2);
}

// ---------------------------------------------------------------------------------------
// cache_update_kernel: c' = cache_update(c, m) of Algorithm 1 with the LRU policy of Sec. 5.1
// (or LFU when use counters are given), from the mask bits and the state alone.  One CTA; keys[] (dynamic shared memory, d words)
// holds (resident flag << 31) | eviction key, the eviction key being the age of the column's
// last use for columns that may be evicted (resident and outside the mask) and 0 otherwise.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(TK_THREADS, 1)
cache_update_kernel(const uint32_t *__restrict__ mask_bits, int d, int32_t *stamp, int32_t *count, int32_t *meta,
                    int capacity, unsigned long long *tr)
{
    DIP_TRACE_MIN(tr, 0);
    DIP_TRACE_MIN(tr, 1);
    extern __shared__ uint32_t keys[];
    __shared__ TkShared s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_res = meta[0];
    const int t_now = meta[1] + 1;
    const int span = ((d + TK_THREADS - 1) / TK_THREADS) * 32;
    const int base = warp * span;
    const unsigned lt = lanemask_lt();

    int hits = 0, misses = 0;
    constexpr int CU = 8;             // iterations whose loads are issued together
    for (int it0 = 0; it0 < span && base + it0 < d; it0 += 32 * CU) {
        unsigned mwv[CU];
        int stv[CU], cnv[CU];
#pragma unroll
        for (int u = 0; u < CU; ++u) {
            const int it = it0 + 32 * u, e = base + it + lane;
            const bool in_span = it < span && base + it < d;
            mwv[u] = in_span ? mask_bits[(base + it) >> 5] : 0u;
            stv[u] = in_span && e < d ? stamp[e] : -1;
            cnv[u] = count && in_span && e < d ? count[e] : 0;
        }
#pragma unroll
        for (int u = 0; u < CU; ++u) {
            const int it = it0 + 32 * u, e = base + it + lane;
            if (!(it < span && base + it < d)) break;          // uniform over the warp
            const bool valid = e < d;
            const unsigned mw = mwv[u];
            const bool keep = valid && ((mw >> lane) & 1u);
            const int st = stv[u];
            const bool res = st >= 0;
            // LRU: age of the last use.  LFU (count given): t + 1 - uses, so that the most rarely
            // used column has the largest key (a column is used at most once per update: uses <= t)
            uint32_t ek = 0u;
            if (res && !keep) ek = count ? (uint32_t)(t_now - cnv[u]) : (uint32_t)(t_now - st);
            if (valid) keys[e] = (res ? 0x80000000u : 0u) | ek;
            const int hw = __popc(__ballot_sync(0xffffffffu, keep && res));
            hits += hw;
            misses += __popc(mw) - hw;
        }
    }
    if (lane == 0) {
        s.wa[warp] = hits;
        s.wc[warp] = misses;
    }
    __syncthreads();
    int total_hits, total_misses, tot;
    (void)warp_array_prefix(s.wa, warp, lane, total_hits);
    int miss_before = warp_array_prefix(s.wc, warp, lane, total_misses);
    const int free_slots = capacity - n_res;
    const int evictable = n_res - total_hits;
    const int n_evict = min(max(0, total_misses - free_slots), evictable);
    const int room = free_slots + n_evict;
    __syncthreads();   // the warp arrays are reused by the select

    // victims: the n_evict largest eviction keys (oldest stamps), lower index first among equals
    uint32_t T2 = 0x7fffffffu;   // no key exceeds it: no victim
    int quota2 = 0, n_eq2 = 0;
    if (n_evict > 0) {
        if (n_evict == evictable)
            T2 = 0u;             // every evictable column (key > 0) goes
        else
            block_radix_select(keys, d, 0x7fffffffu, 32 - __clz(t_now), n_evict, s, T2, quota2, n_eq2);
    }
    // ordered rank of the eviction-key ties (needed only if some of them stay)
    int veq_before = 0;
    const bool ranked_ties = quota2 > 0 && quota2 < n_eq2;
    if (ranked_ties) {
        int veq = 0;
        for (int it = 0; it < span; it += 32) {
            const int e = base + it + lane;
            veq += __popc(__ballot_sync(0xffffffffu, e < d && (keys[e] & 0x7fffffffu) == T2));
        }
        if (lane == 0) s.wb[warp] = veq;
        __syncthreads();
        veq_before = warp_array_prefix(s.wb, warp, lane, tot);
    }
    const bool all_ties = quota2 > 0 && !ranked_ties;

    for (int it = 0; it < span && base + it < d; it += 32) {
        const int e = base + it + lane;
        const bool valid = e < d;
        const uint32_t kv = valid ? keys[e] : 0u;
        const uint32_t vkey = kv & 0x7fffffffu;
        const bool res = (kv >> 31) != 0u;
        const bool keep = valid && ((mask_bits[(base + it) >> 5] >> lane) & 1u);
        const bool vq = valid && vkey == T2 && vkey != 0u;
        bool evict = valid && vkey > T2;
        if (all_ties) evict = evict || vq;
        if (ranked_ties) {
            const unsigned bvq = __ballot_sync(0xffffffffu, vq);
            evict = evict || (vq && (veq_before + __popc(bvq & lt)) < quota2);
            veq_before += __popc(bvq);
        }
        const bool miss = keep && !res;
        const unsigned bm = __ballot_sync(0xffffffffu, miss);
        if (evict) {
            stamp[e] = -1;
        } else if (keep) {
            // a hit, or a miss that still finds room (ascending index order)
            if (!miss || (miss_before + __popc(bm & lt)) < room) stamp[e] = t_now;
        }
        if (count && keep) count[e] += 1;       // used once more (resident or not)
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
    DIP_TRACE_MAX(tr, 2);
}

// ---------------------------------------------------------------------------------------
// mask_to_idx_kernel: ascending index list of a bit mask, or of the union of `nb` masks
// (batched decode: the set of weight columns a step reads once).  CTA r handles masks
// r*nb .. r*nb+nb-1 and writes to idx_out + r*out_stride; thread t owns mask word t.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(TK_THREADS, 1)
mask_to_idx_kernel(const uint32_t *__restrict__ mask_bits, int nb, int d,
                   int32_t *__restrict__ idx_out, int out_stride, int32_t *__restrict__ count_out)
{
    __shared__ int wsum[TK_WARPS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_words = (d + 31) >> 5;
    mask_bits += (size_t)blockIdx.x * nb * n_words;
    uint32_t u = 0;
    if (tid < n_words)
        for (int b = 0; b < nb; ++b) u |= mask_bits[(size_t)b * n_words + tid];
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
    if (idx_out) {
        int32_t *o = idx_out + (size_t)blockIdx.x * out_stride;
        while (u) {
            int bit = __ffs(u) - 1;
            u &= u - 1;
            o[before++] = tid * 32 + bit;
        }
    }
    if (count_out && tid == 0) count_out[blockIdx.x] = total;
}

// ---------------------------------------------------------------------------------------
// residual_rmsnorm_kernel: x_next = (x + y) / rms(x + y), one CTA per row, fixed summation
// order (per-thread strided partial sums, then a shuffle tree).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(TK_THREADS, 1)
residual_rmsnorm_kernel(const float *x, const float *y, int d, float *x_next)
{
    __shared__ float wf[TK_WARPS];
    __shared__ float s_scale;
    const int tid = threadIdx.x;
    const size_t off = (size_t)blockIdx.x * d;
    dip_grid_dependency_wait();
    dip_launch_dependents();
    const float sc = block_residual_scale(x + off, y + off, d, nullptr, wf, &s_scale);
    for (int e = tid; e < d; e += TK_THREADS) x_next[off + e] = (x[off + e] + y[off + e]) * sc;
}

}  // namespace

// ---------------------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------------------
dip_status dip_launch_select(dip_ctx *ctx, const float *xa, const float *xb, float *x_out, int batch, int d, int k,
                             float gamma, const int32_t *stamp, uint32_t *mask_bits, cudaStream_t stream,
                             const uint16_t *coarse)
{
    const size_t smem = (size_t)((d + 3) & ~3) * sizeof(uint32_t);
    const dim3 grid(batch), block(TK_THREADS);
    unsigned long long *tr = dip_trace_slot(ctx, d <= 0 ? 0 : (stamp ? 2 : 1));
    cudaError_t e;
    if (coarse) {
        if (xb || batch != 1 || (d & 31)) return DIP_ERR_INVALID_ARG;
        if (stamp)
            e = dip_launch_pdl(select_coarse_kernel<true>, grid, block, smem, stream, xa, coarse, d, k, gamma, stamp,
                               mask_bits, tr);
        else
            e = dip_launch_pdl(select_coarse_kernel<false>, grid, block, smem, stream, xa, coarse, d, k, 1.0f,
                               (const int32_t *)nullptr, mask_bits, tr);
    } else if (xb) {
        if (stamp)
            e = dip_launch_pdl(select_kernel<true, true>, grid, block, smem, stream, xa, xb, x_out, d, k, gamma, stamp, mask_bits, tr);
        else
            e = dip_launch_pdl(select_kernel<false, true>, grid, block, smem, stream, xa, xb, x_out, d, k, 1.0f,
                               (const int32_t *)nullptr, mask_bits, tr);
    } else {
        if (stamp)
            e = dip_launch_pdl(select_kernel<true, false>, grid, block, smem, stream, xa, (const float *)nullptr,
                               (float *)nullptr, d, k, gamma, stamp, mask_bits, tr);
        else
            e = dip_launch_pdl(select_kernel<false, false>, grid, block, smem, stream, xa, (const float *)nullptr,
                               (float *)nullptr, d, k, 1.0f, (const int32_t *)nullptr, mask_bits, tr);
    }
    DIP_CUDA_TRY(ctx, e);
    return DIP_OK;
}

dip_status dip_launch_cache_update(dip_ctx *ctx, const uint32_t *mask_bits, int d, int32_t *stamp, int32_t *count,
                                   int32_t *meta, int capacity, cudaStream_t stream)
{
    cache_update_kernel<<<1, TK_THREADS, (size_t)d * sizeof(uint32_t), stream>>>(mask_bits, d, stamp, count, meta, capacity,
                                                                                   dip_trace_slot(ctx, 3));
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}

// Per-device set-up: the mask kernels keep up to DIP_MAX_D keys in dynamic shared memory.
dip_status dip_init_mask_kernels(dip_ctx *ctx)
{
    const int bytes = DIP_MAX_D * (int)sizeof(uint32_t);
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_coarse_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_coarse_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(cache_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    return DIP_OK;
}

// rows x (OR of nb masks) -> ascending index lists (and their lengths)
dip_status dip_launch_mask_to_idx(dip_ctx *ctx, const uint32_t *mask_bits, int rows, int nb, int d,
                                  int32_t *idx_out, int out_stride, int32_t *count_out, cudaStream_t stream)
{
    mask_to_idx_kernel<<<rows, TK_THREADS, 0, stream>>>(mask_bits, nb, d, idx_out, out_stride, count_out);
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}

dip_status dip_launch_residual_rmsnorm(dip_ctx *ctx, const float *x, const float *y, int batch, int d,
                                       float *x_next, cudaStream_t stream)
{
    DIP_CUDA_TRY(ctx, dip_launch_pdl(residual_rmsnorm_kernel, dim3(batch), dim3(TK_THREADS), 0, stream, x, y, d, x_next));
    return DIP_OK;
}
