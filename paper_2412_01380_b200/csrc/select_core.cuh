// The select that builds a top-k bit mask (Sec. 3.1, Eq. 7-8; the cache-aware ranking of Eq. 10), as
// device functions for CTAs of 1024 threads: the one-histogram select over the top 15 bits of the
// rank keys with an exact ranking inside the threshold's bin, the general radix select for heavy
// ties (also the cache update's victim search), and the residual scale of a chained layer.  Used by
// the stand-alone select kernels and by the product kernels that select for themselves.
#pragma once

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

template <bool CA>
__device__ __forceinline__ uint32_t rank_key(float v, int stamp, float gamma)
{
    float a = fabsf(v);
    if (CA) a = __fmul_rn(a, stamp >= 0 ? 1.0f : gamma);
    return __float_as_uint(a) & 0x7fffffffu;
}

constexpr int TK_COARSE_ITERS = DIP_MAX_D / 8 / TK_THREADS;    // 16-byte loads of 16-bit keys per thread at the largest d

// ---------------------------------------------------------------------------------------------
// The select in one histogram: the top 15 bits of the rank keys (8 exponent and 7 mantissa bits)
// have 32768 bins of 16 bits in 64 KB of shared memory.  One counting pass, one search for the bin
// of the k-th largest key, one classification pass: every column above that bin is kept, and the
// few dozen columns inside it are ranked exactly by their full keys (lower column first among
// equals).  Cheap enough for every CTA of a product kernel to run for itself.  More than
// TK_TIE_LIMIT columns in the bin (masses of equal keys): the caller falls back to general_select.
// ---------------------------------------------------------------------------------------------
constexpr int TK_FINE_WORDS = 1 << 14;      // two 16-bit counters per word; DIP_MAX_D < 65536 keys cannot overflow one
constexpr int TK_TIE_LIMIT = 256;

struct __align__(16) TkFine {
    unsigned int hist[TK_FINE_WORDS];
    uint32_t ckey[TK_TIE_LIMIT];
    uint16_t cand[TK_TIE_LIMIT];
    int n_cand;
};

__device__ __forceinline__ void fine_zero(TkFine &f)
{
    const int tid = threadIdx.x;
    uint4 *h4 = reinterpret_cast<uint4 *>(f.hist);
#pragma unroll
    for (int i = 0; i < TK_FINE_WORDS / 4 / TK_THREADS; ++i) h4[tid + i * TK_THREADS] = make_uint4(0u, 0u, 0u, 0u);
    if (tid == 0) f.n_cand = 0;
}

// Counter of bin c15: logical word w = c15 / 2 (low half: even bin) is stored at (w % 16) * 1024 + w / 16, so
// that the 16 words of thread t = w / 16 in fine_find are a conflict-free stride apart.
__device__ __forceinline__ void fine_count(TkFine &f, uint32_t c15)
{
    const uint32_t w = c15 >> 1;
    atomicAdd(&f.hist[((w & 15u) << 10) | (w >> 4)], (c15 & 1u) ? 0x10000u : 1u);
}

// The bin of the k-th largest key: s.bcast[0] = bin, [1] = rank of the wanted key inside it (from
// the top, 1-based), [2] = keys in the bin.  Thread t owns bins 32 t .. 32 t + 31.  All threads
// call it; the histogram must be complete and visible; ends with a barrier.
__device__ __forceinline__ void fine_find(const TkFine &f, TkShared &s, int k)
{
    static_assert(TK_FINE_WORDS == 16 * TK_THREADS, "sixteen words per thread");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t wv[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) wv[i] = f.hist[(i << 10) | tid];
    int own = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) own += (int)(wv[i] & 0xffffu) + (int)(wv[i] >> 16);
    int suf = own;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += n;
    }
    if (lane == 0) s.wa[warp] = suf;
    __syncthreads();
    int wsum = s.wa[lane], wsuf = wsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_down_sync(0xffffffffu, wsuf, o);
        if (lane + o < 32) wsuf += n;
    }
    const int cum = __shfl_sync(0xffffffffu, wsuf - wsum, warp) + suf - own;     // keys in bins above this thread's
    // the owner of the k-th key's bins hands them to its warp: a lane per bin
    const unsigned owner = __ballot_sync(0xffffffffu, cum < k && k <= cum + own);
    if (owner) {
        const int ol = __ffs(owner) - 1;
        const int ot = (tid & ~31) | ol;
        const int ocum = __shfl_sync(0xffffffffu, cum, ol);
        const uint32_t wl = f.hist[((lane >> 1) << 10) | ot];
        const int cnt = (lane & 1) ? (int)(wl >> 16) : (int)(wl & 0xffffu);
        int bsuf = cnt;                          // inclusive suffix over the 32 bins, top bin = lane 31
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_down_sync(0xffffffffu, bsuf, o);
            if (lane + o < 32) bsuf += n;
        }
        const int above = ocum + bsuf - cnt;
        if (above < k && k <= above + cnt) {
            s.bcast[0] = 32 * ot + lane;
            s.bcast[1] = k - above;
            s.bcast[2] = cnt;
        }
    }
    __syncthreads();
}

// The n_c <= TK_TIE_LIMIT columns in f.cand[] (any order) are ranked by (full key descending, column
// ascending) and the first krem join maskw.  key_of(col) yields a column's full rank key.  All
// threads call it; f.cand complete and visible; ends with a barrier.
template <typename KeyOf>
__device__ __forceinline__ void fine_complete(TkFine &f, int n_c, int krem, unsigned int *maskw, KeyOf key_of)
{
    const int tid = threadIdx.x;
    uint32_t my = 0u;
    int mc = 0;
    if (tid < n_c) {
        mc = f.cand[tid];
        my = key_of(mc);
        f.ckey[tid] = my;
    }
    __syncthreads();
    if (tid < n_c) {
        int rank = 0;
        for (int j = 0; j < n_c; ++j) {
            const uint32_t kj = f.ckey[j];
            const int cj = f.cand[j];
            rank += (kj > my) || (kj == my && cj < mc);
        }
        if (rank < krem) atomicOr(&maskw[mc >> 5], 1u << (mc & 31));
    }
    __syncthreads();
}

// Second part of select_fine: keys[] and the histogram are complete (not yet synchronised).
__device__ __forceinline__ void select_fine_tail(const uint32_t *keys, int d, int k, TkShared &s, TkFine &f,
                                                 unsigned int *maskw)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    fine_find(f, s, k);
    const uint32_t b = (uint32_t)s.bcast[0];
    const int krem = s.bcast[1], n_c = s.bcast[2];
    if (n_c > TK_TIE_LIMIT) {
        general_select(keys, d, k, s, maskw);
        __syncthreads();
        return;
    }
    // columns above the bin into the mask (a lane's four flags are a nibble, eight neighbouring
    // lanes make a word), the bin's columns into the candidate list
    {
        const int n4 = (d + 3) >> 2;
        const int sh = (lane & 7) * 4;
        for (int q0 = warp * 32; q0 < n4; q0 += TK_THREADS) {
            const int q = q0 + lane;
            uint4 kk = make_uint4(0u, 0u, 0u, 0u);
            unsigned live = 0u;
            if (q < n4) {
                kk = *reinterpret_cast<const uint4 *>(keys + 4 * q);
                live = 4 * q + 4 <= d ? 0xfu : (1u << (d - 4 * q)) - 1u;
            }
            const uint32_t d0 = kk.x >> 16, d1 = kk.y >> 16, d2 = kk.z >> 16, d3 = kk.w >> 16;
            unsigned gt = (d0 > b ? 1u : 0u) | (d1 > b ? 2u : 0u) | (d2 > b ? 4u : 0u) | (d3 > b ? 8u : 0u);
            unsigned eq = ((d0 == b ? 1u : 0u) | (d1 == b ? 2u : 0u) | (d2 == b ? 4u : 0u) | (d3 == b ? 8u : 0u)) & live;
            while (eq) {
                const int t = __ffs(eq) - 1;
                eq &= eq - 1;
                f.cand[atomicAdd(&f.n_cand, 1)] = (uint16_t)(4 * q + t);
            }
            gt = (gt & live) << sh;
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) gt |= __shfl_xor_sync(0xffffffffu, gt, o);
            if ((lane & 7) == 0 && q < n4) maskw[q >> 3] = gt;
        }
    }
    __syncthreads();
    fine_complete(f, n_c, krem, maskw, [&](int col) { return keys[col]; });
}

// The whole select of one row from full rank keys.  On entry f is zero (and that is visible); with
// NORM, keys[] holds the bits of r = xa + xb and `scale` is 1 / rms(r), without NORM the row is
// xa.  The row's values go to x_out and / or x_keep when given, the rank keys to keys[], the mask
// (complete) to maskw[], all in shared memory except x_out.  Ends with a barrier.
template <bool CA, bool NORM>
__device__ __forceinline__ void select_fine(const float *__restrict__ xa, float *__restrict__ x_out, float *x_keep, int d,
                                            int k, float gamma, const int32_t *__restrict__ stamp, float scale,
                                            uint32_t *keys, TkShared &s, TkFine &f, unsigned int *maskw)
{
    const int tid = threadIdx.x;
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
                if (x_out) reinterpret_cast<float4 *>(x_out)[q] = v4[j];
                if (x_keep) reinterpret_cast<float4 *>(x_keep)[q] = v4[j];
                const float vv[4] = {v4[j].x, v4[j].y, v4[j].z, v4[j].w};
                const int sv[4] = {CA ? st4[j].x : 0, CA ? st4[j].y : 0, CA ? st4[j].z : 0, CA ? st4[j].w : 0};
                uint32_t kk[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    kk[t] = rank_key<CA>(vv[t], sv[t], gamma);
                    fine_count(f, kk[t] >> 16);
                }
                *reinterpret_cast<uint4 *>(keys + 4 * q) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
            }
        }
        }
    } else {
        for (int e = tid; e < d; e += TK_THREADS) {
            float v;
            if (NORM) v = __uint_as_float(keys[e]) * scale;
            else v = xa[e];
            if (x_out) x_out[e] = v;
            if (x_keep) x_keep[e] = v;
            const uint32_t key = rank_key<CA>(v, CA ? stamp[e] : 0, gamma);
            keys[e] = key;
            fine_count(f, key >> 16);
        }
    }
    select_fine_tail(keys, d, k, s, f, maskw);
}

// select_fine<CA, true> for d % 4 == 0, d <= 8 * TK_THREADS, with the residual scale folded in: xa, xb
// and the stamps are loaded together and stay in registers across the reduction, so the row costs
// one trip to memory instead of two.  Same summation order as block_residual_scale, same bits.
template <bool CA>
__device__ __forceinline__ void select_fine_chained(const float *__restrict__ xa, const float *__restrict__ xb,
                                                    float *__restrict__ x_out, float *x_keep, int d, int k, float gamma,
                                                    const int32_t *__restrict__ stamp, uint32_t *keys, TkShared &s,
                                                    TkFine &f, unsigned int *maskw)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n4 = d >> 2;
    float4 r[2];
    int4 st[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int q = tid + j * TK_THREADS;
        r[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        st[j] = make_int4(0, 0, 0, 0);
        if (q < n4) {
            const float4 va = reinterpret_cast<const float4 *>(xa)[q], vb = reinterpret_cast<const float4 *>(xb)[q];
            if (CA) st[j] = reinterpret_cast<const int4 *>(stamp)[q];
            r[j] = make_float4(va.x + vb.x, va.y + vb.y, va.z + vb.z, va.w + vb.w);
        }
    }
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        if (tid + j * TK_THREADS < n4) {
            ss = fmaf(r[j].x, r[j].x, ss);
            ss = fmaf(r[j].y, r[j].y, ss);
            ss = fmaf(r[j].z, r[j].z, ss);
            ss = fmaf(r[j].w, r[j].w, ss);
        }
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
            const float rms = sqrtf(v / (float)d);
            s.scale = rms > 0.f ? 1.0f / rms : 1.0f;
        }
    }
    __syncthreads();
    const float scale = s.scale;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int q = tid + j * TK_THREADS;
        if (q < n4) {
            const float4 v4 = make_float4(r[j].x * scale, r[j].y * scale, r[j].z * scale, r[j].w * scale);
            if (x_out) reinterpret_cast<float4 *>(x_out)[q] = v4;
            if (x_keep) reinterpret_cast<float4 *>(x_keep)[q] = v4;
            const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
            const int sv[4] = {st[j].x, st[j].y, st[j].z, st[j].w};
            uint32_t kk[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                kk[t] = rank_key<CA>(vv[t], sv[t], gamma);
                fine_count(f, kk[t] >> 16);
            }
            *reinterpret_cast<uint4 *>(keys + 4 * q) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
        }
    }
    select_fine_tail(keys, d, k, s, f, maskw);
}

// The whole select of one row whose producer left the top 16 bits of every rank key in coarse[]
// (d % 8 == 0, d <= 8 * TK_COARSE_ITERS * TK_THREADS); x and stamp supply the full keys of the
// threshold bin's columns.  On entry f is zero and visible.  The mask (complete) goes to maskw[];
// keys[] (d words) is scratch for the fallback under heavy ties.  Ends with a barrier.
template <bool CA>
__device__ __forceinline__ void select_fine_coarse(const uint16_t *__restrict__ coarse, const float *__restrict__ x,
                                                   const int32_t *__restrict__ stamp, float gamma, int d, int k,
                                                   uint32_t *keys, TkShared &s, TkFine &f, unsigned int *maskw)
{
    const int tid = threadIdx.x, lane = tid & 31;
    const int n8 = d >> 3;
    uint4 ck[TK_COARSE_ITERS];
#pragma unroll
    for (int j = 0; j < TK_COARSE_ITERS; ++j) {
        const int q = tid + j * TK_THREADS;
        ck[j] = make_uint4(0u, 0u, 0u, 0u);
        if (q < n8) ck[j] = __ldcg(reinterpret_cast<const uint4 *>(coarse) + q);
    }
#pragma unroll
    for (int j = 0; j < TK_COARSE_ITERS; ++j) {
        if (tid + j * TK_THREADS < n8) {
            const uint32_t wv[4] = {ck[j].x, ck[j].y, ck[j].z, ck[j].w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                fine_count(f, wv[t] & 0xffffu);
                fine_count(f, wv[t] >> 16);
            }
        }
    }
    __syncthreads();
    fine_find(f, s, k);
    const uint32_t b = (uint32_t)s.bcast[0];
    const int krem = s.bcast[1], n_c = s.bcast[2];
    if (n_c > TK_TIE_LIMIT) {
        for (int e = tid; e < d; e += TK_THREADS) keys[e] = rank_key<CA>(x[e], CA ? stamp[e] : 0, gamma);
        __syncthreads();
        general_select(keys, d, k, s, maskw);
        __syncthreads();
        return;
    }
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
                    const uint32_t lo = wv[t] & 0xffffu, hi = wv[t] >> 16;
                    gt |= (lo > b ? 1u : 0u) << (2 * t) | (hi > b ? 2u : 0u) << (2 * t);
                    eq |= (lo == b ? 1u : 0u) << (2 * t) | (hi == b ? 2u : 0u) << (2 * t);
                }
                if (q >= n8) gt = eq = 0u;
                while (eq) {
                    const int t = __ffs(eq) - 1;
                    eq &= eq - 1;
                    f.cand[atomicAdd(&f.n_cand, 1)] = (uint16_t)(8 * q + t);
                }
                gt <<= sh;
                gt |= __shfl_xor_sync(0xffffffffu, gt, 1);
                gt |= __shfl_xor_sync(0xffffffffu, gt, 2);
                if ((lane & 3) == 0 && q < n8) maskw[q >> 2] = gt;
            }
        }
    }
    __syncthreads();
    fine_complete(f, n_c, krem, maskw,
                  [&](int col) { return rank_key<CA>(__ldcg(x + col), CA ? __ldcg(stamp + col) : 0, gamma); });
}

}  // namespace
