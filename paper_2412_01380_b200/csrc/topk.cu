// Masking kernels: magnitude top-k (Sec. 3.1, Eq. 7-8), the cache-aware ranking of Eq. 10, the
// LRU column-cache update of Algorithm 1, index lists / unions from bit masks, and the residual
// + RMS re-normalisation that chains layers.
//
// The step's critical path only needs the mask, so the work is split in two kernels:
//   select_fine_kernel   rank keys -> k-th largest key by a histogram of their top 15 bits -> bit
//                        mask.  One CTA of 1024 threads per row; the keys live in shared memory.
//   cache_update_kernel  hits, misses, LRU victims and the new stamps from (mask, state).  It
//                        does not feed the GEMVs and runs beside them on another stream.
// Everything here is integer work on bit patterns, so results are exact and unique (ties go
// to the lower column index).
#include "select_core.cuh"

namespace {


// ---------------------------------------------------------------------------------------
// select_fine_kernel: the mask of one row by the one-histogram select of select_core.cuh (the
// select that the fused product kernels run), one CTA per row.
//   CA == false: key = bits(|x|)                              (DIP, Eq. 7-8)
//   CA == true : key = bits(|x| * (resident ? 1 : gamma))     (numerator of Eq. 10); the cache
//                state is only read.
//   NORM == true: the row is first formed as x = (xa + xb) / rms(xa + xb) (the layer chaining
//                of a stack) and written to x_out; the summation order is that of
//                residual_rmsnorm_kernel, so both give the same bits.
// select_fine_coarse_kernel: the same mask as select_fine_kernel<CA, false> for one row whose
// producer has already left the top 16 bits of every rank key in coarse[] (the gate/up product
// does, in its epilogue): one SM reads global memory at a fraction of the device's rate, so the
// bytes this CTA has to pull in are its floor: two bytes per column instead of the eight of value +
// stamp.  Needs d % 8 == 0 and d <= 8 * TK_COARSE_ITERS * TK_THREADS.
// Dynamic shared memory: TkFine, then keys[] (d words rounded up to four).
// ---------------------------------------------------------------------------------------
template <bool CA, bool NORM>
__global__ void __launch_bounds__(TK_THREADS, 1)
select_fine_kernel(const float *__restrict__ xa, const float *__restrict__ xb, float *__restrict__ x_out,
                   int d, int k, float gamma, const int32_t *__restrict__ stamp,
                   uint32_t *__restrict__ mask_bits, unsigned long long *tr)
{
    DIP_TRACE_MIN(tr, 0);
    extern __shared__ __align__(16) unsigned char dyn[];
    TkFine &f = *reinterpret_cast<TkFine *>(dyn);
    uint32_t *keys = reinterpret_cast<uint32_t *>(dyn + sizeof(TkFine));
    __shared__ TkShared s;
    __shared__ unsigned int s_maskw[DIP_MAX_D / 32];
    const int tid = threadIdx.x;
    const int row = blockIdx.x;
    const int n_words = (d + 31) >> 5;
    xa += (size_t)row * d;
    if (NORM) {
        xb += (size_t)row * d;
        x_out += (size_t)row * d;
    }
    mask_bits += (size_t)row * n_words;

    fine_zero(f);
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(tr, 1);
    dip_launch_dependents();
    if (NORM && (d & 3) == 0 && d <= 8 * TK_THREADS) {
        __syncthreads();                                              // histogram zeroed
        select_fine_chained<CA>(xa, xb, x_out, nullptr, d, k, gamma, stamp, keys, s, f, s_maskw);
    } else {
        float scale = 1.0f;
        if (NORM)
            scale = block_residual_scale(xa, xb, d, keys, s.wf, &s.scale);   // ends with a barrier
        else
            __syncthreads();
        select_fine<CA, NORM>(xa, NORM ? x_out : nullptr, nullptr, d, k, gamma, stamp, scale, keys, s, f, s_maskw);
    }
    for (int w = tid; w < n_words; w += TK_THREADS) mask_bits[w] = s_maskw[w];
    DIP_TRACE_MAX(tr, 2);
}

template <bool CA>
__global__ void __launch_bounds__(TK_THREADS, 1)
select_fine_coarse_kernel(const float *__restrict__ x, const uint16_t *__restrict__ coarse, int d, int k, float gamma,
                          const int32_t *__restrict__ stamp, uint32_t *__restrict__ mask_bits, unsigned long long *tr)
{
    DIP_TRACE_MIN(tr, 0);
    extern __shared__ __align__(16) unsigned char dyn[];
    TkFine &f = *reinterpret_cast<TkFine *>(dyn);
    uint32_t *keys = reinterpret_cast<uint32_t *>(dyn + sizeof(TkFine));
    __shared__ TkShared s;
    __shared__ unsigned int s_maskw[DIP_MAX_D / 32];
    const int tid = threadIdx.x;
    const int row = blockIdx.x;                                       // (several rows only without a cache)
    x += (size_t)row * d;
    coarse += (size_t)row * d;
    mask_bits += (size_t)row * (d >> 5);

    fine_zero(f);
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(tr, 1);
    dip_launch_dependents();
    __syncthreads();                                                  // histogram zeroed
    select_fine_coarse<CA>(coarse, x, stamp, gamma, d, k, keys, s, f, s_maskw);
    for (int w = tid; w < (d >> 5); w += TK_THREADS) mask_bits[w] = s_maskw[w];
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
    const size_t smem = sizeof(TkFine) + (size_t)((d + 3) & ~3) * sizeof(uint32_t);
    const dim3 grid(batch), block(TK_THREADS);
    unsigned long long *tr = dip_trace_slot(ctx, d <= 0 ? 0 : (stamp ? 2 : 1));
    cudaError_t e;
    if (coarse) {
        if (xb || (batch != 1 && stamp) || (d & 31)) return DIP_ERR_INVALID_ARG;
        if (stamp)
            e = dip_launch_pdl(select_fine_coarse_kernel<true>, grid, block, smem, stream, xa, coarse, d, k, gamma, stamp,
                               mask_bits, tr);
        else
            e = dip_launch_pdl(select_fine_coarse_kernel<false>, grid, block, smem, stream, xa, coarse, d, k, 1.0f,
                               (const int32_t *)nullptr, mask_bits, tr);
    } else if (xb) {
        if (stamp)
            e = dip_launch_pdl(select_fine_kernel<true, true>, grid, block, smem, stream, xa, xb, x_out, d, k, gamma, stamp, mask_bits, tr);
        else
            e = dip_launch_pdl(select_fine_kernel<false, true>, grid, block, smem, stream, xa, xb, x_out, d, k, 1.0f,
                               (const int32_t *)nullptr, mask_bits, tr);
    } else {
        if (stamp)
            e = dip_launch_pdl(select_fine_kernel<true, false>, grid, block, smem, stream, xa, (const float *)nullptr,
                               (float *)nullptr, d, k, gamma, stamp, mask_bits, tr);
        else
            e = dip_launch_pdl(select_fine_kernel<false, false>, grid, block, smem, stream, xa, (const float *)nullptr,
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
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(cache_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    const int fine_bytes = bytes + (int)sizeof(TkFine);
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_fine_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, fine_bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_fine_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, fine_bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_fine_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, fine_bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_fine_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, fine_bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_fine_coarse_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, fine_bytes));
    DIP_CUDA_TRY(ctx, cudaFuncSetAttribute(select_fine_coarse_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, fine_bytes));
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
