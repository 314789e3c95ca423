// Two-tier execution (Sec. 5: cached columns in a small fast memory, the rest read from a large
// slow one on a miss).  The cache state says which columns are resident; the kernels here keep
// the table of where they are (slots of an arena in device memory) and bring the missing ones in.
#include "common.cuh"

namespace {

constexpr int TA_THREADS = 1024;
constexpr int TA_WORDS = DIP_MAX_D / 32;

struct TierParams {
    int d, capacity, staging;
    unsigned long long row_bytes;
    const uint32_t *mask;      // [words] the step's mask
    const int32_t *stamp;      // [d] cache state AFTER the step's update (>= 0: resident)
    int32_t *slot;             // [d] in: slots before the update; out: after it
    int32_t *loc;              // [d] arena row of each kept column (not touched here)
    int32_t *fetch;            // [0] = misses fetched, [1] = out: rows to install, [4 ..) the misses' columns,
                               // [4 + staging ..) out: install list
    uint32_t *split;           // [0][words] hits, [1][words] misses (written by tier_split_kernel)
    unsigned long long *counters;
    int *status;
    unsigned long long *tr;
};

// Exclusive prefix sums of three per-thread counts over the block; totals to tot[0..2].
__device__ __forceinline__ void block_scan3(int (&v)[3], int (&pre)[3], int (*s_ws)[32], int *tot)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl[3];
#pragma unroll
    for (int c = 0; c < 3; ++c) {
        incl[c] = v[c];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, incl[c], o);
            if (lane >= o) incl[c] += n;
        }
        if (lane == 31) s_ws[c][warp] = incl[c];
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 3; ++c) {
        int before = 0, all = 0;
#pragma unroll
        for (int w = 0; w < TA_THREADS / 32; ++w) {
            const int x = s_ws[c][w];
            before += w < warp ? x : 0;
            all += x;
        }
        pre[c] = before + incl[c] - v[c];
        if (threadIdx.x == 0) tot[c] = all;
    }
    __syncthreads();
}

// Before the cache update: the columns of the mask that are resident (hits) can be multiplied
// right away, out of the slots they are in; the others (misses) have to be fetched first.
// One thread per column, one mask word per warp.
__global__ void __launch_bounds__(256)
tier_split_kernel(const uint32_t *__restrict__ mask, const int32_t *__restrict__ slot, int32_t *__restrict__ loc,
                  uint32_t *__restrict__ split, int d, unsigned long long *tr)
{
    DIP_TRACE_MIN(tr, 0);
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(tr, 1);
    dip_launch_dependents();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int words = (d + 31) / 32, w = i >> 5;
    if (w < words) {                                           // whole warps: d is a multiple of 32
        const uint32_t m = mask[w];
        const int sl = i < d ? slot[i] : -1;
        const bool hit = ((m >> (i & 31)) & 1u) && sl >= 0;
        if (hit) loc[i] = sl;
        const uint32_t hw = __ballot_sync(0xffffffffu, hit);
        if ((i & 31) == 0) {
            split[w] = hw;
            split[words + w] = m & ~hw;
        }
    }
    DIP_TRACE_MAX(tr, 2);
}

// One CTA, after the cache update, beside the products (nothing on the step's path waits for it).
// Compares the slot table (residency before the update) with the stamps (residency after it):
// evicted columns give up their slots, inserted columns take the lowest free slots in ascending
// column order.  Every miss of the step has been fetched into the staging row of its rank among
// the misses; the install list says which staging rows move into which slots.
__global__ void __launch_bounds__(TA_THREADS, 1)
tier_assign_kernel(const TierParams t)
{
    __shared__ uint32_t s_before[TA_WORDS], s_after[TA_WORDS], s_occ[TA_WORDS];
    __shared__ int s_ws[3][32];
    __shared__ int s_tot[3];
    __shared__ int s_bad;
    DIP_TRACE_MIN(t.tr, 0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int words = (t.d + 31) / 32;
    s_occ[tid] = 0u;
    if (tid == 0) s_bad = 0;
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(t.tr, 1);
    dip_launch_dependents();
    __syncthreads();

    constexpr int TU = 8;                  // iterations whose loads are issued together
    for (int base0 = warp * 32; base0 < t.d; base0 += TA_THREADS * TU) {
        int slv[TU], stv[TU];
#pragma unroll
        for (int u = 0; u < TU; ++u) {
            const int i = base0 + u * TA_THREADS + lane;
            slv[u] = i < t.d ? t.slot[i] : -1;
            stv[u] = i < t.d ? t.stamp[i] : -1;
        }
#pragma unroll
        for (int u = 0; u < TU; ++u) {
            const int base = base0 + u * TA_THREADS, i = base + lane;
            if (base >= t.d) break;                            // uniform over the warp
            const int sl = slv[u];
            const bool before = sl >= 0, after = stv[u] >= 0;
            const uint32_t bw = __ballot_sync(0xffffffffu, before), aw = __ballot_sync(0xffffffffu, after);
            if (lane == 0) {
                s_before[base >> 5] = bw;
                s_after[base >> 5] = aw;
            }
            if (before && after) {
                if (sl < t.capacity) atomicOr(&s_occ[sl >> 5], 1u << (sl & 31));
                else s_bad = 1;                                // a slot outside the arena
            }
            if (before && !after) t.slot[i] = -1;              // evicted
        }
    }
    __syncthreads();

    const int w = tid;
    uint32_t m = 0u, B = 0u, A = 0u, fr = 0u;
    if (w < words) {
        m = t.mask[w];
        B = s_before[w];
        A = s_after[w];
    }
    if (w * 32 < t.capacity) {
        fr = ~s_occ[w];
        if (t.capacity - w * 32 < 32) fr &= (1u << (t.capacity - w * 32)) - 1u;
    }
    const uint32_t ins = ~B & A;           // became resident in this step
    const uint32_t miss = m & ~B;          // kept and not resident before: fetched into staging
    if ((ins & ~miss) | (m & B & ~A)) s_bad = 1;   // only misses are inserted; the mask's hits stay
    int v[3] = {__popc(ins), __popc(miss), __popc(fr)}, pre[3];
    block_scan3(v, pre, s_ws, s_tot);
    const int n_ins = s_tot[0], n_miss = s_tot[1], n_free = s_tot[2];
    const bool bad = s_bad || n_ins > n_free || n_miss > t.staging;
    int32_t *inst = t.fetch + 4 + t.staging;                   // install list: (rank among the misses) << 16 | slot
    if (bad) {
        // the table and the cache state disagree: install nothing, say so
        if (tid == 0) {
            t.fetch[1] = 0;
            atomicExch(t.status, 2);
        }
        DIP_TRACE_MAX(t.tr, 2);
        return;
    }
    {
        // the j-th free slot (ascending) goes to the j-th inserted column (ascending)
        int f = pre[2];
        for (uint32_t u = fr; u && f < n_ins; u &= u - 1) inst[f++] = w * 32 + __ffs(u) - 1;
    }
    __syncthreads();
    {
        int r = pre[0];
        for (uint32_t u = ins; u; u &= u - 1, ++r) {
            const int bit = __ffs(u) - 1, col = w * 32 + bit;
            const int rank = pre[1] + __popc(miss & ((1u << bit) - 1u));   // the column's staging row
            const int sl = inst[r];
            t.slot[col] = sl;
            inst[r] = (rank << 16) | sl;
        }
    }
    if (tid == 0) {
        t.fetch[1] = n_ins;
        t.counters[0] += (unsigned long long)n_miss;
        t.counters[1] += (unsigned long long)n_miss * t.row_bytes;
    }
    DIP_TRACE_MAX(t.tr, 2);
}

constexpr int TF_THREADS = 512;
constexpr int TF_UNROLL = 4;
constexpr int TF_CHUNK = TF_THREADS * 16 * TF_UNROLL;     // bytes one CTA moves per turn

// Copies `n` rows src_row(e) -> dst_row(e) of row_bytes each: a grid-stride loop over
// (row, 32 KB chunk) units, 16 bytes per thread and four loads in flight per thread.  The grid
// leaves a few SMs without a CTA of this long-running kernel: the single-CTA book-keeping kernels
// beside it need a whole SM's registers.  Plain loads:
// the source may be host memory mapped into the device's address space.
//   INSTALL = false (fetch): row e of the miss list: slow tier row cols[e] -> staging row
//             capacity + e, and loc[cols[e]] = that row for the product over the misses;
//   INSTALL = true: entry e of the install list: staging row -> cache slot, inside the arena.
template <bool INSTALL>
__global__ void __launch_bounds__(TF_THREADS)
tier_copy_kernel(const char *__restrict__ backing, char *arena, const int32_t *__restrict__ fetch,
                 int32_t *__restrict__ loc, int capacity, int staging, unsigned long long row_bytes,
                 unsigned long long *tr)
{
    DIP_TRACE_MIN(tr, 0);
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(tr, 1);
    dip_launch_dependents();
    const int n = INSTALL ? fetch[1] : min(fetch[0], staging);
    const int32_t *list = fetch + 4 + (INSTALL ? staging : 0);
    const int cpr = (int)((row_bytes + TF_CHUNK - 1) / TF_CHUNK);
    const long long total = (long long)n * cpr;
    for (long long u = blockIdx.x; u < total; u += gridDim.x) {
        const int e = (int)(u / cpr), c = (int)(u % cpr);
        const int v = list[e];
        const size_t off = (size_t)c * TF_CHUNK;
        const int vecs = (int)(min((unsigned long long)TF_CHUNK, row_bytes - off) / 16);
        const char *src_row = INSTALL ? arena + (size_t)(capacity + (v >> 16)) * row_bytes : backing + (size_t)v * row_bytes;
        const int dst_row = INSTALL ? (v & 0xffff) : capacity + e;
        const uint4 *src = reinterpret_cast<const uint4 *>(src_row + off);
        uint4 *dst = reinterpret_cast<uint4 *>(arena + (size_t)dst_row * row_bytes + off);
        if (!INSTALL && c == 0 && threadIdx.x == 0) loc[v] = dst_row;
        uint4 q[TF_UNROLL];
#pragma unroll
        for (int j = 0; j < TF_UNROLL; ++j) {
            const int i = threadIdx.x + j * TF_THREADS;
            if (i < vecs) q[j] = __ldcs(src + i);
        }
#pragma unroll
        for (int j = 0; j < TF_UNROLL; ++j) {
            const int i = threadIdx.x + j * TF_THREADS;
            if (i < vecs) dst[i] = q[j];
        }
    }
    DIP_TRACE_MAX(tr, 2);
}

}  // namespace

dip_status dip_launch_tier_assign(dip_ctx *ctx, const dip_tier *t, const uint32_t *mask_bits, const int32_t *stamp,
                                  cudaStream_t stream)
{
    TierParams p;
    p.d = t->d;
    p.capacity = t->capacity;
    p.staging = t->staging;
    p.row_bytes = t->row_bytes;
    p.mask = mask_bits;
    p.stamp = stamp;
    p.slot = t->slot;
    p.loc = t->loc;
    p.fetch = t->fetch;
    p.split = t->split;
    p.counters = t->counters;
    p.status = ctx->status;
    p.tr = dip_trace_slot(ctx, 6);
    DIP_CUDA_TRY(ctx, dip_launch_pdl(tier_assign_kernel, dim3(1), dim3(TA_THREADS), 0, stream, p));
    return DIP_OK;
}

dip_status dip_launch_tier_split(dip_ctx *ctx, const dip_tier *t, const uint32_t *mask_bits, cudaStream_t stream)
{
    unsigned long long *tr = dip_trace_slot(ctx, 8);
    DIP_CUDA_TRY(ctx, dip_launch_pdl(tier_split_kernel, dim3((t->d + 255) / 256), dim3(256), 0, stream, mask_bits,
                                     (const int32_t *)t->slot, t->loc, t->split, (int)t->d, tr));
    return DIP_OK;
}

dip_status dip_launch_tier_fetch(dip_ctx *ctx, const dip_tier *t, cudaStream_t stream)
{
    unsigned long long *tr = dip_trace_slot(ctx, 7);
    const dim3 grid(ctx->sm_count > 16 ? ctx->sm_count - 8 : ctx->sm_count);
    DIP_CUDA_TRY(ctx, dip_launch_pdl(tier_copy_kernel<false>, grid, dim3(TF_THREADS), 0, stream,
                                     (const char *)t->backing, (char *)t->arena, (const int32_t *)t->fetch, t->loc,
                                     (int)t->capacity, (int)t->staging, (unsigned long long)t->row_bytes, tr));
    return DIP_OK;
}

dip_status dip_launch_tier_install(dip_ctx *ctx, const dip_tier *t, cudaStream_t stream)
{
    unsigned long long *tr = dip_trace_slot(ctx, 10);
    DIP_CUDA_TRY(ctx, dip_launch_pdl(tier_copy_kernel<true>, dim3(2 * ctx->sm_count), dim3(TF_THREADS), 0, stream,
                                     (const char *)t->backing, (char *)t->arena, (const int32_t *)t->fetch, t->loc,
                                     (int)t->capacity, (int)t->staging, (unsigned long long)t->row_bytes, tr));
    return DIP_OK;
}
