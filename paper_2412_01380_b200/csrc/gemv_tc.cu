// Batched decode, 3 to 16 tokens, BF16 weights: the sparse product over the UNION of the tokens' kept
// columns (each row read once; token b uses a row only if its own mask keeps it) is a dense
// contraction D[tokens][outputs] += X^T[tokens][rows] W~[rows][outputs], and runs on the fifth-
// generation tensor cores:
//   * a CTA owns a 512-byte segment of the packed rows (256 outputs) and a part of the union's
//     rows; 16 warps stream the rows with 16-byte asynchronous copies (a whole segment per warp
//     instruction; rounds of 64 rows, three rounds in flight in a ring of four buffers) straight
//     into shared memory in the layout that a 128-byte-swizzled
//     MN-major operand descriptor names: the outputs of a row are contiguous, so the weights are the
//     B operand (N = 256) as they arrive, untransposed, and each byte is read by one MMA only;
//   * the tokens' values of the union's rows, zeroed where a token drops the row and split into two
//     bfloat16, are gathered ONCE per product by xt_build_kernel (16 scattered loads per row), 64
//     bytes per column of the union; the loaders copy them as the MN-major A operand: row n = the
//     high halves of token n, row 16 + n the low halves, the other rows of the M = 128 tile zero;
//   * one thread of a seventeenth warp issues one tcgen05.mma (M = 128, N = 256, K = 16) per 16 rows
//     once the loader warps have arrived on the buffer's "full" barrier; the accumulator lives in
//     tensor memory (256 columns) for the whole kernel, and a tcgen05.commit per round tells the
//     loaders through a second mbarrier when a buffer may be overwritten;
//   * the epilogue (one warp: the 32 useful accumulator rows are its 32 lanes) reads 16 columns at a
//     time with tcgen05.ld, adds the low-half row to the high-half row, and either applies
//     silu(gate) * up (a 16-column chunk is 8 gate outputs and their 8 up outputs; gate/up rows have
//     enough segments for one CTA to see all rows) or leaves the row part for combine_parts_kernel.
// All products are exact in binary32 (bf16 x bf16); sums are binary32 in the tensor core's order.
// Every wait on an mbarrier is bounded; on expiry the kernel records a status word, frees its
// tensor memory and leaves.
#include <cuda_bf16.h>

#include "common.cuh"
#include "gemv_common.cuh"

namespace {

constexpr int TC_LOAD_WARPS = 16;                // warps that stream rows; one more warp issues the MMAs
constexpr int TC_THREADS = (TC_LOAD_WARPS + 1) * 32;
constexpr int TC_U = 4;                          // rows per lane and round
constexpr int TC_ROUND_ROWS = TC_LOAD_WARPS * TC_U;   // 64 rows = 4 K-blocks of 16 per round
constexpr int TC_KB = TC_ROUND_ROWS / 16;
constexpr int TC_BUFS = 4;                       // ring of round buffers: three rounds of copies in flight
constexpr int TC_SEG = 512;                      // bytes of a packed row per CTA: 256 bf16 outputs = N
constexpr int TC_N = 16;                         // tokens
constexpr int TC_A_KB_BYTES = 16 * TC_SEG;       // one K-block of weights: [k group 2][output block 4][8 rows][128 B]
constexpr int TC_B_KB_BYTES = 128 * 16 * 2;      // one K-block of values: [row group 16][k group 2][8 rows][16 B]
constexpr int TC_TMEM_COLS = 256;                // one accumulator: 128 lanes x 256 binary32 columns

// Rows per in-kernel list: a list boundary drains the copy ring, so a part should be one list
// (16 tokens at keep ratio 0.25 keep ~5100 of 5120 gate/up rows, ~2500 down rows per part).
constexpr int TC_LIST_ROWS = 8192;

struct __align__(1024) TcSmem {
    unsigned char a[TC_BUFS][TC_KB * TC_A_KB_BYTES];   // weights, 4 x 32 KB
    unsigned char b[TC_BUFS][TC_KB * TC_B_KB_BYTES];   // token values, 4 x 16 KB
    uint64_t full[TC_BUFS];                      // the loader warps' copies into buffer i have landed
    uint64_t done[TC_BUFS];                      // the MMAs that read buffer i have completed
    uint32_t tmem_base;
    int n_total;
    int fail;
    int wsum[GV_SCAN_THREADS / 32];
    uint32_t words[DIP_MAX_D / 32];
    int pre[DIP_MAX_D / 32];
    uint16_t idx[TC_LIST_ROWS];
};

// Shared-memory operand descriptor: start address, leading / stride byte offsets (in 16-byte units),
// descriptor version 1, layout type (0 = no swizzle, 2 = 128-byte swizzle).
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout)
{
    return (uint64_t)((saddr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | ((uint64_t)layout << 61);
}

// Instruction descriptor of kind::f16: binary32 accumulate, bfloat16 A and B, A (token values)
// MN-major (token slots contiguous), B (weights) MN-major (outputs contiguous), N = 256, M = 128.
constexpr uint32_t TC_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(TC_IDESC), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 64 consecutive columns of this warp's 32 lanes of tensor memory: thread = lane, register = column
// (four 16-column loads in flight, one wait).
__device__ __forceinline__ void tc_ld64(uint32_t taddr, float (&v)[64])
{
    uint32_t r[64];
#pragma unroll
    for (int c = 0; c < 4; ++c)
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                     : "=r"(r[16 * c + 0]), "=r"(r[16 * c + 1]), "=r"(r[16 * c + 2]), "=r"(r[16 * c + 3]), "=r"(r[16 * c + 4]),
                       "=r"(r[16 * c + 5]), "=r"(r[16 * c + 6]), "=r"(r[16 * c + 7]), "=r"(r[16 * c + 8]), "=r"(r[16 * c + 9]),
                       "=r"(r[16 * c + 10]), "=r"(r[16 * c + 11]), "=r"(r[16 * c + 12]), "=r"(r[16 * c + 13]),
                       "=r"(r[16 * c + 14]), "=r"(r[16 * c + 15])
                     : "r"(taddr + 16 * c));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}

}  // namespace

namespace {

// The tokens' values of every column of the union, ready for the tensor core: xt[i][n] = bfloat16 high
// half of token n's value at column i (zero where the token's own mask drops the column or
// n >= batch), xt[i][16 + n] = the low half; columns outside the union are not written (and never
// read).  Built once per product instead of once per CTA (the values are 16 scattered 4-byte loads
// per column).  A block takes two mask words per pass; 16 consecutive threads are the 16 tokens of
// one column.
__global__ void __launch_bounds__(1024, 1)
xt_build_kernel(const uint32_t *__restrict__ mask_bits, const float *__restrict__ v, int batch, int d_in, int mask_words,
                uint16_t *__restrict__ xt)
{
    const int tid = threadIdx.x;
    const int n = tid & 15, bit = (tid >> 4) & 31, half = tid >> 9;
    dip_grid_dependency_wait();
    dip_launch_dependents();
    for (int w = 2 * blockIdx.x + half; w < mask_words; w += 2 * gridDim.x) {
        const int idx = w * 32 + bit;
        const bool mine = n < batch && idx < d_in && ((mask_bits[(size_t)n * mask_words + w] >> bit) & 1u);
        // in the union if any of the 16 tokens (a half-warp) keeps the column
        const unsigned any = __ballot_sync(0xffffffffu, mine) & (0xffffu << (tid & 16));
        if (!any) continue;
        const float x = mine ? __ldg(v + (size_t)n * d_in + idx) : 0.f;
        const __nv_bfloat16 hi = __float2bfloat16_rn(x);
        const __nv_bfloat16 lo = __float2bfloat16_rn(x - __bfloat162float(hi));
        xt[(size_t)idx * 32 + n] = __bfloat16_as_ushort(hi);
        xt[(size_t)idx * 32 + 16 + n] = __bfloat16_as_ushort(lo);
    }
}

template <int WHICH>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemv_tc_kernel(const GemvParams p, const uint16_t *__restrict__ xt)
{
    extern __shared__ unsigned char tc_smem_raw[];
    TcSmem &s = *reinterpret_cast<TcSmem *>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    DIP_TRACE_MIN(p.tr, 0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slab = blockIdx.x, part = blockIdx.y, nparts = gridDim.y;
    const size_t byte_off = (size_t)slab * TC_SEG + lane * 16;
    const bool lane_ok = byte_off < p.row_bytes;

    // ---- set-up: tensor memory for the two accumulator tiles, the buffers' barriers ----
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s.tmem_base)),
                     "n"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int i = 0; i < TC_BUFS; ++i) {
            mbar_init(&s.full[i], TC_LOAD_WARPS);
            mbar_init(&s.done[i], 1);
        }
        s.fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;
    dip_grid_dependency_wait();        // the masks and the vectors come from the previous kernels
    DIP_TRACE_MIN(p.tr, 1);
    dip_launch_dependents();

    // ---- 1. the union of the tokens' mask words and its popcount prefix ----
    if (tid < GV_SCAN_THREADS) {
        uint32_t u[4] = {0u, 0u, 0u, 0u};
        int c = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int w = 4 * tid + j;
            if (w < p.mask_words)
                for (int b = 0; b < p.batch; ++b) u[j] |= p.mask_bits[(size_t)b * p.mask_words + w];
            if (w == p.mask_words - 1 && (p.d_in & 31)) u[j] &= (1u << (p.d_in & 31)) - 1u;
            c += __popc(u[j]);
        }
        int incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += n;
        }
        if (lane == 31) s.wsum[warp] = incl;
        asm volatile("bar.sync 1, %0;" ::"n"(GV_SCAN_THREADS) : "memory");
        int before = 0;
#pragma unroll
        for (int w = 0; w < GV_SCAN_THREADS / 32; ++w) before += w < warp ? s.wsum[w] : 0;
        int pre = before + incl - c;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int w = 4 * tid + j;
            if (w < p.mask_words) {
                s.words[w] = u[j];
                s.pre[w] = pre;
            }
            pre += __popc(u[j]);
        }
        if (tid == GV_SCAN_THREADS - 1) s.n_total = pre;
    }
    __syncthreads();
    const int n_total = s.n_total;
    const int r_begin = (int)(((long long)part * n_total) / nparts);
    const int r_end = (int)(((long long)(part + 1) * n_total) / nparts);
    const char *base = p.W + byte_off;

    // this thread's places in a round: as a loader (warps 0-15), row slot k = warp of K-block u,
    // 16-byte chunk `lane` of the segment; as a builder of B, row tid / 4 and tokens 4 (tid % 4) .. + 3
    const uint32_t a_off = (uint32_t)(((warp & 15) >> 3) * 4096 + (lane >> 3) * 1024 + (warp & 7) * 128 + (((lane & 7) ^ (warp & 7)) << 4));
    // as a mover of the values: row tid / 4 of the round, 16-byte chunk tid % 4 of its 64 bytes in xt
    // (the high halves of tokens 0-7, 8-15, the low halves of tokens 0-7, 8-15) = A rows 8 (tid % 4) .. + 7
    // at that k: core matrices of 8 k x 16 bytes, the 16 row groups 128 B apart, the two k groups 2 KB apart
    const int bb_row = (tid >> 2) & (TC_ROUND_ROWS - 1), bb_mg = tid & 3;   // (threads 0 .. 4 TC_ROUND_ROWS - 1)
    const uint32_t b_off = (uint32_t)((bb_row >> 4) * TC_B_KB_BYTES + ((bb_row & 15) >> 3) * 2048 + bb_mg * 128 + (bb_row & 7) * 16);
    // the rows of the M = 128 tile that no token uses stay zero
    for (int i = tid; i < (int)(sizeof(s.b) / 16); i += TC_THREADS) reinterpret_cast<uint4 *>(&s.b[0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // (the block barriers below order them before any MMA)

    int g = 0;                         // rounds so far (buffer g & 1)
    bool failed = false;

    // The part's rows go through in lists of at most TC_LIST_ROWS (the in-kernel row list), a list in
    // rounds of TC_ROUND_ROWS.  Warps 0-15 load and store; warp 16 issues the MMAs.
    for (int list_begin = r_begin; list_begin < r_end; list_begin += TC_LIST_ROWS) {
        const int n_rows = min(r_end - list_begin, TC_LIST_ROWS);
        if (list_begin != r_begin) __syncthreads();               // everyone is done with the previous list
        {
            const int lo_rank = list_begin, hi_rank = list_begin + n_rows;
            for (int w = tid; w < p.mask_words; w += TC_THREADS) {
                uint32_t u = s.words[w];
                int rank = s.pre[w];
                if (rank >= hi_rank || rank + __popc(u) <= lo_rank) continue;
                while (u) {
                    const int bit = __ffs(u) - 1;
                    u &= u - 1;
                    if (rank >= lo_rank && rank < hi_rank) s.idx[rank - lo_rank] = (uint16_t)(w * 32 + bit);
                    ++rank;
                }
            }
        }
        __syncthreads();
        const int n_rounds = (n_rows + TC_ROUND_ROWS - 1) / TC_ROUND_ROWS;

        if (warp < TC_LOAD_WARPS) {
            // copies of one round, global -> shared memory, 16 bytes each (zero-filled past the end of the
            // list): this lane's piece of rows warp, warp + 16, ... and (threads 0-255) this thread's 16
            // bytes of the tokens' values of row tid / 4; one copy group per round
            auto copy_round = [&](int mr) {
                const int gr = g + mr;                                      // round number over the whole kernel
                if (mr < n_rounds) {
                    // the MMAs that read this ring slot four rounds ago must be through
                    if (gr >= TC_BUFS && !failed) {
                        if (s.fail || !mbar_wait(&s.done[gr % TC_BUFS], ((gr / TC_BUFS) - 1) & 1, p.wait_limit_ns)) failed = true;
                    }
                    const uint32_t ab = smem_u32(s.a[gr % TC_BUFS]) + a_off, bb = smem_u32(s.b[gr % TC_BUFS]) + b_off;
#pragma unroll
                    for (int u = 0; u < TC_U; ++u) {
                        const int r = mr * TC_ROUND_ROWS + warp + u * TC_LOAD_WARPS;
                        const bool ok = r < n_rows && lane_ok;
                        const char *src = ok ? base + (size_t)s.idx[r] * p.row_bytes : p.W;
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(ab + u * TC_A_KB_BYTES), "l"(src),
                                     "r"(ok ? 16 : 0) : "memory");
                    }
                    if (tid < TC_ROUND_ROWS * 4) {
                        const int r = mr * TC_ROUND_ROWS + bb_row;
                        const bool ok = r < n_rows;
                        const uint16_t *src = ok ? xt + (size_t)s.idx[r] * 32 + bb_mg * 8 : xt;
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(bb), "l"(src), "r"(ok ? 16 : 0) : "memory");
                    }
                }
                asm volatile("cp.async.commit_group;" ::: "memory");           // (an empty group past the last round)
            };
#pragma unroll
            for (int mr = 0; mr < TC_BUFS - 1; ++mr) copy_round(mr);
            for (int mr = 0; mr < n_rounds; ++mr) {
                const int gg = g + mr;
                // this thread's copies of round mr have landed (the two younger groups may be in flight)
                asm volatile("cp.async.wait_group %0;" ::"n"(TC_BUFS - 2) : "memory");
                // -> visible to the tensor core's (async proxy) reads
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(&s.full[gg % TC_BUFS]);
                copy_round(mr + TC_BUFS - 1);
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");              // (only empty groups are left)
        } else if (lane == 0) {
            // the MMA thread: per round, wait for the 16 loader warps, then two tiles x (hi, lo) per K-block
            for (int mr = 0; mr < n_rounds; ++mr) {
                const int gg = g + mr, buf = gg % TC_BUFS;
                if (failed) break;
                if (s.fail || !mbar_wait(&s.full[buf], (gg / TC_BUFS) & 1, p.wait_limit_ns)) {
                    failed = true;
                    break;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int rows_here = min(TC_ROUND_ROWS, n_rows - mr * TC_ROUND_ROWS);
                const int nkb = (rows_here + 15) >> 4;
                // descriptors of K-block 0; K-block kb is kb * bytes further (start address field in 16-byte units).
                // values: MN-major (token slots contiguous), no swizzle: 8-row groups 128 B apart, the two 8-k groups 2 KB apart;
                // weights: MN-major, 128-byte swizzle: 64-output blocks 1 KB apart, rows 0-7 / 8-15 4 KB apart
                const uint64_t x_d0 = tc_smem_desc(smem_u32(s.b[buf]), 2048, 128, 0);
                const uint64_t w_d0 = tc_smem_desc(smem_u32(s.a[buf]), 1024, 4096, 2);
                for (int kb = 0; kb < nkb; ++kb)
                    tc_mma(tmem, x_d0 + (uint64_t)(kb * (TC_B_KB_BYTES >> 4)), w_d0 + (uint64_t)(kb * (TC_A_KB_BYTES >> 4)),
                           (gg > 0 || kb > 0) ? 1u : 0u);
                tc_commit(&s.done[buf]);
            }
        }
        g += n_rounds;
    }
    DIP_TRACE_MAX(p.tr, 3);            // streaming done
    if (failed) s.fail = 1;
    __syncthreads();
    failed = s.fail != 0;

    // ---- the last round's commit covers every MMA of the kernel ----
    if (g > 0 && !failed) {
        if (!mbar_wait(&s.done[(g - 1) % TC_BUFS], ((g - 1) / TC_BUFS) & 1, p.wait_limit_ns)) failed = true;
    }
    if (failed && lane == 0) atomicExch(p.status, 1);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    // ---- epilogue: the useful accumulator rows 0-31 are tensor-memory lanes 0-31, which the warps 0, 4, 8
    //      and 12 reach (a warp reads the lane quarter warp % 4): token n's high-half sums in lane n, the
    //      low-half sums in lane 16 + n; 16 columns = 16 packed outputs at a time, four such chunks per warp ----
    if ((warp & 3) == 0 && warp < 16) {
        const int n = lane & 15, c0 = warp;                        // this warp's columns: 16 c0 .. 16 c0 + 63 (c0 = 0, 4, 8, 12)
        float v[64];
        if (g > 0 && !failed) {
            tc_ld64(tmem + 16 * c0, v);
        } else {
#pragma unroll
            for (int i = 0; i < 64; ++i) v[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < 64; ++i) v[i] += __shfl_down_sync(0xffffffffu, v[i], 16);       // + the low halves' sums
        if (lane < TC_N) {
            if (nparts > 1 || p.defer) {
                // row parts: [part][segment][token][256 packed elements], added up by combine_parts_kernel
                float *dst = p.partials + ((size_t)(p.part_base + part) * gridDim.x + slab) * (TC_N * 256) + n * 256 + 16 * c0;
#pragma unroll
                for (int i = 0; i < 64; i += 4)
                    *reinterpret_cast<float4 *>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
            } else if (n < p.batch) {
                if (WHICH == 0) {
                    // every 16 columns: 8 gate outputs followed by their 8 up outputs
                    const int j = slab * 128 + c0 * 8;
                    float *dst = p.out + (size_t)n * p.d_out + j;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float h[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) h[i] = silu_f32(v[16 * c + i]) * v[16 * c + 8 + i];
                        if (j + 8 * c + 8 <= p.d_out) {
                            *reinterpret_cast<float4 *>(dst + 8 * c) = make_float4(h[0], h[1], h[2], h[3]);
                            *reinterpret_cast<float4 *>(dst + 8 * c + 4) = make_float4(h[4], h[5], h[6], h[7]);
                            if (p.key_coarse) {
                                // top 16 bits of the rank keys |h_j| for the select that follows (no cache with several tokens)
                                uint32_t kk[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i)
                                    kk[i] = ((__float_as_uint(h[2 * i]) & 0x7fffffffu) >> 16) |
                                            ((__float_as_uint(h[2 * i + 1]) & 0x7fffffffu) & 0xffff0000u);
                                *reinterpret_cast<uint4 *>(p.key_coarse + (size_t)n * p.d_out + j + 8 * c) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                if (j + 8 * c + i < p.d_out) dst[8 * c + i] = h[i];
                        }
                    }
                } else {
                    const int j = slab * 256 + 16 * c0;
                    float *dst = p.out + (size_t)n * p.d_out + j;
#pragma unroll
                    for (int i = 0; i < 64; i += 4) {
                        if (j + i + 4 <= p.d_out) {
                            *reinterpret_cast<float4 *>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (j + i + e < p.d_out) dst[i + e] = v[i + e];
                        }
                    }
                }
            }
        }
    }
    // ---- free the tensor memory ----
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(TC_TMEM_COLS) : "memory");
    DIP_TRACE_MAX(p.tr, 2);
}

}  // namespace

// One CTA per 512-byte segment and row part; all resident at once.  Rows with at least as many
// segments as SMs' worth of work need no parts (gate/up); otherwise the parts are summed by
// combine_parts_kernel right after.
dip_status dip_launch_gemv_tc(dip_ctx *ctx, GemvParams &p, int which, int n_kept_max, cudaStream_t stream)
{
    const int n_slabs = (int)((p.row_bytes + TC_SEG - 1) / TC_SEG);
    int nparts = ctx->sm_count / n_slabs;
    if (nparts > n_kept_max / TC_ROUND_ROWS) nparts = n_kept_max / TC_ROUND_ROWS;   // at least a round of rows per part
    if (nparts < 1) nparts = 1;
    if (nparts > 1 && (size_t)nparts * n_slabs * TC_N * 256 > ctx->partials_floats) return DIP_ERR_WORKSPACE;
    p.defer = 0;
    p.part_base = 0;
    if (nparts > 1 || which != 0 || (p.d_out & 7)) p.key_coarse = nullptr;      // only the epilogue that sees whole sums forms the keys
    const size_t smem = sizeof(TcSmem) + 1024;
    static_assert(sizeof(TcSmem) + 1024 <= 227 * 1024, "fits a CTA's shared memory");
    static dip_per_device_once once[2];
    // the tokens' values of the union's rows, once for all CTAs
    const int xt_ctas = min((p.mask_words + 1) / 2, 2 * ctx->sm_count);
    DIP_CUDA_TRY(ctx, dip_launch_pdl(xt_build_kernel, dim3(xt_ctas), dim3(1024), 0, stream, p.mask_bits, p.v, p.batch, p.d_in,
                                     p.mask_words, ctx->xt));
    const uint16_t *xt = ctx->xt;
    if (which == 0) {
        DIP_CUDA_TRY(ctx, dip_raise_smem_limit(once[0], ctx->device, gemv_tc_kernel<0>, smem));
        DIP_CUDA_TRY(ctx, dip_launch_pdl(gemv_tc_kernel<0>, dim3(n_slabs, nparts), dim3(TC_THREADS), smem, stream, p, xt));
    } else {
        DIP_CUDA_TRY(ctx, dip_raise_smem_limit(once[1], ctx->device, gemv_tc_kernel<1>, smem));
        DIP_CUDA_TRY(ctx, dip_launch_pdl(gemv_tc_kernel<1>, dim3(n_slabs, nparts), dim3(TC_THREADS), smem, stream, p, xt));
    }
    if (nparts > 1)
        return dip_launch_combine_parts(ctx, which, nparts, n_slabs, TC_N, 256, 8, p.batch, p.d_out, p.out, stream);
    return DIP_OK;
}
