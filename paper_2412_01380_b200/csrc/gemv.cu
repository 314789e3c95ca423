// Sparse vector-matrix products over the kept weight columns (Eq. 3 with the masks of Eq. 7-8).
//
// A packed matrix stores column i of W as row i (see dip.h), so a kept column is one contiguous
// row.  The kernel is a gather-GEMV: grid = (output slabs of SEG bytes of row) x (row parts),
// sized to one CTA per SM.  Each CTA
//   1. reads the mask bits, prefix-sums their popcounts and extracts the kept rows whose rank
//      falls in its part (so parts are balanced whatever the mask looks like);
//   2. streams its rows' slab segments from HBM into a ring of shared-memory stages with
//      bulk asynchronous copies (cp.async.bulk + mbarrier transaction counts), issued by one
//      producer warp, so that ~160 KB per SM are in flight independent of register pressure;
//   3. eight consumer warps (column groups x row groups) multiply-accumulate from shared
//      memory, 16 bytes of a row per lane, in binary32;
//   4. the row groups are combined through shared memory, the parts through a scratch buffer in
//      part order by the last CTA to arrive at the slab (an arrival counter).
// The order of every sum is fixed, so results are bit-reproducible; no float atomics.
//
// One token with F32 / BF16 weights takes gemv_direct_kernel further down instead: plain loads, a
// 512-byte segment per CTA, and for gate/up no row parts at all.  INT4 weights (gemv_int4.cu) and
// BF16 batches of three or more tokens (gemv_tc.cu) run on the tensor cores; this kernel serves
// batches of F32 weights, two BF16 tokens, and the two-tier step.
//
// which = 0 (gate/up bundle): the epilogue applies silu(gate) * up (Eq. 2).  which = 1: down.
// Every wait on an mbarrier is bounded; on expiry the kernel records a status word and leaves.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "gemv_common.cuh"

namespace {

constexpr int GV_CONSUMER_WARPS = 8;
constexpr int GV_THREADS = (GV_CONSUMER_WARPS + 1) * 32;   // + one producer warp
constexpr int GV_STAGES = 5;
// Rows per round for BT tokens: the tokens' values of a round's rows stay in shared memory
// (BT x rows floats, at most 32 KB).
template <int BT> struct GvRound { static constexpr int ROWS = BT <= 4 ? GV_MAX_ROWS : (BT == 8 ? 1024 : 512); };

// Bulk asynchronous copy global -> this CTA's shared memory, completion counted on `bar`.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, unsigned bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

constexpr int GV_STAGE_BYTES = 32768;

static_assert(DIP_MAX_D <= 32768, "the row lists in shared memory are 16-bit");
template <int SEG> struct __align__(16) GemvSmem {
    // [stage][row][SEG + 16]: rows are 16 bytes apart from a multiple of 2 KB, so that the row groups'
    // 16-byte reads of neighbouring rows fall into different banks
    unsigned char ring[GV_STAGES][GV_STAGE_BYTES + (GV_STAGE_BYTES / SEG) * 16];
    uint64_t full[GV_STAGES];
    uint64_t empty[GV_STAGES];
    uint16_t idx[GV_MAX_ROWS];   // the round's columns (< DIP_MAX_D = 2^15)
    uint16_t row[GV_MAX_ROWS];   // two-tier: the arena row of each (< 2 * DIP_MAX_D = 2^16)
    uint32_t words[DIP_MAX_D / 32];
    int pre[DIP_MAX_D / 32];
    int wsum[GV_SCAN_THREADS / 32];
    int n_total;
    int last;
    int issued;          // stages the producer has issued copies for
    volatile int abort;
};

// SEG = bytes of one row handled by a CTA (512, 1024 or 2048): SEG/512 column groups of one warp
// each (16 bytes per lane), 8/(SEG/512) row groups; a stage holds 32 KB = 32768/SEG rows.
template <int WT, int WHICH, int BT, int SEG>
__global__ void __launch_bounds__(GV_THREADS, 1)
gemv_kernel(const GemvParams p)
{
    constexpr int E = WTraits<WT>::E;
    constexpr int SLAB = (SEG / 16) * E;                      // packed elements per slab
    constexpr int OUT_PER_SLAB = WHICH == 0 ? SLAB / 2 : SLAB;
    constexpr int C = WTraits<WT>::C;                         // gate/up interleave chunk (elements)
    constexpr int CG = SEG / 512;                             // column groups (warps across the segment)
    constexpr int RG = GV_CONSUMER_WARPS / CG;                // row groups
    constexpr int R = GV_STAGE_BYTES / SEG;                   // rows per stage
    constexpr int RS = SEG + 16;                              // row stride inside a stage
    extern __shared__ __align__(128) unsigned char smem_raw[];
    GemvSmem<SEG> &s = *reinterpret_cast<GemvSmem<SEG> *>(smem_raw);
    constexpr int ROWS = GvRound<BT>::ROWS;                   // rows per round
    float *s_v = reinterpret_cast<float *>(smem_raw + sizeof(GemvSmem<SEG>));   // [ROWS][BT]

    DIP_TRACE_MIN(p.tr, 0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slab = blockIdx.x, part = blockIdx.y, nparts = gridDim.y;
    const size_t seg_off = (size_t)slab * SEG;
    const int seg_bytes = (int)min((size_t)SEG, p.row_bytes - seg_off);

    if (tid == 0) {
        for (int i = 0; i < GV_STAGES; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], GV_CONSUMER_WARPS);
        }
        s.abort = 0;
        s.issued = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    dip_grid_dependency_wait();        // the mask and the vector come from the previous kernels
    DIP_TRACE_MIN(p.tr, 1);
    dip_launch_dependents();

    // ---- 1. the mask words and their popcount prefix ----
    if (tid < GV_SCAN_THREADS) {
        // thread t owns words 4t .. 4t+3 (ascending), OR-ed over the tokens of the batch
        uint32_t u[4] = {0u, 0u, 0u, 0u};
        int c = 0;
        if (4 * tid < p.mask_words) {
            if ((p.mask_words & 3) == 0) {
                for (int b = 0; b < p.batch; ++b) {
                    const uint4 q = *reinterpret_cast<const uint4 *>(p.mask_bits + (size_t)b * p.mask_words + 4 * tid);
                    u[0] |= q.x; u[1] |= q.y; u[2] |= q.z; u[3] |= q.w;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (4 * tid + j < p.mask_words)
                        for (int b = 0; b < p.batch; ++b) u[j] |= p.mask_bits[(size_t)b * p.mask_words + 4 * tid + j];
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int w = 4 * tid + j;
            if (w == p.mask_words - 1 && (p.d_in & 31)) u[j] &= (1u << (p.d_in & 31)) - 1u;   // no column beyond d_in
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

    const int cw = warp % CG, rg = warp / CG;                 // consumer roles
    const int byte_off = cw * 512 + lane * 16;
    const bool lane_ok = byte_off < seg_bytes;
    float acc[BT][E];
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[b][e] = 0.f;
    bool failed = false;
    int it_base = 0;                                          // stages issued in earlier rounds

    // The part's rows go through in rounds of at most ROWS (the in-kernel row list).
    for (int round_begin = r_begin; round_begin < r_end; round_begin += ROWS) {
        const int n_rows = min(r_end - round_begin, ROWS);
        if (round_begin != r_begin) {
            __syncthreads();                                  // everyone is done with the previous list
            if (s.abort) break;                               // uniform: read after the barrier
        }
        // ---- 2. the round's rows in rank order: each mask word that overlaps the round's rank
        //         range is expanded by one thread ----
        {
            const int lo_rank = round_begin, hi_rank = round_begin + n_rows;
            for (int w = tid; w < p.mask_words; w += GV_THREADS) {
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
        if (p.loc) {
            // two-tier: look the rows' places up together, ahead of the copies
            for (int r = tid; r < n_rows; r += GV_THREADS) s.row[r] = (uint16_t)p.loc[s.idx[r]];
            __syncthreads();
        }
        const int n_stages = (n_rows + R - 1) / R;

        if (warp == GV_CONSUMER_WARPS) {
            // ---- 3. producer warp: its lanes copy the rows of each stage ----
            for (int i = 0; i < n_stages && !failed; ++i) {
                const int it = it_base + i;
                const int st = it % GV_STAGES;
                if (it >= GV_STAGES) {
                    if (!mbar_wait(&s.empty[st], ((it / GV_STAGES) - 1) & 1, p.wait_limit_ns)) failed = true;
                }
                failed = __any_sync(0xffffffffu, failed) || s.abort;
                if (failed) break;
                const int rows_here = min(R, n_rows - i * R);
                if (lane == 0) mbar_expect_tx(&s.full[st], (unsigned)(rows_here * seg_bytes));
                __syncwarp();
                for (int r = lane; r < rows_here; r += 32) {
                    const int row = p.loc ? s.row[i * R + r] : s.idx[i * R + r];
                    bulk_g2s(&s.ring[st][r * RS], p.W + (size_t)row * p.row_bytes + seg_off, (unsigned)seg_bytes,
                             &s.full[st]);
                }
                if (lane == 0) s.issued = it + 1;
            }
            if (failed && lane == 0) {
                s.abort = 1;
                atomicExch(p.status, 1);
            }
        } else {
            // ---- 4. consumers ----
            // the tokens' values for the kept rows (zero where a token's own mask drops the row),
            // stored [row][token]; all of a row's loads are independent and issued together
            for (int r = tid; r < n_rows; r += GV_CONSUMER_WARPS * 32) {
                const int idx = s.idx[r];
                constexpr int GB = BT < 8 ? BT : 8;           // tokens gathered together
#pragma unroll
                for (int b0 = 0; b0 < BT; b0 += GB) {
                    float vv[GB];
                    uint32_t mw[GB];
#pragma unroll
                    for (int b = 0; b < GB; ++b) {
                        vv[b] = 0.f;
                        mw[b] = 0u;
                        if (b0 + b < p.batch) {
                            vv[b] = p.v[(size_t)(b0 + b) * p.d_in + idx];
                            // one token: every listed row is its own; several: ask the token's mask
                            mw[b] = p.batch == 1 ? 0xffffffffu
                                                 : p.mask_bits[(size_t)(b0 + b) * p.mask_words + (idx >> 5)];
                        }
                    }
#pragma unroll
                    for (int b = 0; b < GB; ++b) {
                        const float val = ((mw[b] >> (idx & 31)) & 1u) ? vv[b] : 0.f;
                        s_v[r * BT + b0 + b] = val;
                    }
                }
            }
            asm volatile("bar.sync 2, %0;" ::"n"(GV_CONSUMER_WARPS * 32) : "memory");

            for (int i = 0; i < n_stages; ++i) {
                const int it = it_base + i;
                const int st = it % GV_STAGES;
                if (!mbar_wait(&s.full[st], (it / GV_STAGES) & 1, p.wait_limit_ns)) failed = true;
                if (failed || s.abort) { failed = true; break; }
                const int rows_here = min(R, n_rows - i * R);
                if (lane_ok) {
                    {
#pragma unroll
                        for (int rr = 0; rr < R / RG; ++rr) {
                            const int r = rr * RG + rg;
                            if (r < rows_here) {
                                const uint4 raw = *reinterpret_cast<const uint4 *>(&s.ring[st][r * RS + byte_off]);
                                float w[E];
                                decode16<WT>(raw, w);
                                float xv[BT];
                                if constexpr (BT >= 4) {
#pragma unroll
                                    for (int b = 0; b < BT; b += 4) {
                                        const float4 t4 = *reinterpret_cast<const float4 *>(&s_v[(i * R + r) * BT + b]);
                                        xv[b] = t4.x; xv[b + 1] = t4.y; xv[b + 2] = t4.z; xv[b + 3] = t4.w;
                                    }
                                } else {
#pragma unroll
                                    for (int b = 0; b < BT; ++b) xv[b] = s_v[(i * R + r) * BT + b];
                                }
#pragma unroll
                                for (int b = 0; b < BT; ++b)
#pragma unroll
                                    for (int e = 0; e < E; ++e) acc[b][e] = fmaf(w[e], xv[b], acc[b][e]);
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&s.empty[st]);
            }
            if (failed) {
                s.abort = 1;
                if (lane == 0) atomicExch(p.status, 1);
            }
        }
        it_base += n_stages;
    }

    DIP_TRACE_MAX(p.tr, 3);            // streaming done
    // ---- 5. combine the row groups through the (now idle) ring, in group order ----
    __syncthreads();
    if (s.abort) {
        // a wait ran out: let the copies already issued into this CTA's shared memory land
        // (bounded again) before the ring is reused or the CTA leaves
        if (tid == 0) {
            for (int it = max(0, s.issued - GV_STAGES); it < s.issued; ++it)
                (void)mbar_wait(&s.full[it % GV_STAGES], (it / GV_STAGES) & 1, p.wait_limit_ns);
        }
        __syncthreads();
    }
    float *red = reinterpret_cast<float *>(&s.ring[0][0]);    // [RG-1][CG*32 lanes][BT][E]
    float *own = red + (RG - 1) * CG * 32 * BT * E;           // [BT][SLAB] sums of this CTA, after red
    static_assert(((RG - 1) * CG * 32 * BT * E + BT * SLAB) * sizeof(float) <= sizeof(s.ring), "ring too small");
    {
    if (warp < GV_CONSUMER_WARPS && rg > 0) {
#pragma unroll
            for (int b = 0; b < BT; ++b)
#pragma unroll
                for (int e = 0; e < E; ++e)
                    red[((((rg - 1) * CG + cw) * 32 + lane) * BT + b) * E + e] = acc[b][e];
        }
        __syncthreads();
        if (warp < GV_CONSUMER_WARPS && rg == 0) {
            float *dst = (nparts > 1 || p.defer) ? p.partials + ((size_t)(p.part_base + part) * gridDim.x + slab) * (BT * SLAB) : own;
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                float sum[E];
#pragma unroll
                for (int e = 0; e < E; ++e) sum[e] = acc[b][e];
#pragma unroll
                for (int g = 1; g < RG; ++g)
#pragma unroll
                    for (int e = 0; e < E; ++e) sum[e] += red[((((g - 1) * CG + cw) * 32 + lane) * BT + b) * E + e];
                float *d = dst + b * SLAB + (cw * 32 + lane) * E;
#pragma unroll
                for (int e = 0; e < E; e += 4)
                    *reinterpret_cast<float4 *>(d + e) = make_float4(sum[e], sum[e + 1], sum[e + 2], sum[e + 3]);
            }
        }
    }

    // ---- 6. combine the parts ----
    if ((BT >= 8 && nparts > 1) || p.defer) {
        // many tokens: the partial sums of a slab are too much for one CTA to add up alone;
        // combine_parts_kernel does it right after this kernel, spread over the whole device.
        // (Also when the caller adds the parts of two launches.)
        DIP_TRACE_MAX(p.tr, 2);
        return;
    }
    if (nparts > 1) {
        __threadfence();
        __syncthreads();
        if (tid == 0) s.last = atomicAdd(&p.tickets[slab], 1u) == (unsigned)(nparts - 1);
        __syncthreads();
        if (!s.last) {
            DIP_TRACE_MAX(p.tr, 2);
            return;
        }
        __threadfence();
    } else {
        __syncthreads();
    }
    if (s.abort) {
        // a wait ran out somewhere in this CTA: no result; leave the slab's counter clean
        if (tid == 0 && nparts > 1) p.tickets[slab] = 0;
        return;
    }
    // four consecutive outputs per thread (16-byte loads of the partial sums)
    for (int t = tid; t < BT * (OUT_PER_SLAB / 4); t += GV_THREADS) {
        const int b = t / (OUT_PER_SLAB / 4), o = (t % (OUT_PER_SLAB / 4)) * 4;
        const int j = slab * OUT_PER_SLAB + o;
        if (b >= p.batch || j >= p.d_out) continue;
        int e0, e1 = 0;
        if (WHICH == 0) {
            e0 = (o / C) * 2 * C + (o % C);      // gate elements of outputs o .. o+3
            e1 = e0 + C;                         // matching up elements
        } else {
            e0 = o;
        }
        float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
        if (nparts > 1) {
            // parts in part order; eight loads in flight at a time
            const size_t stride = (size_t)gridDim.x * (BT * SLAB);
            const float *pp = p.partials + (size_t)slab * (BT * SLAB) + b * SLAB;
            for (int q0 = 0; q0 < nparts; q0 += 8) {
                float4 a0[8], a1[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    a0[q] = a1[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (q0 + q < nparts) {
                        a0[q] = __ldcg(reinterpret_cast<const float4 *>(pp + (size_t)(q0 + q) * stride + e0));
                        if (WHICH == 0)
                            a1[q] = __ldcg(reinterpret_cast<const float4 *>(pp + (size_t)(q0 + q) * stride + e1));
                    }
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    s0.x += a0[q].x; s0.y += a0[q].y; s0.z += a0[q].z; s0.w += a0[q].w;
                    s1.x += a1[q].x; s1.y += a1[q].y; s1.z += a1[q].z; s1.w += a1[q].w;
                }
            }
        } else {
            s0 = *reinterpret_cast<const float4 *>(own + b * SLAB + e0);
            if (WHICH == 0) s1 = *reinterpret_cast<const float4 *>(own + b * SLAB + e1);
        }
        float4 r = s0;
        if (WHICH == 0) r = make_float4(silu_f32(s0.x) * s1.x, silu_f32(s0.y) * s1.y, silu_f32(s0.z) * s1.z, silu_f32(s0.w) * s1.w);
        *reinterpret_cast<float4 *>(p.out + (size_t)b * p.d_out + j) = r;
    }
    if (nparts > 1 && tid == 0) p.tickets[slab] = 0;   // ready for the next launch
    DIP_TRACE_MAX(p.tr, 2);
}


// ---------------------------------------------------------------------------------------------
// One token, F32 / BF16: the same product with plain loads instead of the copy ring.  A CTA
// owns a 512-byte segment of the packed rows (one 16-byte piece per lane) and, with enough
// segments, ALL kept rows of it, so that nothing is left to combine across CTAs: its warps take
// the rows round robin, each lane keeps the E sums of its piece, U loads per lane are in flight
// (NW x U x 512 bytes per SM), the warps' sums meet in shared memory and the epilogue writes
// the outputs.  Only when the rows have few segments (down: 20) are the rows split into parts,
// combined as above by the last CTA of a segment.  At any moment all CTAs read neighbouring
// segments of the same few rows, so DRAM sees whole rows.
// ---------------------------------------------------------------------------------------------
constexpr int GD_SEG = 512;

template <int NW> struct __align__(16) GemvDirectSmem {
    uint16_t idx[GV_MAX_ROWS];
    uint32_t words[DIP_MAX_D / 32];
    int pre[DIP_MAX_D / 32];
    int wsum[GV_SCAN_THREADS / 32];
    int n_total;
    int last;
    float red[NW][32 * 8];           // [warp][lane * E + e], E <= 8
    float sum[32 * 8];
};

template <int WT, int WHICH, int NW, int U>
__global__ void __launch_bounds__(NW * 32, 1)
gemv_direct_kernel(const GemvParams p)
{
    constexpr int E = WTraits<WT>::E;
    constexpr int SLAB = 32 * E;                              // packed elements per segment
    constexpr int OUT_PER_SLAB = WHICH == 0 ? SLAB / 2 : SLAB;
    constexpr int C = WTraits<WT>::C;
    constexpr int THREADS = NW * 32;
    static_assert(THREADS >= GV_SCAN_THREADS && E <= 8, "");
    __shared__ GemvDirectSmem<NW> s;

    DIP_TRACE_MIN(p.tr, 0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slab = blockIdx.x, part = blockIdx.y, nparts = gridDim.y;
    const size_t byte_off = (size_t)slab * GD_SEG + lane * 16;
    const bool lane_ok = byte_off < p.row_bytes;
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(p.tr, 1);
    dip_launch_dependents();

    // the stamp that the epilogue's rank key needs travels while the rows stream
    int key_stamp = 0;
    if (WHICH == 0 && p.key_coarse && p.key_stamp && tid < OUT_PER_SLAB && slab * OUT_PER_SLAB + tid < p.d_out)
        key_stamp = __ldcg(p.key_stamp + slab * OUT_PER_SLAB + tid);

    // ---- 1. the mask words and their popcount prefix (as in gemv_kernel) ----
    if (tid < GV_SCAN_THREADS) {
        uint32_t u[4] = {0u, 0u, 0u, 0u};
        int c = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int w = 4 * tid + j;
            if (w < p.mask_words) u[j] = p.mask_bits[w];
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

    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    const char *base = p.W + byte_off;

    for (int round_begin = r_begin; round_begin < r_end; round_begin += GV_MAX_ROWS) {
        const int n_rows = min(r_end - round_begin, GV_MAX_ROWS);
        if (round_begin != r_begin) __syncthreads();
        // ---- 2. the round's rows in rank order ----
        {
            const int lo_rank = round_begin, hi_rank = round_begin + n_rows;
            for (int w = tid; w < p.mask_words; w += THREADS) {
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
        // ---- 3. stream: warp w takes rows w, w + NW, ...; U of them in flight per lane.  The
        //         first batch of loads goes out before the vector's values are fetched ----
        for (int r0 = warp; r0 < n_rows; r0 += NW * U) {
            uint4 q[U];
            float xv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = r0 + u * NW;
                q[u] = make_uint4(0u, 0u, 0u, 0u);
                xv[u] = 0.f;
                if (r < n_rows) {
                    const int idx = s.idx[r];
                    if (lane_ok) q[u] = __ldcs(reinterpret_cast<const uint4 *>(base + (size_t)idx * p.row_bytes));
                    xv[u] = __ldg(p.v + idx);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float w[E];
                decode16<WT>(q[u], w);
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] = fmaf(w[e], xv[u], acc[e]);
            }
        }
    }
    DIP_TRACE_MAX(p.tr, 3);            // streaming done

    // ---- 4. the warps' sums, in warp order ----
#pragma unroll
    for (int e = 0; e < E; ++e) s.red[warp][lane * E + e] = acc[e];
    __syncthreads();
    if (tid < SLAB) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) t += s.red[w][tid];
        if (nparts > 1) p.partials[((size_t)part * gridDim.x + slab) * SLAB + tid] = t;
        else s.sum[tid] = t;
    }
    // ---- 5. the parts, in part order, by the last CTA of the segment ----
    if (nparts > 1) {
        __threadfence();
        __syncthreads();
        if (tid == 0) s.last = atomicAdd(&p.tickets[slab], 1u) == (unsigned)(nparts - 1);
        __syncthreads();
        if (!s.last) {
            DIP_TRACE_MAX(p.tr, 2);
            return;
        }
        __threadfence();
        if (tid < SLAB) {
            const size_t stride = (size_t)gridDim.x * SLAB;
            const float *pp = p.partials + (size_t)slab * SLAB + tid;
            float t = 0.f;
            for (int q0 = 0; q0 < nparts; q0 += 8) {
                float a[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) a[q] = q0 + q < nparts ? __ldcg(pp + (size_t)(q0 + q) * stride) : 0.f;
#pragma unroll
                for (int q = 0; q < 8; ++q) t += a[q];
            }
            s.sum[tid] = t;
        }
        if (tid == 0) p.tickets[slab] = 0;                    // ready for the next launch
    }
    __syncthreads();
    // ---- 6. epilogue ----
    if (tid < OUT_PER_SLAB) {
        const int o = tid, j = slab * OUT_PER_SLAB + o;
        if (j < p.d_out) {
            float r;
            if (WHICH == 0) {
                const int e0 = (o / C) * 2 * C + (o % C);     // gate element; its up element is C further
                r = silu_f32(s.sum[e0]) * s.sum[e0 + C];
            } else {
                r = s.sum[o];
            }
            p.out[j] = r;
            if (WHICH == 0 && p.key_coarse) {
                // what the select would form from h_j and the stamp, cut to its top 16 bits
                float a = fabsf(r);
                if (p.key_stamp) a = __fmul_rn(a, key_stamp >= 0 ? 1.0f : p.key_gamma);
                p.key_coarse[j] = (uint16_t)((__float_as_uint(a) & 0x7fffffffu) >> 16);
            }
        }
    }
    DIP_TRACE_MAX(p.tr, 2);
}

template <int WT, int WHICH, int NW, int U>
dip_status launch_direct_cfg(dip_ctx *ctx, GemvParams &p, int n_kept_max, cudaStream_t stream)
{
    constexpr int SLAB = 32 * WTraits<WT>::E;
    const int n_slabs = (int)((p.row_bytes + GD_SEG - 1) / GD_SEG);
    int nparts = ctx->sm_count / n_slabs;
    if (nparts > n_kept_max) nparts = n_kept_max;
    if (nparts < 1) nparts = 1;
    if (n_slabs > ctx->n_tickets) return DIP_ERR_WORKSPACE;
    if (nparts > 1 && (size_t)nparts * n_slabs * SLAB > ctx->partials_floats) return DIP_ERR_WORKSPACE;
    p.defer = 0;
    p.part_base = 0;
    DIP_CUDA_TRY(ctx, dip_launch_pdl(gemv_direct_kernel<WT, WHICH, NW, U>, dim3(n_slabs, nparts), dim3(NW * 32), 0,
                                     stream, p));
    return DIP_OK;
}

// 32 warps x 4 loads in flight per lane (64 KB per SM) measured best: more warps beat deeper
// unrolling (16 x 8: 3 % slower, 8 x 16: 12 % slower on Phi-3-Medium shapes).
template <int WT, int WHICH>
dip_status launch_direct(dip_ctx *ctx, GemvParams &p, int n_kept_max, cudaStream_t stream)
{
    return launch_direct_cfg<WT, WHICH, 32, 4>(ctx, p, n_kept_max, stream);
}

// Self-test of the bounded wait: one CTA arms a barrier for bytes that no copy will ever deliver,
// waits on it the way the copy-ring consumers do, and on expiry records status 1 and returns.
__global__ void bounded_wait_selftest_kernel(int *status, unsigned long long limit_ns, unsigned long long *waited_ns)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(&bar, 16u);                  // one arrival made, 16 bytes still owed: the phase never completes
        const unsigned long long t0 = dip_gtime();
        const bool ok = mbar_wait(&bar, 0u, limit_ns);
        if (waited_ns) *waited_ns = dip_gtime() - t0;
        if (!ok) atomicExch(status, 1);
    }
}

}  // namespace

dip_status dip_launch_bounded_wait_selftest(dip_ctx *ctx, unsigned long long limit_ns, unsigned long long *waited_ns,
                                            cudaStream_t stream)
{
    bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(ctx->status, limit_ns, waited_ns);
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}

namespace {

// Bit set from an ascending index list (the list-based entry points).
__global__ void idx_to_mask_kernel(const int32_t *__restrict__ idx, int n, int d, uint32_t *__restrict__ mask)
{
    for (int r = blockIdx.x * blockDim.x + threadIdx.x; r < n; r += gridDim.x * blockDim.x) {
        const int i = idx[r];
        if (i >= 0 && i < d) atomicOr(&mask[i >> 5], 1u << (i & 31));   // out-of-range entries are ignored
    }
}

// Sum of the row parts and the epilogue as a kernel of its own (large batches; the two launches
// of the two-tier step).  CP_LANES (1 or 8) neighbouring lanes share four outputs: lane l adds the
// parts l, l + CP_LANES, ... (its loads in flight together), then the lanes' sums meet in a fixed
// shuffle tree, so the result is reproducible.  Eight lanes pay when there are many parts.  partials: [nparts][n_slabs][bt][slab]; gate/up rows are
// interleaved in chunks of c.
template <int WHICH, int CP_LANES>
__global__ void __launch_bounds__(256)
combine_parts_kernel(const float *__restrict__ partials, int nparts, int n_slabs, int bt, int slab_elems, int c,
                     int batch, int d_out, float *__restrict__ out)
{
    dip_grid_dependency_wait();
    dip_launch_dependents();
    const int out_per_slab = WHICH == 0 ? slab_elems / 2 : slab_elems;
    const int groups = out_per_slab / 4;
    const long long total = (long long)n_slabs * batch * groups;
    const size_t stride = (size_t)n_slabs * bt * slab_elems;
    const int pl = threadIdx.x % CP_LANES;
    const long long first = (blockIdx.x * (long long)blockDim.x + threadIdx.x) / CP_LANES;
    const long long step = (long long)gridDim.x * blockDim.x / CP_LANES;
    // whole warps iterate together (the bound is rounded up to the warp's four groups)
    for (long long t0 = first - (threadIdx.x % 32) / CP_LANES; t0 < total; t0 += step) {
        const long long t = t0 + (threadIdx.x % 32) / CP_LANES;
        const bool live = t < total;
        const int o = live ? (int)(t % groups) * 4 : 0;
        const int b = live ? (int)((t / groups) % batch) : 0;
        const int slab = live ? (int)(t / ((long long)groups * batch)) : 0;
        const int j = slab * out_per_slab + o;
        const int e0 = WHICH == 0 ? (o / c) * 2 * c + (o % c) : o;
        const int e1 = e0 + c;
        const float *pp = partials + ((size_t)slab * bt + b) * slab_elems;
        float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
        for (int q0 = pl; q0 < nparts; q0 += 8 * CP_LANES) {
            float4 a0[8], a1[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                a0[q] = a1[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                const int part = q0 + q * CP_LANES;
                if (live && part < nparts) {
                    a0[q] = __ldcg(reinterpret_cast<const float4 *>(pp + (size_t)part * stride + e0));
                    if (WHICH == 0) a1[q] = __ldcg(reinterpret_cast<const float4 *>(pp + (size_t)part * stride + e1));
                }
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                s0.x += a0[q].x; s0.y += a0[q].y; s0.z += a0[q].z; s0.w += a0[q].w;
                s1.x += a1[q].x; s1.y += a1[q].y; s1.z += a1[q].z; s1.w += a1[q].w;
            }
        }
#pragma unroll
        for (int m = 1; m < CP_LANES; m <<= 1) {
            s0.x += __shfl_xor_sync(0xffffffffu, s0.x, m); s0.y += __shfl_xor_sync(0xffffffffu, s0.y, m);
            s0.z += __shfl_xor_sync(0xffffffffu, s0.z, m); s0.w += __shfl_xor_sync(0xffffffffu, s0.w, m);
            if (WHICH == 0) {
                s1.x += __shfl_xor_sync(0xffffffffu, s1.x, m); s1.y += __shfl_xor_sync(0xffffffffu, s1.y, m);
                s1.z += __shfl_xor_sync(0xffffffffu, s1.z, m); s1.w += __shfl_xor_sync(0xffffffffu, s1.w, m);
            }
        }
        if (live && pl == 0 && j < d_out) {
            float4 r = s0;
            if (WHICH == 0)
                r = make_float4(silu_f32(s0.x) * s1.x, silu_f32(s0.y) * s1.y, silu_f32(s0.z) * s1.z, silu_f32(s0.w) * s1.w);
            *reinterpret_cast<float4 *>(out + (size_t)b * d_out + j) = r;
        }
    }
}

}  // namespace

dip_status dip_launch_combine_parts(dip_ctx *ctx, int which, int total_parts, int n_slabs, int bt, int slab_elems, int c,
                                    int batch, int d_out, float *out, cudaStream_t stream)
{
    const long long groups = (long long)n_slabs * batch * ((which == 0 ? slab_elems / 2 : slab_elems) / 4);
    const float *partials = ctx->partials;
    // eight lanes per group of outputs pay when there are many parts
    const bool wide = total_parts >= 16;
    const int blocks = (int)(((wide ? groups * 8 : groups) + 255) / 256);
    cudaError_t e;
    if (which == 0)
        e = wide ? dip_launch_pdl(combine_parts_kernel<0, 8>, dim3(blocks), dim3(256), 0, stream, partials, total_parts,
                                  n_slabs, bt, slab_elems, c, batch, d_out, out)
                 : dip_launch_pdl(combine_parts_kernel<0, 1>, dim3(blocks), dim3(256), 0, stream, partials, total_parts,
                                  n_slabs, bt, slab_elems, c, batch, d_out, out);
    else
        e = wide ? dip_launch_pdl(combine_parts_kernel<1, 8>, dim3(blocks), dim3(256), 0, stream, partials, total_parts,
                                  n_slabs, bt, slab_elems, c, batch, d_out, out)
                 : dip_launch_pdl(combine_parts_kernel<1, 1>, dim3(blocks), dim3(256), 0, stream, partials, total_parts,
                                  n_slabs, bt, slab_elems, c, batch, d_out, out);
    DIP_CUDA_TRY(ctx, e);
    return DIP_OK;
}

namespace {

template <int WT, int WHICH, int BT, int SEG>
dip_status launch_seg(dip_ctx *ctx, GemvParams &p, int n_slabs, int nparts, int mode, cudaStream_t stream)
{
    constexpr int SLAB = (SEG / 16) * WTraits<WT>::E;
    const size_t per_part = (size_t)n_slabs * BT * SLAB;
    // mode 1 / 2: first / second of two launches whose row parts one combine kernel adds up
    const int total_parts = mode ? 2 * nparts : nparts;
    if ((nparts > 1 || mode) && (size_t)total_parts * per_part > ctx->partials_floats) return DIP_ERR_WORKSPACE;
    p.defer = mode != 0;
    p.part_base = mode == 2 ? nparts : 0;
    const size_t smem = sizeof(GemvSmem<SEG>) + (size_t)BT * (GvRound<BT>::ROWS + 8) * sizeof(float);
    static dip_per_device_once once;   // per instantiation
    DIP_CUDA_TRY(ctx, dip_raise_smem_limit(once, ctx->device, gemv_kernel<WT, WHICH, BT, SEG>, smem));
    dim3 grid(n_slabs, nparts);
    DIP_CUDA_TRY(ctx, dip_launch_pdl(gemv_kernel<WT, WHICH, BT, SEG>, grid, dim3(GV_THREADS), smem, stream, p));
    if ((BT >= 8 && nparts > 1 && !mode) || mode == 2)
        return dip_launch_combine_parts(ctx, WHICH, total_parts, n_slabs, BT, SLAB, WTraits<WT>::C, p.batch, p.d_out,
                                        p.out, stream);
    return DIP_OK;
}

// Segment width and number of row parts: one CTA per SM, all resident at once.  A wide
// segment is kinder to DRAM, but few slabs mean many parts, and the CTA that finishes a slab
// then has nparts * SEG bytes of partial sums to add up alone.  Bulk copies shorter than 2 KB
// run into the copy engine's request rate (measured: 1 KB segments stream a third slower), so
// the segment is narrowed only when that tail would get very long.
template <int WT, int WHICH, int BT>
dip_status launch_one(dip_ctx *ctx, GemvParams &p, int n_kept_max, int mode, cudaStream_t stream)
{
    int seg = ctx->gemv_seg;
    int n_slabs = 0, nparts = 1;
    const int cands[3] = {2048, 1024, 512};
    for (int c = 0; c < 3; ++c) {
        const int sg = seg ? seg : cands[c];
        n_slabs = (int)((p.row_bytes + sg - 1) / sg);
        nparts = ctx->sm_count / n_slabs;
        if (nparts > n_kept_max) nparts = n_kept_max;
        if (nparts < 1) nparts = 1;
        // bytes of partial sums the CTA that completes a slab adds up: nparts x slab floats
        const long long tail = (long long)nparts * (sg / 16) * WTraits<WT>::E * 4;
        if (seg || tail <= 131072 || sg == 512) {
            seg = sg;
            break;
        }
    }
    if (n_slabs > ctx->n_tickets) return DIP_ERR_WORKSPACE;
    switch (seg) {
    case 2048: return launch_seg<WT, WHICH, BT, 2048>(ctx, p, n_slabs, nparts, mode, stream);
    case 1024: return launch_seg<WT, WHICH, BT, 1024>(ctx, p, n_slabs, nparts, mode, stream);
    default: return launch_seg<WT, WHICH, BT, 512>(ctx, p, n_slabs, nparts, mode, stream);
    }
}

template <int WT, int WHICH>
dip_status launch_bt(dip_ctx *ctx, GemvParams &p, int n_kept_max, int mode, cudaStream_t stream)
{
    if (p.batch == 1) return launch_one<WT, WHICH, 1>(ctx, p, n_kept_max, mode, stream);
    if (p.batch == 2) return launch_one<WT, WHICH, 2>(ctx, p, n_kept_max, mode, stream);
    if (p.batch <= 4 && WT != DIP_W_BF16) return launch_one<WT, WHICH, 4>(ctx, p, n_kept_max, mode, stream);
    if (p.batch <= 8) return launch_one<WT, WHICH, 8>(ctx, p, n_kept_max, mode, stream);
    return launch_one<WT, WHICH, 16>(ctx, p, n_kept_max, mode, stream);
}

}  // namespace

dip_status dip_launch_gemv(dip_ctx *ctx, const dip_mlp_weights *w, int which,
                           const float *v, int batch, const uint32_t *mask_bits, int n_kept_max,
                           float *out, cudaStream_t stream, const dip_gemv_rows *rows, dip_gemv_keys *keys)
{
    const int mode = rows ? rows->mode : 0;
    if (keys) keys->written = 0;
    if (mode && batch != 1) return DIP_ERR_UNSUPPORTED;
    const bool int4 = w->wtype == DIP_W_INT4_G128;
    if (int4 && batch > 1) return DIP_ERR_UNSUPPORTED;      // the 4-bit path is single-token
    const size_t row_elems = which == 0 ? (size_t)2 * w->d_ff : (size_t)w->d_model;
    GemvParams p;
    p.W = rows ? (const char *)rows->base : (const char *)(which == 0 ? w->gate_up : w->down);
    p.loc = rows ? rows->loc : nullptr;
    p.row_bytes = w->wtype == DIP_W_F32 ? row_elems * 4 : w->wtype == DIP_W_BF16 ? row_elems * 2 : row_elems / 2;
    p.scales = (const uint16_t *)(which == 0 ? w->gate_up_scales : w->down_scales);
    p.scale_row_elems = row_elems;
    p.d_in = which == 0 ? w->d_model : w->d_ff;
    p.d_out = which == 0 ? w->d_ff : w->d_model;
    p.mask_words = (p.d_in + 31) / 32;
    p.partials = ctx->partials;
    p.tickets = ctx->tickets;
    p.status = ctx->status;
    p.wait_limit_ns = ctx->wait_limit_ns;
    p.key_coarse = nullptr;
    p.key_stamp = nullptr;
    p.key_gamma = 1.0f;

    // all tokens of the batch in one launch (up to 16 sets of accumulators in registers): the
    // union of their rows is read once
    for (int b0 = 0; b0 < batch; b0 += 16) {
        p.batch = batch - b0 < 16 ? batch - b0 : 16;
        p.v = v + (size_t)b0 * p.d_in;
        p.mask_bits = mask_bits + (size_t)b0 * p.mask_words;
        p.out = out + (size_t)b0 * p.d_out;
        p.tr = dip_trace_slot(ctx, which == 0 ? 4 : 5);
        dip_status st;
        if (ctx->gemv_direct && !int4 && p.batch == 1 && !rows) {
            if (keys && which == 0 && batch == 1 && keys->coarse) {
                p.key_coarse = keys->coarse;
                p.key_stamp = keys->stamp;
                p.key_gamma = keys->gamma;
                keys->written = 1;
            }
            if (w->wtype == DIP_W_F32)
                st = which == 0 ? launch_direct<DIP_W_F32, 0>(ctx, p, n_kept_max, stream)
                                : launch_direct<DIP_W_F32, 1>(ctx, p, n_kept_max, stream);
            else
                st = which == 0 ? launch_direct<DIP_W_BF16, 0>(ctx, p, n_kept_max, stream)
                                : launch_direct<DIP_W_BF16, 1>(ctx, p, n_kept_max, stream);
        } else if (int4) {
            if (keys && which == 0 && keys->coarse) {
                p.key_coarse = keys->coarse;
                p.key_stamp = keys->stamp;
                p.key_gamma = keys->gamma;
            }
            st = dip_launch_gemv_int4(ctx, p, which, n_kept_max, mode, stream);
            if (st == DIP_OK && p.key_coarse && !mode) keys->written = 1;
        }
        else if (ctx->gemv_direct && p.batch == 2 && !rows) {
            if (keys && which == 0 && keys->coarse && batch <= 16) {
                p.key_coarse = keys->coarse;
                keys->written = 1;
            }
            st = dip_launch_gemv_direct_bt(ctx, p, w->wtype, which, n_kept_max, stream);   // two tokens: plain loads and FMAs keep up
        }
        else if (w->wtype == DIP_W_F32)
            st = which == 0 ? launch_bt<DIP_W_F32, 0>(ctx, p, n_kept_max, mode, stream)
                            : launch_bt<DIP_W_F32, 1>(ctx, p, n_kept_max, mode, stream);
        else if (p.batch >= 3 && !mode) {
            if (keys && which == 0 && keys->coarse && batch <= 16) p.key_coarse = keys->coarse;
            st = dip_launch_gemv_tc(ctx, p, which, n_kept_max, stream);       // a dense contraction: tensor cores
            if (st == DIP_OK && p.key_coarse) keys->written = 1;      // (the launcher drops the request when it splits the rows)
        }
        else
            st = which == 0 ? launch_bt<DIP_W_BF16, 0>(ctx, p, n_kept_max, mode, stream)
                            : launch_bt<DIP_W_BF16, 1>(ctx, p, n_kept_max, mode, stream);
        if (st != DIP_OK) return st;
    }
    return DIP_OK;
}

dip_status dip_launch_idx_to_mask(dip_ctx *ctx, const int32_t *idx, int n, int d, uint32_t *mask, cudaStream_t stream)
{
    DIP_CUDA_TRY(ctx, cudaMemsetAsync(mask, 0, sizeof(uint32_t) * ((d + 31) / 32), stream));
    idx_to_mask_kernel<<<(n + 255) / 256, 256, 0, stream>>>(idx, n, d, mask);
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}
