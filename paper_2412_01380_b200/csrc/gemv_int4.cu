// The sparse vector-matrix product over the kept weight columns (Eq. 3 with the masks of Eq. 7-8)
// for INT4-g128 weights, one token: W[j, i] = (code[j, i] - 8) * S[i / 128][j].
//
// Decoding 4-bit codes on the plain ALUs costs several instructions per weight and bounds the
// product far below the memory rate.  Here the multiply-adds go to the tensor cores and the ALUs
// only move nibbles:
//   * a packed row is a sequence of chunks of 128 codes laid out (by dip_pack_weights) so that the
//     8 bytes a lane loads are exactly its share of the A fragments of eight 16 x 16 tiles
//     (m16n8k16: 16 outputs x 16 kept rows): words w and w + 8 of the chunk, nibble m of word w
//     being output 16 m + w;
//   * a code becomes a binary16 number without arithmetic: left in the low mantissa bits of a
//     half whose other bits are zero it IS the subnormal code * 2^-24 (2^-20 from the upper
//     nibble of a byte); one byte permute joins the bytes of two rows and one AND per fragment
//     register isolates the nibble pair;
//   * B holds the token's values, pre-scaled by a power of two to the top of the binary16 range
//     and split hi + lo (two columns), in the columns of the row's scale group: the eight columns
//     are four consecutive groups x (hi, lo), so one accumulator tile serves four groups and the
//     16 rows of an MMA may straddle group boundaries;
//   * a ninth tile of ones yields sum(x) per group for the -8 offset of the codes;
//   * every four groups the accumulators are multiplied by the groups' binary16 scales into
//     binary32 sums.  All products are exact in binary32; sums are binary32, in a fixed order.
// Rows are loaded straight from global memory into the fragment registers (8-byte loads, four
// K-blocks = 64 rows in flight per warp); a CTA owns a segment of the packed rows (its warps
// split the segment's chunks and, when there are few chunks, the K-blocks, each warp a contiguous
// run of them) and a part of the rows.
#include <cuda_fp16.h>

#include "common.cuh"
#include "gemv_common.cuh"

namespace {

constexpr int I4_WARPS = 16;
constexpr int I4_THREADS = I4_WARPS * 32;
constexpr int I4_U = 4;                     // K-blocks in flight per warp
constexpr int I4_ROUND_ROWS = 1024;         // kept rows per round
constexpr int I4_MAX_QUADS = DIP_MAX_D / 512;
constexpr int I4_MAX_KB = I4_ROUND_ROWS / 16 + I4_MAX_QUADS;   // K-blocks per round (each quad pads its last one)
constexpr uint32_t I4_PAD = 0xffffffffu;
constexpr int I4_SCALE_BYTES = 32768;       // shared memory for the scale rows of a round's groups
constexpr int I4_STAGE_LOADS = I4_SCALE_BYTES / 16 / I4_THREADS;   // 16-byte pieces per thread

struct __align__(16) I4Smem {
    __half bt[I4_MAX_KB][8][16];            // B^T of each K-block: [column = 2 * group-in-quad + (hi, lo)][slot]
    uint32_t kb_off[I4_MAX_KB][16];         // packed row of each slot, in 16-byte units; I4_PAD = empty slot
    int kb_quad[I4_MAX_KB];
    uint32_t words[DIP_MAX_D / 32];
    int pre[DIP_MAX_D / 32];
    uint16_t idx[I4_ROUND_ROWS];
    int qstart[I4_MAX_QUADS], qend[I4_MAX_QUADS], qblk[I4_MAX_QUADS];
    int wsum[GV_SCAN_THREADS / 32];
    float wmax[I4_WARPS];
    int n_total;
    int n_kb;
    int last;
};
// after I4Smem (dynamic): float sums[kgroups][seg_chunks * 128], float total[seg_chunks * 128], and
// I4_SCALE_BYTES of staged scales [group][seg_chunks * 128]

__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Local element e of a chunk of a gate/up row: e < 64 gate output e, else up output e - 64.
// WHICH = 0: grid.x segments of seg_chunks chunks of the bundled rows; WHICH = 1: of the down rows.
template <int WHICH, int SEGC>
__global__ void __launch_bounds__(I4_THREADS, 1)
gemv_int4_kernel(const GemvParams p, int n_chunks)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    I4Smem &s = *reinterpret_cast<I4Smem *>(smem_raw);
    constexpr int seg_chunks = SEGC;                            // chunks of 128 codes per segment
    constexpr int seg_elems = seg_chunks * 128;
    constexpr int kgroups = I4_WARPS / seg_chunks;
    float *s_sums = reinterpret_cast<float *>(smem_raw + sizeof(I4Smem));      // [kgroups][seg_elems]
    float *s_total = s_sums + kgroups * seg_elems;                             // [seg_elems]
    uint16_t *s_scale = reinterpret_cast<uint16_t *>(s_total + seg_elems);     // [staged groups][seg_elems]

    DIP_TRACE_MIN(p.tr, 0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int slab = blockIdx.x, part = blockIdx.y, nparts = gridDim.y;
    const int chunk = warp % seg_chunks, kgroup = warp / seg_chunks;
    const int gchunk = slab * seg_chunks + chunk;               // chunk of the packed row
    const bool chunk_ok = gchunk < n_chunks;
    const int n_groups = p.d_in / DIP_INT4_GROUP;
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(p.tr, 1);
    dip_launch_dependents();

    // the stamps that the epilogue's rank keys need travel while the rows stream
    int key_stamp[2] = {0, 0};
    if (WHICH == 0 && p.key_coarse && p.key_stamp) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int o = tid + i * I4_THREADS;
            const int j = (slab * seg_chunks + (o >> 6)) * 64 + (o & 63);
            if (o < seg_chunks * 64 && j < p.d_out) key_stamp[i] = __ldcg(p.key_stamp + j);
        }
    }
    // ---- 1. the mask words and their popcount prefix ----
    uint32_t u[4] = {0u, 0u, 0u, 0u};
    if (tid < GV_SCAN_THREADS) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int w = 4 * tid + j;
            if (w < p.mask_words) u[j] = p.mask_bits[w];
        }
    }
    if (tid < GV_SCAN_THREADS) {
        int c = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) c += __popc(u[j]);
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
    // The largest magnitude among the values of the columns that the mask words of this part's
    // rank range cover (a superset of the part's rows) fixes the power of two that lifts the
    // values to the top of the binary16 range: the largest lands in [2^14, 2^15).
    float scale_up, scale_down;
    {
        float amax = 0.f;
        for (int w = tid; w < p.mask_words; w += I4_THREADS) {
            const int lo = s.pre[w];
            if (lo < r_end && lo + __popc(s.words[w]) > r_begin) {
                const float4 *v4 = reinterpret_cast<const float4 *>(p.v + 32 * w);
                float4 v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = __ldg(v4 + i);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    amax = fmaxf(fmaxf(amax, fmaxf(fabsf(v[i].x), fabsf(v[i].y))), fmaxf(fabsf(v[i].z), fabsf(v[i].w)));
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        if (lane == 0) s.wmax[warp] = amax;
        __syncthreads();
        float m = s.wmax[lane & (I4_WARPS - 1)];
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        // binary32 exponent field of the largest magnitude (0 or a non-finite value: no scaling)
        const int ef = (int)((__float_as_uint(m) >> 23) & 0xffu);
        const int e = (ef == 0 || ef == 255) ? 0 : max(-100, min(100, 141 - ef));   // 2^e * m lies in [2^14, 2^15)
        scale_up = __uint_as_float((uint32_t)(127 + e) << 23);
        scale_down = __uint_as_float((uint32_t)(127 - e) << 23);
    }

    // binary32 sums of this lane: tile m, fragment rows g and g + 8, still split over the four
    // groups of a quad (lane's t)
    float acc[8][2];
#pragma unroll
    for (int m = 0; m < 8; ++m) acc[m][0] = acc[m][1] = 0.f;
    const char *wbase = p.W + (size_t)gchunk * 64 + g * 8;
    const uint16_t *sbase = p.scales + (size_t)gchunk * 128 + g * 8;

    for (int round_begin = r_begin; round_begin < r_end; round_begin += I4_ROUND_ROWS) {
        const int n_rows = min(r_end - round_begin, I4_ROUND_ROWS);
        if (round_begin != r_begin) __syncthreads();
        // ---- 2. the round's rows in rank order; clear the K-block tables ----
        {
            const int lo_rank = round_begin, hi_rank = round_begin + n_rows;
            for (int w = tid; w < p.mask_words; w += I4_THREADS) {
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
            uint4 *z = reinterpret_cast<uint4 *>(&s.bt[0][0][0]);
            for (int i = tid; i < (int)(sizeof(s.bt) / 16); i += I4_THREADS) z[i] = make_uint4(0u, 0u, 0u, 0u);
            uint4 *o = reinterpret_cast<uint4 *>(&s.kb_off[0][0]);
            for (int i = tid; i < (int)(sizeof(s.kb_off) / 16); i += I4_THREADS) o[i] = make_uint4(I4_PAD, I4_PAD, I4_PAD, I4_PAD);
            if (tid < I4_MAX_QUADS) s.qstart[tid] = s.qend[tid] = 0;
        }
        __syncthreads();
        // the scale rows of the round's groups for this segment go to shared memory if they fit
        // (loads issued here, stored after the tables are built)
        const int grp_first = 4 * (s.idx[0] >> 9);
        const int grp_count_all = min(4 * (s.idx[n_rows - 1] >> 9) + 4, n_groups) - grp_first;
        const int pieces_per_group = seg_chunks * 16;               // 16-byte pieces of a group's segment
        const int grp_staged = grp_count_all * pieces_per_group <= I4_STAGE_LOADS * I4_THREADS ? grp_count_all : 0;
        uint4 stage[I4_STAGE_LOADS];
#pragma unroll
        for (int i = 0; i < I4_STAGE_LOADS; ++i) {
            const int piece = tid + i * I4_THREADS;
            stage[i] = make_uint4(0u, 0u, 0u, 0u);
            if (piece < grp_staged * pieces_per_group) {
                const int gi = piece / pieces_per_group, o = (piece % pieces_per_group) * 8;
                if ((size_t)slab * seg_elems + o < p.scale_row_elems)
                    stage[i] = __ldg(reinterpret_cast<const uint4 *>(p.scales + (size_t)(grp_first + gi) * p.scale_row_elems +
                                                                     (size_t)slab * seg_elems + o));
            }
        }
        // ---- 3. where each quad (four scale groups = 512 columns) starts and ends in the list ----
        for (int r = tid; r < n_rows; r += I4_THREADS) {
            const int q = s.idx[r] >> 9;
            if (r == 0 || (s.idx[r - 1] >> 9) != q) s.qstart[q] = r;
            if (r == n_rows - 1 || (s.idx[r + 1] >> 9) != q) s.qend[q] = r + 1;
        }
        __syncthreads();
        if (warp == 0) {
            // K-blocks before each quad (a quad's rows are padded to a multiple of 16)
            int total = 0;
            for (int q0 = 0; q0 < I4_MAX_QUADS; q0 += 32) {
                const int q = q0 + lane;
                const int nb = q < I4_MAX_QUADS ? (s.qend[q] - s.qstart[q] + 15) >> 4 : 0;
                int incl = nb;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    int n = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += n;
                }
                if (q < I4_MAX_QUADS) s.qblk[q] = total + incl - nb;
                total += __shfl_sync(0xffffffffu, incl, 31);
            }
            if (lane == 0) s.n_kb = total;
        }
        __syncthreads();
        // ---- 4. the K-block tables: row address and B^T entries of every slot ----
        for (int r = tid; r < n_rows; r += I4_THREADS) {
            const int idx = s.idx[r], q = idx >> 9;
            const int within = r - s.qstart[q];
            const int kb = s.qblk[q] + (within >> 4), slot = within & 15;
            const uint32_t row = p.loc ? (uint32_t)p.loc[idx] : (uint32_t)idx;
            s.kb_off[kb][slot] = row * (uint32_t)(p.row_bytes >> 4);
            if (slot == 0) s.kb_quad[kb] = q;
            const float xs = __ldg(p.v + idx) * scale_up;
            const __half hi = __float2half_rn(xs);
            const __half lo = __float2half_rn(xs - __half2float(hi));
            const int c = (idx >> 7) & 3;
            s.bt[kb][2 * c][slot] = hi;
            s.bt[kb][2 * c + 1][slot] = lo;
        }
#pragma unroll
        for (int i = 0; i < I4_STAGE_LOADS; ++i) {
            const int piece = tid + i * I4_THREADS;
            if (piece < grp_staged * pieces_per_group) reinterpret_cast<uint4 *>(s_scale)[piece] = stage[i];
        }
        __syncthreads();
        const int n_kb = s.n_kb;

        // ---- 5. stream: warp (chunk, kgroup) takes the K-blocks kgroup, kgroup + kgroups, ... of
        //         its chunk; accumulators of the current quad in d[], flushed when the quad changes ----
        float d[9][4];
#pragma unroll
        for (int m = 0; m < 9; ++m) d[m][0] = d[m][1] = d[m][2] = d[m][3] = 0.f;
        int cur_quad = -1;
        uint4 sc0 = make_uint4(0u, 0u, 0u, 0u), sc1 = sc0;      // scales of group 4 * quad + t, rows g and g + 8

        auto flush = [&]() {
            const float x8 = -8.0f * (d[8][0] + d[8][1]);           // -8 * sum of the group's values (hi + lo)
            const uint32_t w0[4] = {sc0.x, sc0.y, sc0.z, sc0.w}, w1[4] = {sc1.x, sc1.y, sc1.z, sc1.w};
#pragma unroll
            for (int mp = 0; mp < 4; ++mp) {
                // tiles 2 mp (lower nibble of a byte: codes scaled by 2^-24) and 2 mp + 1 (upper: 2^-20)
                const float2 s0 = __half22float2(*reinterpret_cast<const __half2 *>(&w0[mp]));
                const float2 s1 = __half22float2(*reinterpret_cast<const __half2 *>(&w1[mp]));
                acc[2 * mp][0] = fmaf(s0.x * scale_down, fmaf(d[2 * mp][0] + d[2 * mp][1], 16777216.0f, x8), acc[2 * mp][0]);
                acc[2 * mp][1] = fmaf(s1.x * scale_down, fmaf(d[2 * mp][2] + d[2 * mp][3], 16777216.0f, x8), acc[2 * mp][1]);
                acc[2 * mp + 1][0] = fmaf(s0.y * scale_down, fmaf(d[2 * mp + 1][0] + d[2 * mp + 1][1], 1048576.0f, x8), acc[2 * mp + 1][0]);
                acc[2 * mp + 1][1] = fmaf(s1.y * scale_down, fmaf(d[2 * mp + 1][2] + d[2 * mp + 1][3], 1048576.0f, x8), acc[2 * mp + 1][1]);
            }
#pragma unroll
            for (int m = 0; m < 9; ++m) d[m][0] = d[m][1] = d[m][2] = d[m][3] = 0.f;
        };

        if (chunk_ok) {
            // this warp's K-blocks: a contiguous range (so that it meets few quads and flushes
            // seldom); I4_U of them in flight: the loads of block j + I4_U go out as soon as block j's
            // registers have been used
            uint2 raw[I4_U][4];
            auto issue = [&](uint2 (&r)[4], int kb, int kb_end) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    r[q] = make_uint2(0u, 0u);
                    if (kb < kb_end) {
                        const uint32_t off = s.kb_off[kb][2 * t + (q & 1) + 8 * (q >> 1)];
                        if (off != I4_PAD) r[q] = __ldcs(reinterpret_cast<const uint2 *>(wbase + (size_t)off * 16));
                    }
                }
            };
            const int kb_lo = (kgroup * n_kb) / kgroups, kb_hi = ((kgroup + 1) * n_kb) / kgroups;
#pragma unroll
            for (int u = 0; u < I4_U; ++u) issue(raw[u], kb_lo + u, kb_hi);
            for (int kb0 = kb_lo; kb0 < kb_hi; kb0 += I4_U) {
#pragma unroll
                for (int u = 0; u < I4_U; ++u) {
                    const int kb = kb0 + u;
                    if (kb >= kb_hi) break;
                    const int quad = s.kb_quad[kb];
                    if (quad != cur_quad) {
                        if (cur_quad >= 0) flush();
                        cur_quad = quad;
                        const int grp = 4 * quad + t;
                        sc0 = sc1 = make_uint4(0u, 0u, 0u, 0u);
                        if (grp < n_groups) {
                            if (grp - grp_first < grp_staged) {
                                const uint16_t *sp = s_scale + (size_t)(grp - grp_first) * seg_elems + chunk * 128 + g * 8;
                                sc0 = *reinterpret_cast<const uint4 *>(sp);
                                sc1 = *reinterpret_cast<const uint4 *>(sp + 64);
                            } else {
                                const uint16_t *sp = sbase + (size_t)grp * p.scale_row_elems;
                                sc0 = __ldg(reinterpret_cast<const uint4 *>(sp));
                                sc1 = __ldg(reinterpret_cast<const uint4 *>(sp + 64));
                            }
                        }
                    }
                    const uint32_t b0 = *reinterpret_cast<const uint32_t *>(&s.bt[kb][g][2 * t]);
                    const uint32_t b1 = *reinterpret_cast<const uint32_t *>(&s.bt[kb][g][2 * t + 8]);
#pragma unroll
                    for (int bi = 0; bi < 4; ++bi) {
                        // byte bi of words g / g + 8 of rows (2t, 2t+1) and (2t+8, 2t+9): tiles 2 bi, 2 bi + 1
                        const uint32_t sel = bi | (bi << 4) | ((4 + bi) << 8) | ((4 + bi) << 12);
                        const uint32_t p0 = __byte_perm(raw[u][0].x, raw[u][1].x, sel);
                        const uint32_t p1 = __byte_perm(raw[u][0].y, raw[u][1].y, sel);
                        const uint32_t p2 = __byte_perm(raw[u][2].x, raw[u][3].x, sel);
                        const uint32_t p3 = __byte_perm(raw[u][2].y, raw[u][3].y, sel);
                        mma_f16(d[2 * bi], p0 & 0x000f000fu, p1 & 0x000f000fu, p2 & 0x000f000fu, p3 & 0x000f000fu, b0, b1);
                        mma_f16(d[2 * bi + 1], p0 & 0x00f000f0u, p1 & 0x00f000f0u, p2 & 0x00f000f0u, p3 & 0x00f000f0u, b0, b1);
                    }
                    mma_f16(d[8], 0x3c003c00u, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u, b0, b1);
                    issue(raw[u], kb + I4_U, kb_hi);
                }
            }
            if (cur_quad >= 0) flush();                             // the round's scale differs from the next one's
        }
    }
    DIP_TRACE_MAX(p.tr, 3);            // streaming done

    // ---- 6. a lane's sums of the four groups, then the K-groups of the CTA, in fixed order ----
#pragma unroll
    for (int m = 0; m < 8; ++m)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float v = acc[m][r];
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            if (t == 0) s_sums[kgroup * seg_elems + chunk * 128 + m * 16 + g + 8 * r] = v;
        }
    __syncthreads();
    float *dst = (nparts > 1 || p.defer) ? p.partials + ((size_t)(p.part_base + part) * gridDim.x + slab) * seg_elems : s_total;
    for (int e = tid; e < seg_elems; e += I4_THREADS) {
        float v = 0.f;
        for (int k = 0; k < kgroups; ++k) v += s_sums[k * seg_elems + e];
        dst[e] = v;
    }
    // ---- 7. the row parts ----
    if (p.defer) {
        DIP_TRACE_MAX(p.tr, 2);
        return;                        // the caller adds the parts of two launches with a kernel of its own
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
        // all parts' loads in flight together: R = I4_THREADS / (seg_elems / 4) threads share four
        // outputs, thread r of them adds the parts r, r + R, ...; the R sums meet in shared memory in
        // order of r
        const size_t stride = (size_t)gridDim.x * seg_elems;
        constexpr int n4 = seg_elems / 4, R = I4_THREADS / n4;
        const int e4 = tid % n4, r = tid / n4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        const float *pp = p.partials + (size_t)slab * seg_elems + 4 * e4;
        for (int q0 = r; q0 < nparts; q0 += 8 * R) {
            float4 a[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                a[q] = q0 + q * R < nparts ? __ldcg(reinterpret_cast<const float4 *>(pp + (size_t)(q0 + q * R) * stride))
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int q = 0; q < 8; ++q) { v.x += a[q].x; v.y += a[q].y; v.z += a[q].z; v.w += a[q].w; }
        }
        *reinterpret_cast<float4 *>(s_sums + (size_t)r * seg_elems + 4 * e4) = v;
        __syncthreads();
        for (int e = tid; e < seg_elems; e += I4_THREADS) {
            float t4 = 0.f;
#pragma unroll
            for (int k = 0; k < R; ++k) t4 += s_sums[(size_t)k * seg_elems + e];
            s_total[e] = t4;
        }
        if (tid == 0) p.tickets[slab] = 0;                      // ready for the next launch
    }
    __syncthreads();
    // ---- 8. epilogue: outputs in their logical order ----
    if (WHICH == 0) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int o = tid + i * I4_THREADS;
            const int c = o >> 6, e = o & 63;
            const int j = (slab * seg_chunks + c) * 64 + e;
            if (o >= seg_chunks * 64 || j >= p.d_out) continue;
            const float r = silu_f32(s_total[c * 128 + e]) * s_total[c * 128 + 64 + e];
            p.out[j] = r;
            if (p.key_coarse) {
                // what the select would form from h_j and the stamp, cut to its top 16 bits
                float a = fabsf(r);
                if (p.key_stamp) a = __fmul_rn(a, key_stamp[i] >= 0 ? 1.0f : p.key_gamma);
                p.key_coarse[j] = (uint16_t)((__float_as_uint(a) & 0x7fffffffu) >> 16);
            }
        }
    } else {
        for (int o = tid; o < seg_elems; o += I4_THREADS) {
            const int j = slab * seg_elems + o;
            if (j < p.d_out) p.out[j] = s_total[o];
        }
    }
    DIP_TRACE_MAX(p.tr, 2);
}

}  // namespace

// Segment width and row parts: one CTA per SM.  The CTA that completes a segment adds up
// nparts x (segment outputs) partial sums alone, so the segment is narrowed (and the warps of a
// CTA split the K-blocks instead) until that tail is short.
namespace {

template <int WHICH, int SEGC>
dip_status launch_int4(dip_ctx *ctx, GemvParams &p, int n_chunks, int n_slabs, int nparts, size_t smem, cudaStream_t stream)
{
    static dip_per_device_once once;
    constexpr size_t smem_max = sizeof(I4Smem) + (size_t)2 * I4_WARPS * 128 * sizeof(float) + I4_SCALE_BYTES;
    DIP_CUDA_TRY(ctx, dip_raise_smem_limit(once, ctx->device, gemv_int4_kernel<WHICH, SEGC>, smem_max));
    DIP_CUDA_TRY(ctx, dip_launch_pdl(gemv_int4_kernel<WHICH, SEGC>, dim3(n_slabs, nparts), dim3(I4_THREADS), smem, stream, p,
                                     n_chunks));
    return DIP_OK;
}

template <int WHICH>
dip_status launch_int4_seg(dip_ctx *ctx, GemvParams &p, int seg_chunks, int n_chunks, int n_slabs, int nparts, size_t smem,
                           cudaStream_t stream)
{
    switch (seg_chunks) {
    case 16: return launch_int4<WHICH, 16>(ctx, p, n_chunks, n_slabs, nparts, smem, stream);
    case 8: return launch_int4<WHICH, 8>(ctx, p, n_chunks, n_slabs, nparts, smem, stream);
    case 4: return launch_int4<WHICH, 4>(ctx, p, n_chunks, n_slabs, nparts, smem, stream);
    case 2: return launch_int4<WHICH, 2>(ctx, p, n_chunks, n_slabs, nparts, smem, stream);
    default: return launch_int4<WHICH, 1>(ctx, p, n_chunks, n_slabs, nparts, smem, stream);
    }
}

}  // namespace

dip_status dip_launch_gemv_int4(dip_ctx *ctx, GemvParams &p, int which, int n_kept_max, int mode, cudaStream_t stream)
{
    const int n_chunks = (int)(p.row_bytes / 64);
    int seg_chunks = 16, n_slabs = 0, nparts = 1;
    // wide rows: the widest segment with which the segments alone occupy most of the SMs, so that
    // one CTA sees all kept rows of its segment and nothing is combined across CTAs
    bool whole = false;
    for (int sc = 16; sc >= 1 && !whole; sc >>= 1) {
        const int ns = (n_chunks + sc - 1) / sc;
        if (ns <= ctx->sm_count && 5 * ns >= 3 * ctx->sm_count) {
            seg_chunks = sc;
            n_slabs = ns;
            whole = true;
        }
    }
    for (; !whole; seg_chunks >>= 1) {
        n_slabs = (n_chunks + seg_chunks - 1) / seg_chunks;
        nparts = ctx->sm_count / n_slabs;
        if (nparts > n_kept_max / 16) nparts = n_kept_max / 16;     // at least one K-block of rows per part
        if (nparts < 1) nparts = 1;
        const long long tail = (long long)nparts * seg_chunks * 128 * 4;
        if (tail <= 49152 || seg_chunks == 1) break;
    }
    if (n_slabs > ctx->n_tickets) return DIP_ERR_WORKSPACE;
    const int seg_elems = seg_chunks * 128;
    const int total_parts = mode ? 2 * nparts : nparts;
    if ((nparts > 1 || mode) && (size_t)total_parts * n_slabs * seg_elems > ctx->partials_floats) return DIP_ERR_WORKSPACE;
    p.defer = mode != 0;
    p.part_base = mode == 2 ? nparts : 0;
    const int kgroups = I4_WARPS / seg_chunks;
    const size_t smem = sizeof(I4Smem) + (size_t)(kgroups + 1) * seg_elems * sizeof(float) + I4_SCALE_BYTES;
    const dip_status st = which == 0 ? launch_int4_seg<0>(ctx, p, seg_chunks, n_chunks, n_slabs, nparts, smem, stream)
                                     : launch_int4_seg<1>(ctx, p, seg_chunks, n_chunks, n_slabs, nparts, smem, stream);
    if (st != DIP_OK) return st;
    if (mode == 2)
        return dip_launch_combine_parts(ctx, which, total_parts, n_slabs, 1, seg_elems, 64, 1, p.d_out, p.out, stream);
    return DIP_OK;
}
