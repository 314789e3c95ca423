// Two tokens, F32 / BF16 weights: the product over the union of the tokens' kept rows (Eq. 3 with one
// mask of Eq. 7-8 per token) with plain loads, as gemv_direct_kernel does it for one token.  A weight
// byte is read once and multiplied into every token that keeps its row.  A CTA owns a 512-byte
// segment of the packed rows and a share of the union's rows; a lane keeps BT x E sums; a token that
// drops a row enters it with the value zero.  With two tokens the sums still fit the 64 registers of
// a 1024-thread block (32 warps x 4 loads in flight); with four they do not, and 16 warps x 8 loads
// measured 133 us per layer-step at Phi-3-Medium shapes against 103 us on the tensor-core kernel,
// which therefore takes three tokens and more.
#include "gemv_common.cuh"

namespace {

constexpr int GB_SEG = 512;

constexpr int GB_MAX_ROWS = 8192;          // rows of the union per round (a part's share of them)

struct __align__(16) GemvBtSmem {
    uint16_t idx[GB_MAX_ROWS];
    unsigned char tok[GB_MAX_ROWS];        // bit b: token b keeps the row
    uint32_t words[DIP_MAX_D / 32];        // the union of the masks
    int pre[DIP_MAX_D / 32];
    int wsum[GV_SCAN_THREADS / 32];
    int n_total;
    int last;
};
// after GemvBtSmem (dynamic): float red[NW][BT][SLAB], float sum[BT][SLAB]

template <int WT, int WHICH, int BT, int NW, int U>
__global__ void __launch_bounds__(NW * 32, 1)
gemv_direct_bt_kernel(const GemvParams p)
{
    constexpr int E = WTraits<WT>::E;
    constexpr int SLAB = 32 * E;                              // packed elements per segment
    constexpr int OUT_PER_SLAB = WHICH == 0 ? SLAB / 2 : SLAB;
    constexpr int C = WTraits<WT>::C;
    constexpr int THREADS = NW * 32;
    static_assert(THREADS >= GV_SCAN_THREADS && E <= 8 && BT <= 8, "");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    GemvBtSmem &s = *reinterpret_cast<GemvBtSmem *>(smem_raw);
    float *s_red = reinterpret_cast<float *>(smem_raw + sizeof(GemvBtSmem));     // [NW][BT][SLAB]
    float *s_sum = s_red + NW * BT * SLAB;                                       // [BT][SLAB]

    DIP_TRACE_MIN(p.tr, 0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slab = blockIdx.x, part = blockIdx.y, nparts = gridDim.y;
    const size_t byte_off = (size_t)slab * GB_SEG + lane * 16;
    const bool lane_ok = byte_off < p.row_bytes;
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(p.tr, 1);
    dip_launch_dependents();

    // ---- 1. the union of the masks and its popcount prefix ----
    if (tid < GV_SCAN_THREADS) {
        uint32_t u[4] = {0u, 0u, 0u, 0u};
        int c = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int w = 4 * tid + j;
            if (w < p.mask_words) {
#pragma unroll
                for (int b = 0; b < BT; ++b)
                    if (b < p.batch) u[j] |= p.mask_bits[(size_t)b * p.mask_words + w];
            }
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

    float acc[BT][E];
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[b][e] = 0.f;
    const char *base = p.W + byte_off;

    for (int round_begin = r_begin; round_begin < r_end; round_begin += GB_MAX_ROWS) {
        const int n_rows = min(r_end - round_begin, GB_MAX_ROWS);
        if (round_begin != r_begin) __syncthreads();
        // ---- 2. the round's rows in rank order, each with the set of tokens that keep it ----
        {
            const int lo_rank = round_begin, hi_rank = round_begin + n_rows;
            for (int w = tid; w < p.mask_words; w += THREADS) {
                uint32_t u = s.words[w];
                int rank = s.pre[w];
                if (rank >= hi_rank || rank + __popc(u) <= lo_rank) continue;
                uint32_t mb[BT];
#pragma unroll
                for (int b = 0; b < BT; ++b) mb[b] = b < p.batch ? p.mask_bits[(size_t)b * p.mask_words + w] : 0u;
                while (u) {
                    const int bit = __ffs(u) - 1;
                    u &= u - 1;
                    if (rank >= lo_rank && rank < hi_rank) {
                        unsigned tk = 0u;
#pragma unroll
                        for (int b = 0; b < BT; ++b) tk |= ((mb[b] >> bit) & 1u) << b;
                        s.idx[rank - lo_rank] = (uint16_t)(w * 32 + bit);
                        s.tok[rank - lo_rank] = (unsigned char)tk;
                    }
                    ++rank;
                }
            }
        }
        __syncthreads();
        // ---- 3. stream: warp w takes rows w, w + NW, ...; U of them in flight per lane ----
        for (int r0 = warp; r0 < n_rows; r0 += NW * U) {
            uint4 q[U];
            float xv[U][BT];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = r0 + u * NW;
                q[u] = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int b = 0; b < BT; ++b) xv[u][b] = 0.f;
                if (r < n_rows) {
                    const int idx = s.idx[r];
                    const unsigned tk = s.tok[r];
                    if (lane_ok) q[u] = __ldcs(reinterpret_cast<const uint4 *>(base + (size_t)idx * p.row_bytes));
#pragma unroll
                    for (int b = 0; b < BT; ++b)
                        if ((tk >> b) & 1u) xv[u][b] = __ldg(p.v + (size_t)b * p.d_in + idx);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float w[E];
                decode16<WT>(q[u], w);
#pragma unroll
                for (int b = 0; b < BT; ++b)
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[b][e] = fmaf(w[e], xv[u][b], acc[b][e]);
            }
        }
    }
    DIP_TRACE_MAX(p.tr, 3);            // streaming done

    // ---- 4. the warps' sums, in warp order ----
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int e = 0; e < E; ++e) s_red[(warp * BT + b) * SLAB + lane * E + e] = acc[b][e];
    __syncthreads();
    for (int i = tid; i < BT * SLAB; i += THREADS) {
        const int b = i / SLAB, el = i % SLAB;
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) t += s_red[(w * BT + b) * SLAB + el];
        if (nparts > 1) p.partials[((size_t)part * gridDim.x + slab) * (BT * SLAB) + i] = t;
        else s_sum[i] = t;
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
        for (int i = tid; i < BT * SLAB; i += THREADS) {
            const size_t stride = (size_t)gridDim.x * (BT * SLAB);
            const float *pp = p.partials + (size_t)slab * (BT * SLAB) + i;
            float t = 0.f;
            for (int q0 = 0; q0 < nparts; q0 += 8) {
                float a[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) a[q] = q0 + q < nparts ? __ldcg(pp + (size_t)(q0 + q) * stride) : 0.f;
#pragma unroll
                for (int q = 0; q < 8; ++q) t += a[q];
            }
            s_sum[i] = t;
        }
        if (tid == 0) p.tickets[slab] = 0;                    // ready for the next launch
    }
    __syncthreads();
    // ---- 6. epilogue ----
    for (int i = tid; i < BT * OUT_PER_SLAB; i += THREADS) {
        const int b = i / OUT_PER_SLAB, o = i % OUT_PER_SLAB, j = slab * OUT_PER_SLAB + o;
        if (b < p.batch && j < p.d_out) {
            float r;
            if (WHICH == 0) {
                const int e0 = (o / C) * 2 * C + (o % C);     // gate element; its up element is C further
                r = silu_f32(s_sum[b * SLAB + e0]) * s_sum[b * SLAB + e0 + C];
            } else {
                r = s_sum[b * SLAB + o];
            }
            p.out[(size_t)b * p.d_out + j] = r;
            // top 16 bits of the rank key |h_j| for the select that follows (no cache with several tokens)
            if (WHICH == 0 && p.key_coarse)
                p.key_coarse[(size_t)b * p.d_out + j] = (uint16_t)((__float_as_uint(r) & 0x7fffffffu) >> 16);
        }
    }
    DIP_TRACE_MAX(p.tr, 2);
}

template <int WT, int WHICH, int BT, int NW, int U>
dip_status launch_cfg(dip_ctx *ctx, GemvParams &p, int n_kept_max, cudaStream_t stream)
{
    constexpr int SLAB = 32 * WTraits<WT>::E;
    const int n_slabs = (int)((p.row_bytes + GB_SEG - 1) / GB_SEG);
    int nparts = ctx->sm_count / n_slabs;
    if (nparts > n_kept_max) nparts = n_kept_max;
    if (nparts < 1) nparts = 1;
    if (n_slabs > ctx->n_tickets) return DIP_ERR_WORKSPACE;
    if (nparts > 1 && (size_t)nparts * n_slabs * BT * SLAB > ctx->partials_floats) return DIP_ERR_WORKSPACE;
    p.defer = 0;
    p.part_base = 0;
    const size_t smem = sizeof(GemvBtSmem) + sizeof(float) * (NW + 1) * BT * SLAB;
    static dip_per_device_once once;
    DIP_CUDA_TRY(ctx, dip_raise_smem_limit(once, ctx->device, gemv_direct_bt_kernel<WT, WHICH, BT, NW, U>, smem));
    DIP_CUDA_TRY(ctx, dip_launch_pdl(gemv_direct_bt_kernel<WT, WHICH, BT, NW, U>, dim3(n_slabs, nparts), dim3(NW * 32), smem,
                                     stream, p));
    return DIP_OK;
}

template <int WT, int WHICH>
dip_status launch_wt(dip_ctx *ctx, GemvParams &p, int n_kept_max, cudaStream_t stream)
{
    return launch_cfg<WT, WHICH, 2, 32, 4>(ctx, p, n_kept_max, stream);
}

}  // namespace

dip_status dip_launch_gemv_direct_bt(dip_ctx *ctx, GemvParams &p, int wtype, int which, int n_kept_max, cudaStream_t stream)
{
    if (p.batch != 2 || (wtype != DIP_W_F32 && wtype != DIP_W_BF16)) return DIP_ERR_UNSUPPORTED;
    if (wtype == DIP_W_F32)
        return which == 0 ? launch_wt<DIP_W_F32, 0>(ctx, p, n_kept_max, stream) : launch_wt<DIP_W_F32, 1>(ctx, p, n_kept_max, stream);
    return which == 0 ? launch_wt<DIP_W_BF16, 0>(ctx, p, n_kept_max, stream) : launch_wt<DIP_W_BF16, 1>(ctx, p, n_kept_max, stream);
}
