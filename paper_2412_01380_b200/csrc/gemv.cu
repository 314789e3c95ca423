// Sparse vector-matrix products over the kept weight columns (Eq. 3 with the masks of Eq. 7-8).
//
// A packed matrix stores column i of W as row i (see dip.h), so a kept column is one
// contiguous row.  The kernel is a gather-GEMV: grid = (output slabs) x (row parts).
// A warp reads one kept row's slab segment per step, 32 bytes per lane (two 16-byte loads,
// a full 1 KB contiguous piece per warp), and keeps E binary32 accumulators per lane and
// token.  The warps of a CTA take different rows; their sums are combined through shared
// memory in warp order, the row parts through a scratch buffer in part order by the last
// CTA to arrive at the slab (an arrival counter).  The order of every sum is fixed, so the
// result is bit-reproducible; no floating-point atomics are used.
//
// which = 0 (gate/up bundle): a lane's 32 bytes are [gate chunk | up chunk] of the same
// outputs, so the silu(gate) * up epilogue (Eq. 2) needs no data exchange.
// which = 1 (down): plain sums.
#include "common.cuh"

namespace {

constexpr int GV_THREADS = 256;
constexpr int GV_WARPS = GV_THREADS / 32;
constexpr int GV_UNROLL = 8;     // rows in flight per warp

template <int WT> struct WTraits;
template <> struct WTraits<DIP_W_F32>  { static constexpr int E = 8;  static constexpr int BYTES = 32; };
template <> struct WTraits<DIP_W_BF16> { static constexpr int E = 16; static constexpr int BYTES = 32; };

struct Raw32 { uint4 a, b; };

__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ Raw32 ld_row32(const char *p)
{
    Raw32 r;
    r.a = ld_stream16(p);
    r.b = ld_stream16(p + 16);
    return r;
}

template <int WT> __device__ __forceinline__ void decode(const Raw32 &r, float (&w)[WTraits<WT>::E]);

template <> __device__ __forceinline__ void decode<DIP_W_F32>(const Raw32 &r, float (&w)[8])
{
    w[0] = __uint_as_float(r.a.x); w[1] = __uint_as_float(r.a.y);
    w[2] = __uint_as_float(r.a.z); w[3] = __uint_as_float(r.a.w);
    w[4] = __uint_as_float(r.b.x); w[5] = __uint_as_float(r.b.y);
    w[6] = __uint_as_float(r.b.z); w[7] = __uint_as_float(r.b.w);
}

// bfloat16 is the upper half of a binary32: widening is a shift or a mask.
template <> __device__ __forceinline__ void decode<DIP_W_BF16>(const Raw32 &r, float (&w)[16])
{
    const uint32_t u[8] = {r.a.x, r.a.y, r.a.z, r.a.w, r.b.x, r.b.y, r.b.z, r.b.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        w[2 * i] = __uint_as_float(u[i] << 16);
        w[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
}

struct GemvParams {
    const char *W;            // packed rows
    size_t row_bytes;         // bytes of one packed row
    int row_elems;            // elements of one packed row (2*d_ff or d_model)
    const float *v;           // [batch][d_in]
    int d_in;
    const int32_t *kept_idx;
    int n_kept;
    const int32_t *n_kept_dev;
    const uint32_t *mask_bits; // [batch][ceil(d_in/32)] or nullptr
    int mask_words;
    float *out;               // [batch][d_out]
    int d_out;
    int batch;                // tokens in this launch (<= BT)
    float *partials;
    unsigned int *tickets;
};

__device__ __forceinline__ float silu_f32(float g) { return g / (1.0f + expf(-g)); }

template <int WT, int WHICH, int BT>
__global__ void __launch_bounds__(GV_THREADS)
gemv_kernel(const GemvParams p)
{
    constexpr int E = WTraits<WT>::E;
    constexpr int SLAB = 32 * E;                              // packed elements per slab
    constexpr int OUT_PER_SLAB = WHICH == 0 ? SLAB / 2 : SLAB;
    constexpr int C = E / 2;                                  // gate/up chunk (outputs per lane)
    __shared__ float s_red[GV_WARPS][SLAB];
    __shared__ float s_sum[BT][SLAB];
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slab = blockIdx.x, part = blockIdx.y, nparts = gridDim.y;
    const int n_rows = p.n_kept_dev ? *p.n_kept_dev : p.n_kept;
    const int r_begin = (int)(((long long)part * n_rows) / nparts);
    const int r_end = (int)(((long long)(part + 1) * n_rows) / nparts);

    const int elem0 = slab * SLAB + lane * E;                 // first packed element of this lane
    const bool lane_ok = elem0 < p.row_elems;
    const char *wbase = p.W + (size_t)(lane_ok ? elem0 : 0) * (WTraits<WT>::BYTES / E);

    float acc[BT][E];
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[b][e] = 0.f;

    // this warp's rows: r_begin + warp, + GV_WARPS, ...
    const int n_mine = (r_end - r_begin - warp + GV_WARPS - 1) / GV_WARPS;
    for (int c0 = 0; c0 < n_mine; c0 += 32) {
        // lane l stages row c0 + l of this warp: its column index and the tokens' values
        int my_idx = 0;
        float my_v[BT];
#pragma unroll
        for (int b = 0; b < BT; ++b) my_v[b] = 0.f;
        if (c0 + lane < n_mine) {
            my_idx = p.kept_idx[r_begin + warp + (c0 + lane) * GV_WARPS];
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                if (b < p.batch) {
                    bool on = true;
                    if (p.mask_bits)
                        on = (p.mask_bits[(size_t)b * p.mask_words + (my_idx >> 5)] >> (my_idx & 31)) & 1u;
                    my_v[b] = on ? p.v[(size_t)b * p.d_in + my_idx] : 0.f;
                }
            }
        }
        const int n_here = min(32, n_mine - c0);
        for (int j0 = 0; j0 < n_here; j0 += GV_UNROLL) {
            Raw32 raw[GV_UNROLL];
#pragma unroll
            for (int u = 0; u < GV_UNROLL; ++u) {
                int idx = __shfl_sync(0xffffffffu, my_idx, (j0 + u) & 31);
                if (j0 + u < n_here && lane_ok)
                    raw[u] = ld_row32(wbase + (size_t)idx * p.row_bytes);
                else
                    raw[u].a = raw[u].b = make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < GV_UNROLL; ++u) {
                float w[E];
                decode<WT>(raw[u], w);
#pragma unroll
                for (int b = 0; b < BT; ++b) {
                    float xv = __shfl_sync(0xffffffffu, my_v[b], (j0 + u) & 31);
                    if (j0 + u >= n_here) xv = 0.f;
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[b][e] = fmaf(w[e], xv, acc[b][e]);
                }
            }
        }
    }

    // combine the warps in warp order, one token at a time
#pragma unroll
    for (int b = 0; b < BT; ++b) {
#pragma unroll
        for (int e = 0; e < E; ++e) s_red[warp][lane * E + e] = acc[b][e];
        __syncthreads();
        for (int t = tid; t < SLAB; t += GV_THREADS) {
            float sum = 0.f;
#pragma unroll
            for (int w = 0; w < GV_WARPS; ++w) sum += s_red[w][t];
            s_sum[b][t] = sum;
        }
        __syncthreads();
    }

    if (nparts > 1) {
        float *my_part = p.partials + ((size_t)part * gridDim.x + slab) * (BT * SLAB);
        for (int t = tid; t < BT * SLAB; t += GV_THREADS) my_part[t] = s_sum[t / SLAB][t % SLAB];
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            unsigned prev = atomicAdd(&p.tickets[slab], 1u);
            s_last = prev == (unsigned)(nparts - 1);
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
    }

    // epilogue by the CTA that completes the slab
    for (int t = tid; t < BT * OUT_PER_SLAB; t += GV_THREADS) {
        const int b = t / OUT_PER_SLAB, o = t % OUT_PER_SLAB;
        const int j = slab * OUT_PER_SLAB + o;
        if (b >= p.batch || j >= p.d_out) continue;
        int e0, e1 = 0;
        if (WHICH == 0) {
            e0 = (o / C) * E + (o % C);      // gate element of output o
            e1 = e0 + C;                     // matching up element
        } else {
            e0 = o;
        }
        float s0 = 0.f, s1 = 0.f;
        if (nparts > 1) {
            for (int q = 0; q < nparts; ++q) {
                const float *pp = p.partials + ((size_t)q * gridDim.x + slab) * (BT * SLAB) + b * SLAB;
                s0 += __ldcg(pp + e0);
                if (WHICH == 0) s1 += __ldcg(pp + e1);
            }
        } else {
            s0 = s_sum[b][e0];
            if (WHICH == 0) s1 = s_sum[b][e1];
        }
        p.out[(size_t)b * p.d_out + j] = WHICH == 0 ? silu_f32(s0) * s1 : s0;
    }
    if (nparts > 1 && tid == 0) p.tickets[slab] = 0;   // ready for the next launch
}

}  // namespace

namespace {

template <int WT, int WHICH, int BT>
dip_status launch_one(dip_ctx *ctx, GemvParams &p, int n_kept_max, cudaStream_t stream)
{
    constexpr int SLAB = 32 * WTraits<WT>::E;
    const int n_slabs = (p.row_elems + SLAB - 1) / SLAB;
    if (n_slabs > ctx->n_tickets) return DIP_ERR_WORKSPACE;
    // enough CTAs to fill the device a few times over, but no part thinner than a few rows per warp
    const int target = ctx->sm_count * 4;
    int nparts = (target + n_slabs - 1) / n_slabs;
    const int max_by_rows = n_kept_max / (2 * GV_WARPS);
    if (nparts > max_by_rows) nparts = max_by_rows;
    const size_t per_part = (size_t)n_slabs * BT * SLAB;
    if ((size_t)nparts * per_part > ctx->partials_floats) nparts = (int)(ctx->partials_floats / per_part);
    if (nparts < 1) nparts = 1;
    dim3 grid(n_slabs, nparts);
    gemv_kernel<WT, WHICH, BT><<<grid, GV_THREADS, 0, stream>>>(p);
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}

template <int WT, int WHICH>
dip_status launch_bt(dip_ctx *ctx, GemvParams &p, int n_kept_max, cudaStream_t stream)
{
    switch (p.batch) {
    case 1: return launch_one<WT, WHICH, 1>(ctx, p, n_kept_max, stream);
    case 2: return launch_one<WT, WHICH, 2>(ctx, p, n_kept_max, stream);
    default: return launch_one<WT, WHICH, 4>(ctx, p, n_kept_max, stream);
    }
}

}  // namespace

dip_status dip_launch_gemv(dip_ctx *ctx, const dip_mlp_weights *w, int which,
                           const float *v, int batch,
                           const int32_t *kept_idx, int n_kept_max, const int32_t *n_kept_dev,
                           const uint32_t *mask_bits, float *out, cudaStream_t stream)
{
    if (w->wtype != DIP_W_F32 && w->wtype != DIP_W_BF16) return DIP_ERR_UNSUPPORTED;
    const int elem_bytes = w->wtype == DIP_W_F32 ? 4 : 2;
    GemvParams p;
    p.W = (const char *)(which == 0 ? w->gate_up : w->down);
    p.row_elems = which == 0 ? 2 * w->d_ff : w->d_model;
    p.row_bytes = (size_t)p.row_elems * elem_bytes;
    p.d_in = which == 0 ? w->d_model : w->d_ff;
    p.d_out = which == 0 ? w->d_ff : w->d_model;
    p.kept_idx = kept_idx;
    p.n_kept = n_kept_max;
    p.n_kept_dev = n_kept_dev;
    p.mask_words = (p.d_in + 31) / 32;
    p.partials = ctx->partials;
    p.tickets = ctx->tickets;
    // tokens go through in groups of at most four (accumulators live in registers)
    for (int b0 = 0; b0 < batch; b0 += 4) {
        p.batch = batch - b0 < 4 ? batch - b0 : 4;
        p.v = v + (size_t)b0 * p.d_in;
        p.mask_bits = mask_bits ? mask_bits + (size_t)b0 * p.mask_words : nullptr;
        p.out = out + (size_t)b0 * p.d_out;
        dip_status st;
        if (w->wtype == DIP_W_F32)
            st = which == 0 ? launch_bt<DIP_W_F32, 0>(ctx, p, n_kept_max, stream)
                            : launch_bt<DIP_W_F32, 1>(ctx, p, n_kept_max, stream);
        else
            st = which == 0 ? launch_bt<DIP_W_BF16, 0>(ctx, p, n_kept_max, stream)
                            : launch_bt<DIP_W_BF16, 1>(ctx, p, n_kept_max, stream);
        if (st != DIP_OK) return st;
    }
    return DIP_OK;
}
