// One token, F32 / BF16 weights: a product kernel that builds its own mask.
//
// In a step, each product (Eq. 1-3) needs the top-k mask of its input (Eq. 7-8, or the cache-aware
// ranking of Algorithm 1), and a select kernel in front of it costs a kernel boundary, the mask's
// trip through global memory, and a device that idles while one CTA selects.  The select by one
// 15-bit histogram (select_core.cuh) is short enough for every CTA of the product to run it for
// itself - same code, same inputs, hence the same mask everywhere, with nothing to wait for -
// and to go straight on to its rows.  CTA 0 also writes the mask (and, for the gate/up input of a
// chained layer, the normalised x) to global memory for the cache update and the caller.  The
// mask is bit for bit the stand-alone select's, and the product is gemv_direct_kernel's: a CTA owns
// a 512-byte segment of the packed rows and a share of the kept rows, 32 warps x 4 loads in flight.
#include "gemv_common.cuh"
#include "select_core.cuh"

namespace {

constexpr int GF_SEG = 512;
constexpr int GF_NW = TK_THREADS / 32;     // 32 warps
constexpr int GF_U = 4;                    // loads in flight per lane
constexpr size_t GF_SMEM_LIMIT = (size_t)220 * 1024;   // dynamic shared memory a launch may ask for

struct FusedParams {
    // product
    const char *W;
    size_t row_bytes;
    int d_in, d_out;
    int n_slabs, nparts;
    float *out;
    float *partials;             // [nparts][n_slabs][segment elements]
    unsigned int *tickets;
    unsigned long long *tr;
    uint16_t *key_coarse;        // gate/up: top 16 bits of the rank keys of h (nullptr: not wanted)
    const int32_t *key_stamp;
    float key_gamma;
    // select
    const float *xa;             // gate/up: x, or the previous layer's x when xb is given; down: h
    const float *xb;             // gate/up, chained: the previous layer's y
    float *x_out;                // gate/up, chained: where CTA 0 writes x = (xa + xb) / rms(xa + xb)
    const uint16_t *coarse;      // down: top 16 bits of the rank keys of h
    int k;
    float gamma;
    const int32_t *stamp;        // cache state of this input (CA) or unused
    uint32_t *mask_out;
};

struct __align__(16) FusedSmem {
    TkFine fine;                           // the select's histogram; afterwards the warps' sums ([warp][lane * E + e])
    TkShared ts;
    unsigned int maskw[DIP_MAX_D / 32];    // the mask
    int wsum[GF_NW];
    int last;
    float sum[32 * 8];
};
static_assert(sizeof(float) * GF_NW * 32 * 8 <= sizeof(unsigned int) * TK_FINE_WORDS, "the warps' sums fit the histogram");

// This part's share of the rows in `words` (a bit set in shared memory, complete and visible), by
// rank, as a list in idx[]; returns the share's size.  One word per thread (DIP_MAX_D / 32 words at
// most); all threads call it; ends with a barrier.
__device__ __forceinline__ int list_rows(FusedSmem &s, const unsigned int *words, int mask_words, int d_in, int part,
                                         int nparts, uint16_t *idx)
{
    static_assert(DIP_MAX_D / 32 <= TK_THREADS, "one mask word per thread");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t u = tid < mask_words ? words[tid] : 0u;
    if (tid == mask_words - 1 && (d_in & 31)) u &= (1u << (d_in & 31)) - 1u;
    const int c = __popc(u);
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    if (lane == 31) s.wsum[warp] = incl;
    __syncthreads();
    int total;
    const int before = warp_array_prefix(s.wsum, warp, lane, total);
    int lo = 0, hi = total;
    if (nparts > 1) {
        // (part * total fits 32 bits: at most one part per SM, at most DIP_MAX_D rows)
        lo = (int)((unsigned)part * (unsigned)total / (unsigned)nparts);
        hi = (int)((unsigned)(part + 1) * (unsigned)total / (unsigned)nparts);
    }
    int rank = before + incl - c;
    if (rank < hi && rank + c > lo) {
        uint16_t *out = idx + (rank - lo);
        int col = tid * 32;
        while (u) {
            const int sh = __ffs(u);             // 1-based position of the next row's bit
            col += sh;
            u = sh < 32 ? u >> sh : 0u;
            if (rank >= lo && rank < hi) *out = (uint16_t)(col - 1);
            ++out;
            ++rank;
        }
    }
    __syncthreads();
    return hi - lo;
}

// acc += sum over rows idx[first], idx[first + stride], ... below n_rows of row segment x value,
// U rows in flight per lane.
template <int WT>
__device__ __forceinline__ void stream_rows(const uint16_t *idx, int first, int stride, int n_rows, const char *base,
                                            size_t row_bytes, bool lane_ok, const float *xsrc,
                                            float (&acc)[WTraits<WT>::E])
{
    constexpr int E = WTraits<WT>::E;
    for (int r0 = first; r0 < n_rows; r0 += stride * GF_U) {
        uint4 q[GF_U];
        float xv[GF_U];
#pragma unroll
        for (int u = 0; u < GF_U; ++u) {
            const int r = r0 + u * stride;
            q[u] = make_uint4(0u, 0u, 0u, 0u);
            xv[u] = 0.f;
            if (r < n_rows) {
                const int i = idx[r];
                if (lane_ok) q[u] = __ldcs(reinterpret_cast<const uint4 *>(base + (size_t)i * row_bytes));
                xv[u] = xsrc[i];
            }
        }
#pragma unroll
        for (int u = 0; u < GF_U; ++u) {
            float w[E];
            decode16<WT>(q[u], w);
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] = fmaf(w[e], xv[u], acc[e]);
        }
    }
}

// Block part * n_slabs + slab owns segment `slab`, row part `part`.  Dynamic shared memory:
// FusedSmem, then keys[] (d_in words rounded up to four: rank keys, later this CTA's row list),
// then for a chained gate/up input the d_in values of x.
template <int WT, int WHICH, bool CA, bool NORM>
__global__ void __launch_bounds__(TK_THREADS, 1)
gemv_fused_kernel(const FusedParams p)
{
    constexpr int E = WTraits<WT>::E;
    constexpr int SLAB = 32 * E;
    constexpr int OUT_PER_SLAB = WHICH == 0 ? SLAB / 2 : SLAB;
    constexpr int C = WTraits<WT>::C;
    extern __shared__ __align__(16) unsigned char dyn[];
    FusedSmem &s = *reinterpret_cast<FusedSmem *>(dyn);
    const int dpad = (p.d_in + 3) & ~3;
    uint32_t *keys = reinterpret_cast<uint32_t *>(dyn + sizeof(FusedSmem));
    float *xs = reinterpret_cast<float *>(keys + dpad);

    DIP_TRACE_MIN(p.tr, 0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slab = (int)blockIdx.x % p.n_slabs, part = (int)blockIdx.x / p.n_slabs, nparts = p.nparts;
    const bool first = blockIdx.x == 0;
    const int mask_words = (p.d_in + 31) >> 5;
    const size_t byte_off = (size_t)slab * GF_SEG + lane * 16;
    const bool lane_ok = byte_off < p.row_bytes;

    fine_zero(s.fine);
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(p.tr, 1);
    dip_launch_dependents();

    // the stamp that the epilogue's rank key needs travels while the rows stream
    int key_stamp = 0;
    if (WHICH == 0 && p.key_coarse && p.key_stamp && tid < OUT_PER_SLAB && slab * OUT_PER_SLAB + tid < p.d_out)
        key_stamp = __ldcg(p.key_stamp + slab * OUT_PER_SLAB + tid);

    // ---- the mask of the input, in every CTA ----
    if (WHICH == 0) {
        float *x_out = NORM && first ? p.x_out : nullptr;
        if (NORM && (p.d_in & 3) == 0 && p.d_in <= 8 * TK_THREADS) {
            __syncthreads();                                  // histogram zeroed
            select_fine_chained<CA>(p.xa, p.xb, x_out, xs, p.d_in, p.k, p.gamma, p.stamp, keys, s.ts, s.fine, s.maskw);
        } else {
            float scale = 1.0f;
            if (NORM)
                scale = block_residual_scale(p.xa, p.xb, p.d_in, keys, s.ts.wf, &s.ts.scale);   // ends with a barrier
            else
                __syncthreads();
            select_fine<CA, NORM>(p.xa, x_out, NORM ? xs : nullptr, p.d_in, p.k, p.gamma, p.stamp, scale, keys, s.ts,
                                  s.fine, s.maskw);
        }
    } else {
        __syncthreads();
        select_fine_coarse<CA>(p.coarse, p.xa, p.stamp, p.gamma, p.d_in, p.k, keys, s.ts, s.fine, s.maskw);
    }
    if (first)
        for (int w = tid; w < mask_words; w += TK_THREADS) p.mask_out[w] = s.maskw[w];

    // ---- this part's rows (the list lives where the rank keys were: d_in 16-bit entries always fit) ----
    const float *xsrc = (WHICH == 0 && NORM) ? xs : p.xa;
    uint16_t *idx = reinterpret_cast<uint16_t *>(keys);
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    const int n_rows = list_rows(s, s.maskw, mask_words, p.d_in, part, nparts, idx);
    stream_rows<WT>(idx, warp, GF_NW, n_rows, p.W + byte_off, p.row_bytes, lane_ok, xsrc, acc);
    DIP_TRACE_MAX(p.tr, 3);            // streaming done

    // ---- the warps' sums, in warp order ----
    float (*red)[32 * 8] = reinterpret_cast<float (*)[32 * 8]>(s.fine.hist);
#pragma unroll
    for (int e = 0; e < E; ++e) red[warp][lane * E + e] = acc[e];
    __syncthreads();
    if (tid < SLAB) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < GF_NW; ++w) t += red[w][tid];
        if (nparts > 1) p.partials[((size_t)part * p.n_slabs + slab) * SLAB + tid] = t;
        else s.sum[tid] = t;
    }
    // ---- the parts, in part order, by the last CTA of the segment ----
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
            const size_t stride = (size_t)p.n_slabs * SLAB;
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
    // ---- epilogue ----
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

template <int WT, int WHICH, bool CA, bool NORM>
dip_status launch_fused(dip_ctx *ctx, const FusedParams &p, size_t smem, cudaStream_t stream)
{
    static dip_per_device_once once;
    DIP_CUDA_TRY(ctx, dip_raise_smem_limit(once, ctx->device, gemv_fused_kernel<WT, WHICH, CA, NORM>, GF_SMEM_LIMIT));
    DIP_CUDA_TRY(ctx, dip_launch_pdl(gemv_fused_kernel<WT, WHICH, CA, NORM>, dim3(p.n_slabs * p.nparts),
                                     dim3(TK_THREADS), smem, stream, p));
    return DIP_OK;
}

template <int WT>
dip_status launch_fused_wt(dip_ctx *ctx, const FusedParams &p, int which, bool ca, bool norm, size_t smem,
                           cudaStream_t stream)
{
    if (which == 0) {
        if (ca) return norm ? launch_fused<WT, 0, true, true>(ctx, p, smem, stream)
                            : launch_fused<WT, 0, true, false>(ctx, p, smem, stream);
        return norm ? launch_fused<WT, 0, false, true>(ctx, p, smem, stream)
                    : launch_fused<WT, 0, false, false>(ctx, p, smem, stream);
    }
    return ca ? launch_fused<WT, 1, true, false>(ctx, p, smem, stream)
              : launch_fused<WT, 1, false, false>(ctx, p, smem, stream);
}

size_t fused_smem_bytes(int which, int d_in, bool norm)
{
    const size_t dpad = ((size_t)d_in + 3) & ~(size_t)3;
    return sizeof(FusedSmem) + dpad * 4 + (which == 0 && norm ? dpad * 4 : 0);
}

// Segments and row parts of a launch; false when the shape does not fit this path.
bool fused_plan(const dip_ctx *ctx, const dip_mlp_weights *w, int which, bool norm, FusedParams &p)
{
    if (!ctx->gemv_direct || !ctx->fuse_select) return false;
    if (w->wtype != DIP_W_F32 && w->wtype != DIP_W_BF16) return false;
    p.d_in = which == 0 ? w->d_model : w->d_ff;
    p.d_out = which == 0 ? w->d_ff : w->d_model;
    if (which == 1 && ((p.d_in & 31) != 0 || p.d_in > 8 * TK_COARSE_ITERS * TK_THREADS)) return false;
    if (fused_smem_bytes(which, p.d_in, norm) > GF_SMEM_LIMIT) return false;
    const size_t row_elems = which == 0 ? (size_t)2 * w->d_ff : (size_t)w->d_model;
    p.row_bytes = w->wtype == DIP_W_F32 ? row_elems * 4 : row_elems * 2;
    p.n_slabs = (int)((p.row_bytes + GF_SEG - 1) / GF_SEG);
    if (p.n_slabs > ctx->n_tickets) return false;
    const int slab_elems = w->wtype == DIP_W_F32 ? 128 : 256;
    int nparts = ctx->sm_count / p.n_slabs;
    if (nparts < 1) nparts = 1;
    while (nparts > 1 && (size_t)nparts * p.n_slabs * slab_elems > ctx->partials_floats) --nparts;
    p.nparts = nparts;
    return true;
}

}  // namespace

bool dip_gemv_fused_supported(const dip_ctx *ctx, const dip_mlp_weights *w, int which, bool norm)
{
    FusedParams p;
    return fused_plan(ctx, w, which, norm, p);
}

dip_status dip_launch_gemv_fused(dip_ctx *ctx, const dip_mlp_weights *w, int which, const dip_fused_select *sel,
                                 float *out, cudaStream_t stream, dip_gemv_keys *keys)
{
    const bool norm = which == 0 && sel->xb != nullptr;
    FusedParams p;
    if (!fused_plan(ctx, w, which, norm, p)) return DIP_ERR_UNSUPPORTED;
    if (p.nparts > sel->k) p.nparts = sel->k;
    p.W = (const char *)(which == 0 ? w->gate_up : w->down);
    p.out = out;
    p.partials = ctx->partials;
    p.tickets = ctx->tickets;
    p.tr = dip_trace_slot(ctx, which == 0 ? 4 : 5);
    p.key_coarse = nullptr;
    p.key_stamp = nullptr;
    p.key_gamma = 1.0f;
    if (keys) keys->written = 0;
    if (which == 0 && keys && keys->coarse) {
        p.key_coarse = keys->coarse;
        p.key_stamp = keys->stamp;
        p.key_gamma = keys->gamma;
        keys->written = 1;
    }
    p.xa = sel->xa;
    p.xb = sel->xb;
    p.x_out = sel->x_out;
    p.coarse = sel->coarse;
    p.k = sel->k;
    p.gamma = sel->gamma;
    p.stamp = sel->stamp;
    p.mask_out = sel->mask_out;
    const size_t smem = fused_smem_bytes(which, p.d_in, norm);
    return w->wtype == DIP_W_F32 ? launch_fused_wt<DIP_W_F32>(ctx, p, which, sel->stamp != nullptr, norm, smem, stream)
                                 : launch_fused_wt<DIP_W_BF16>(ctx, p, which, sel->stamp != nullptr, norm, smem, stream);
}
