// Neuron-major products for Gate pruning / Up pruning (Sec. 3.2, Eq. 5): out_j = W[j, :] . x for
// all neurons j (the dense, ranking activation) or for a list of kept neurons (the other
// first-layer matrix, pruned by rows).  W is [d_ff][d_model] row-major, so a neuron is one
// contiguous row: one warp per row, 16 bytes per lane per load, four loads in flight per lane,
// x staged in shared memory, a shuffle reduction per row.  HBM-bound: every weight is used once.
#include <cuda_bf16.h>

#include "common.cuh"

namespace {

constexpr int RD_THREADS = 1024;
constexpr int RD_UNROLL = 4;

struct RowdotParams {
    const char *W;             // [d_ff][d_model]
    int d_model, d_ff;
    const float *x;            // [d_model]
    const int32_t *rows;       // kept neurons (ascending) or nullptr = all
    int n_rows;                // number of rows to do
    int silu;                  // apply silu to the product
    const float *mul;          // [d_ff] or nullptr: out_j *= mul_j
    float *out;                // [d_ff]
    unsigned long long *tr;
};

__device__ __forceinline__ float rd_silu(float g) { return g / (1.0f + expf(-g)); }

// E weights per 16 bytes.  x sits in shared memory so that the float4 reads of a warp are
// contiguous: F32 as is; BF16 (8 weights per lane) as two planes, the first and the second four
// x of every group of eight.
template <int WT> struct RdTraits;
template <> struct RdTraits<DIP_W_F32> { static constexpr int E = 4; };
template <> struct RdTraits<DIP_W_BF16> { static constexpr int E = 8; };

template <int WT>
__global__ void __launch_bounds__(RD_THREADS, 1)
rowdot_kernel(const RowdotParams p)
{
    constexpr int E = RdTraits<WT>::E;
    extern __shared__ __align__(16) float xs[];
    DIP_TRACE_MIN(p.tr, 0);
    dip_grid_dependency_wait();
    DIP_TRACE_MIN(p.tr, 1);
    dip_launch_dependents();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int vecs = p.d_model / E;                            // 16-byte pieces per row
    for (int i = tid; i < p.d_model; i += RD_THREADS) {
        const float v = p.x[i];
        if (E == 4) xs[i] = v;
        else xs[((i & 4) ? p.d_model / 2 : 0) + (i >> 3) * 4 + (i & 3)] = v;
    }
    __syncthreads();
    const float4 *x_lo = reinterpret_cast<const float4 *>(xs);
    const float4 *x_hi = reinterpret_cast<const float4 *>(xs + p.d_model / 2);
    const int n_warps = gridDim.x * (RD_THREADS / 32);
    const size_t row_bytes = (size_t)p.d_model * (WT == DIP_W_F32 ? 4 : 2);
    for (int r = blockIdx.x * (RD_THREADS / 32) + warp; r < p.n_rows; r += n_warps) {
        const int j = p.rows ? p.rows[r] : r;
        const uint4 *row = reinterpret_cast<const uint4 *>(p.W + (size_t)j * row_bytes);
        float acc = 0.f;
        for (int v0 = 0; v0 < vecs; v0 += 32 * RD_UNROLL) {
            uint4 q[RD_UNROLL];
#pragma unroll
            for (int u = 0; u < RD_UNROLL; ++u) {
                const int v = v0 + u * 32 + lane;
                q[u] = v < vecs ? __ldcs(row + v) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < RD_UNROLL; ++u) {
                const int v = v0 + u * 32 + lane;
                if (v >= vecs) continue;
                if (WT == DIP_W_F32) {
                    const float4 xv = x_lo[v];
                    acc = fmaf(__uint_as_float(q[u].x), xv.x, acc);
                    acc = fmaf(__uint_as_float(q[u].y), xv.y, acc);
                    acc = fmaf(__uint_as_float(q[u].z), xv.z, acc);
                    acc = fmaf(__uint_as_float(q[u].w), xv.w, acc);
                } else {
                    // bfloat16 is the upper half of a binary32
                    const float4 xa = x_lo[v], xb = x_hi[v];
                    acc = fmaf(__uint_as_float(q[u].x << 16), xa.x, acc);
                    acc = fmaf(__uint_as_float(q[u].x & 0xffff0000u), xa.y, acc);
                    acc = fmaf(__uint_as_float(q[u].y << 16), xa.z, acc);
                    acc = fmaf(__uint_as_float(q[u].y & 0xffff0000u), xa.w, acc);
                    acc = fmaf(__uint_as_float(q[u].z << 16), xb.x, acc);
                    acc = fmaf(__uint_as_float(q[u].z & 0xffff0000u), xb.y, acc);
                    acc = fmaf(__uint_as_float(q[u].w << 16), xb.z, acc);
                    acc = fmaf(__uint_as_float(q[u].w & 0xffff0000u), xb.w, acc);
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) {
            float v = p.silu ? rd_silu(acc) : acc;
            if (p.mul) v *= p.mul[j];
            p.out[j] = v;
        }
    }
    DIP_TRACE_MAX(p.tr, 2);
}

}  // namespace

dip_status dip_launch_rowdot(dip_ctx *ctx, int wtype, const void *W, int d_model, int d_ff, const float *x,
                             const int32_t *rows, int n_rows, int silu, const float *mul, float *out,
                             cudaStream_t stream)
{
    if (wtype != DIP_W_F32 && wtype != DIP_W_BF16) return DIP_ERR_UNSUPPORTED;
    RowdotParams p;
    p.W = (const char *)W;
    p.d_model = d_model;
    p.d_ff = d_ff;
    p.x = x;
    p.rows = rows;
    p.n_rows = n_rows;
    p.silu = silu;
    p.mul = mul;
    p.out = out;
    p.tr = dip_trace_slot(ctx, 9);
    const size_t smem = sizeof(float) * (size_t)d_model;
    const int warps_needed = n_rows;
    int blocks = (warps_needed + RD_THREADS / 32 - 1) / (RD_THREADS / 32);
    if (blocks > ctx->sm_count) blocks = ctx->sm_count;
    if (blocks < 1) blocks = 1;
    if (wtype == DIP_W_F32) {
        static dip_per_device_once once;
        DIP_CUDA_TRY(ctx, dip_raise_smem_limit(once, ctx->device, rowdot_kernel<DIP_W_F32>, sizeof(float) * DIP_MAX_D));
        DIP_CUDA_TRY(ctx, dip_launch_pdl(rowdot_kernel<DIP_W_F32>, dim3(blocks), dim3(RD_THREADS), smem, stream, p));
    } else {
        static dip_per_device_once once;
        DIP_CUDA_TRY(ctx, dip_raise_smem_limit(once, ctx->device, rowdot_kernel<DIP_W_BF16>, sizeof(float) * DIP_MAX_D));
        DIP_CUDA_TRY(ctx, dip_launch_pdl(rowdot_kernel<DIP_W_BF16>, dim3(blocks), dim3(RD_THREADS), smem, stream, p));
    }
    return DIP_OK;
}
