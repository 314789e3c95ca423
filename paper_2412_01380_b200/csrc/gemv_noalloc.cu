// dip_sparse_gemv_down_noalloc: the down-projection GEMV over kept columns for callers that
// must not allocate device memory (see include/dip.h).  Its scratch -- the split-row partial
// sums and the per-slab arrival counters that the context-based entry point keeps in a
// cudaMalloc'd workspace -- lives in a file-scope __device__ array of fixed size instead.
// The paper has no counterpart of this entry point; the arithmetic is that of
// dip_sparse_gemv_down (Eq. 1 inside Eq. 3 with the mask of Eq. 8).
#include <mutex>

#include "common.cuh"

namespace {

constexpr int NA_THREADS = 256;
constexpr int NA_WARPS = NA_THREADS / 32;
constexpr int NA_UNROLL = 8;
constexpr int NA_MAX_SLABS = 128;                  // arrival counters
constexpr size_t NA_PARTIAL_FLOATS = 1u << 20;     // 4 MB of partial sums
constexpr int NA_MAX_D_MODEL = 16384;              // largest output length accepted
constexpr int NA_MAX_DEVICES = 64;

struct NaScratch {
    unsigned int tickets[NA_MAX_SLABS];
    float partials[NA_PARTIAL_FLOATS];
};

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char na_scratch[sizeof(NaScratch)];

struct NaDevice {
    bool ready;
    NaScratch *scratch;   // device address of na_scratch on this device
    int sm_count;
};
NaDevice na_dev[NA_MAX_DEVICES];
std::mutex na_mutex;

template <int WT> struct NaTraits;
template <> struct NaTraits<DIP_W_F32>  { static constexpr int E = 8; };
template <> struct NaTraits<DIP_W_BF16> { static constexpr int E = 16; };

__device__ __forceinline__ uint4 na_ld16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

template <int WT> __device__ __forceinline__ void na_decode(uint4 a, uint4 b, float (&w)[NaTraits<WT>::E]);
template <> __device__ __forceinline__ void na_decode<DIP_W_F32>(uint4 a, uint4 b, float (&w)[8])
{
    const uint32_t u[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = __uint_as_float(u[i]);
}
template <> __device__ __forceinline__ void na_decode<DIP_W_BF16>(uint4 a, uint4 b, float (&w)[16])
{
    const uint32_t u[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        w[2 * i] = __uint_as_float(u[i] << 16);
        w[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
}

// grid = (output slabs of 32*E elements) x (row parts).  Same scheme as the context-based
// kernel: a warp reads one kept row's 1 KB slab segment per step; warps are combined in warp
// order, parts in part order by the last CTA to arrive at the slab.
template <int WT>
__global__ void __launch_bounds__(NA_THREADS)
down_noalloc_kernel(const char *__restrict__ W, size_t row_bytes, int d_model, int d_ff,
                    const float *__restrict__ h, const int32_t *__restrict__ kept_idx, int n_kept,
                    float *__restrict__ y, NaScratch *scratch)
{
    constexpr int E = NaTraits<WT>::E;
    constexpr int SLAB = 32 * E;
    constexpr int EB = 32 / E;                       // bytes per element
    __shared__ float s_red[NA_WARPS][SLAB];
    __shared__ int s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slab = blockIdx.x, part = blockIdx.y, nparts = gridDim.y;
    const int r_begin = (int)(((long long)part * n_kept) / nparts);
    const int r_end = (int)(((long long)(part + 1) * n_kept) / nparts);
    const int elem0 = slab * SLAB + lane * E;
    const bool lane_ok = elem0 < d_model;
    const char *wbase = W + (size_t)(lane_ok ? elem0 : 0) * EB;

    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;

    const int n_mine = (r_end - r_begin - warp + NA_WARPS - 1) / NA_WARPS;
    for (int c0 = 0; c0 < n_mine; c0 += 32) {
        int my_idx = 0;
        float my_v = 0.f;
        if (c0 + lane < n_mine) {
            my_idx = kept_idx[r_begin + warp + (c0 + lane) * NA_WARPS];
            // an entry outside [0, d_ff) names no column: it contributes nothing and reads nothing
            if ((unsigned)my_idx >= (unsigned)d_ff) my_idx = 0;
            else my_v = h[my_idx];
        }
        const int n_here = min(32, n_mine - c0);
        for (int j0 = 0; j0 < n_here; j0 += NA_UNROLL) {
            uint4 ra[NA_UNROLL], rb[NA_UNROLL];
#pragma unroll
            for (int u = 0; u < NA_UNROLL; ++u) {
                int idx = __shfl_sync(0xffffffffu, my_idx, (j0 + u) & 31);
                if (j0 + u < n_here && lane_ok) {
                    const char *p = wbase + (size_t)idx * row_bytes;
                    ra[u] = na_ld16(p);
                    rb[u] = na_ld16(p + 16);
                } else {
                    ra[u] = rb[u] = make_uint4(0, 0, 0, 0);
                }
            }
#pragma unroll
            for (int u = 0; u < NA_UNROLL; ++u) {
                float w[E];
                na_decode<WT>(ra[u], rb[u], w);
                float hv = __shfl_sync(0xffffffffu, my_v, (j0 + u) & 31);
                if (j0 + u >= n_here) hv = 0.f;
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] = fmaf(w[e], hv, acc[e]);
            }
        }
    }
#pragma unroll
    for (int e = 0; e < E; ++e) s_red[warp][lane * E + e] = acc[e];
    __syncthreads();

    float *my_part = scratch->partials + ((size_t)part * gridDim.x + slab) * SLAB;
    if (nparts > 1) {
        for (int t = tid; t < SLAB; t += NA_THREADS) {
            float sum = 0.f;
#pragma unroll
            for (int w = 0; w < NA_WARPS; ++w) sum += s_red[w][t];
            my_part[t] = sum;
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = atomicAdd(&scratch->tickets[slab], 1u) == (unsigned)(nparts - 1);
        __syncthreads();
        if (!s_last) return;
        __threadfence();
    }
    for (int t = tid; t < SLAB; t += NA_THREADS) {
        const int j = slab * SLAB + t;
        if (j >= d_model) continue;
        float sum = 0.f;
        if (nparts > 1) {
            for (int q = 0; q < nparts; ++q)
                sum += __ldcg(scratch->partials + ((size_t)q * gridDim.x + slab) * SLAB + t);
        } else {
#pragma unroll
            for (int w = 0; w < NA_WARPS; ++w) sum += s_red[w][t];
        }
        y[j] = sum;
    }
}

// Once per device, with that device current: resolve the device address of the scratch
// array (its name in host code is only a stand-in for the symbol) and read the SM count.
dip_status na_setup(int device, NaDevice **out)
{
    if (device < 0 || device >= NA_MAX_DEVICES) return DIP_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(na_mutex);
    NaDevice &nd = na_dev[device];
    if (!nd.ready) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, na_scratch) != cudaSuccess || !ptr) return DIP_ERR_CUDA;
        if (cudaDeviceGetAttribute(&nd.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
            return DIP_ERR_CUDA;
        nd.scratch = (NaScratch *)ptr;
        nd.ready = true;
    }
    *out = &nd;
    return DIP_OK;
}

}  // namespace

extern "C" dip_status dip_sparse_gemv_down_noalloc(const dip_mlp_weights *w, const float *h,
                                                   const int32_t *kept_idx, int n_kept,
                                                   float *y, void *stream)
{
    if (!w || !h || !kept_idx || !y || !w->down) return DIP_ERR_INVALID_ARG;
    if (!dip_aligned16(w->down) || !dip_aligned16(h) || !dip_aligned16(y)) return DIP_ERR_INVALID_ARG;
    if (w->wtype != DIP_W_F32 && w->wtype != DIP_W_BF16) return DIP_ERR_UNSUPPORTED;
    if (w->d_model < 32 || w->d_model % 32 || w->d_ff < 1 || w->d_ff > DIP_MAX_D) return DIP_ERR_INVALID_ARG;
    if (n_kept < 1 || n_kept > w->d_ff) return DIP_ERR_INVALID_ARG;
    if (w->d_model > NA_MAX_D_MODEL) return DIP_ERR_WORKSPACE;      // beyond the fixed scratch

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return DIP_ERR_CUDA;
    NaDevice *nd = nullptr;
    dip_status st = na_setup(device, &nd);
    if (st != DIP_OK) return st;

    const int E = w->wtype == DIP_W_F32 ? 8 : 16;
    const int slab = 32 * E;
    const int n_slabs = (w->d_model + slab - 1) / slab;
    if (n_slabs > NA_MAX_SLABS) return DIP_ERR_WORKSPACE;
    int nparts = (nd->sm_count * 4 + n_slabs - 1) / n_slabs;
    const int max_by_rows = n_kept / (2 * NA_WARPS);
    if (nparts > max_by_rows) nparts = max_by_rows;
    const size_t per_part = (size_t)n_slabs * slab;
    if ((size_t)nparts * per_part > NA_PARTIAL_FLOATS) nparts = (int)(NA_PARTIAL_FLOATS / per_part);
    if (nparts < 1) nparts = 1;

    cudaStream_t s = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the arrival counters must start at zero
    if (cudaMemsetAsync(nd->scratch->tickets, 0, sizeof(unsigned int) * NA_MAX_SLABS, s) != cudaSuccess)
        return DIP_ERR_CUDA;
    dim3 grid(n_slabs, nparts);
    const size_t row_bytes = (size_t)w->d_model * (w->wtype == DIP_W_F32 ? 4 : 2);
    if (w->wtype == DIP_W_F32)
        down_noalloc_kernel<DIP_W_F32><<<grid, NA_THREADS, 0, s>>>((const char *)w->down, row_bytes, w->d_model,
                                                                    w->d_ff, h, kept_idx, n_kept, y, nd->scratch);
    else
        down_noalloc_kernel<DIP_W_BF16><<<grid, NA_THREADS, 0, s>>>((const char *)w->down, row_bytes, w->d_model,
                                                                     w->d_ff, h, kept_idx, n_kept, y, nd->scratch);
    return cudaGetLastError() == cudaSuccess ? DIP_OK : DIP_ERR_CUDA;
}
