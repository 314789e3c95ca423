// Declarations shared by the product kernels (gemv.cu, gemv_fused.cu, gemv_direct_bt.cu, gemv_int4.cu, gemv_tc.cu).
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"

constexpr int GV_MAX_ROWS = 2048;                          // kept rows per round (index list in smem)
constexpr int GV_SCAN_THREADS = 256;                       // threads that scan the mask words

struct GemvParams {
    const char *W;             // packed rows
    size_t row_bytes;          // bytes of one packed row
    const uint16_t *scales;    // INT4: binary16 scales [d_in/128][row elements], laid out like a row
    size_t scale_row_elems;    // INT4: elements of one scale row
    const float *v;            // [batch][d_in]
    int d_in;
    const uint32_t *mask_bits; // [batch][mask_words]; rows read = OR over the batch
    int mask_words;
    float *out;                // [batch][d_out]
    int d_out;
    int batch;                 // tokens in this launch (<= BT)
    float *partials;
    unsigned int *tickets;
    int *status;               // device status word (0 = fine)
    unsigned long long wait_limit_ns;   // a wait on a copy's arrival gives up after this long
    unsigned long long *tr;    // timeline slot or nullptr
    const int32_t *loc;        // two-tier: packed row of column i is W + loc[i] * row_bytes (nullptr: row i)
    int defer;                 // 1: leave the row parts in `partials` for combine_parts_kernel
    int part_base;             // first part index of this launch inside `partials`
    // gate/up, single-token launches only: top 16 bits of the rank key of every h_j for the select
    // that follows (nullptr: not wanted); the key is |h_j| * (key_stamp[j] >= 0 ? 1 : key_gamma),
    // or |h_j| without stamps
    uint16_t *key_coarse;
    const int32_t *key_stamp;
    float key_gamma;
};


__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait for the phase with the given parity; false if limit_ns ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, unsigned parity, unsigned long long limit_ns)
{
    const uint32_t a = smem_u32(bar);
    unsigned long long t0 = 0;
    for (unsigned i = 0;; ++i) {
        unsigned ok;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                     " selp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(a), "r"(parity) : "memory");
        if (ok) return true;
        if ((i & 255u) == 255u) {
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) return false;
        }
    }
}

__device__ __forceinline__ float silu_f32(float g) { return g / (1.0f + expf(-g)); }

__device__ __forceinline__ float half_bits_to_float(uint16_t h)
{
    return __half2float(__ushort_as_half(h));
}

namespace {

template <int WT> struct WTraits;
// E = weights in a lane's 16 bytes; C = gate/up interleave chunk of the bundled rows (weights)
template <> struct WTraits<DIP_W_F32>       { static constexpr int E = 4;  static constexpr int C = 4; };
template <> struct WTraits<DIP_W_BF16>      { static constexpr int E = 8;  static constexpr int C = 8; };

template <int WT> __device__ __forceinline__ void decode16(const uint4 &r, float (&w)[WTraits<WT>::E]);
template <> __device__ __forceinline__ void decode16<DIP_W_F32>(const uint4 &r, float (&w)[4])
{
    w[0] = __uint_as_float(r.x); w[1] = __uint_as_float(r.y);
    w[2] = __uint_as_float(r.z); w[3] = __uint_as_float(r.w);
}
// bfloat16 is the upper half of a binary32: widening is a shift or a mask.
template <> __device__ __forceinline__ void decode16<DIP_W_BF16>(const uint4 &r, float (&w)[8])
{
    const uint32_t u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        w[2 * i] = __uint_as_float(u[i] << 16);
        w[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
}

}  // namespace

// gemv.cu: sum of the row parts left in ctx->partials ([parts][n_slabs][bt][slab_elems]; gate/up
// elements interleaved in chunks of c) and the epilogue, spread over the device.
dip_status dip_launch_combine_parts(dip_ctx *ctx, int which, int total_parts, int n_slabs, int bt, int slab_elems, int c,
                                    int batch, int d_out, float *out, cudaStream_t stream);

// gemv_direct_bt.cu: F32 / BF16 weights, two tokens: the product over the union of the tokens' rows with
// plain loads and FMAs.
dip_status dip_launch_gemv_direct_bt(dip_ctx *ctx, GemvParams &p, int wtype, int which, int n_kept_max, cudaStream_t stream);

// gemv_tc.cu: BF16 weights, 8 to 16 tokens: the product over the union of the tokens' rows on tcgen05 tensor cores.
dip_status dip_launch_gemv_tc(dip_ctx *ctx, GemvParams &p, int which, int n_kept_max, cudaStream_t stream);

// gemv_int4.cu: the single-token product for INT4-g128 weights.  mode as dip_gemv_rows.mode.
dip_status dip_launch_gemv_int4(dip_ctx *ctx, GemvParams &p, int which, int n_kept_max, int mode, cudaStream_t stream);
