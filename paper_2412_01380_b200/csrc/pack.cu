// One-off repacking of canonical weight matrices ([d_out][d_in] row-major, the paper's
// orientation) into the column-contiguous layout the kernels read: row i of the packed array
// is column i of W, and the gate and up columns that share a mask (Eq. 7) are bundled in one
// row, interleaved per lane chunk.  Values are moved bit for bit.
#include "common.cuh"

namespace {

// Transpose src[d_out][d_in] into dst rows of `dst_row_elems` elements.
// mode 0: dst[i][j];  mode 1 (gate) / 2 (up): dst[i][(j / C) * 2C + (j % C) + (mode == 2 ? C : 0)].
template <typename T>
__global__ void pack_transpose_kernel(const T *__restrict__ src, T *__restrict__ dst,
                                      int d_out, int d_in, int dst_row_elems, int mode, int C)
{
    __shared__ T tile[32][33];
    const int i0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        int j = j0 + r, i = i0 + threadIdx.x;
        if (j < d_out && i < d_in) tile[r][threadIdx.x] = src[(size_t)j * d_in + i];
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        int i = i0 + r, j = j0 + threadIdx.x;
        if (i < d_in && j < d_out) {
            size_t col = mode == 0 ? (size_t)j : (size_t)(j / C) * (2 * C) + (j % C) + (mode == 2 ? C : 0);
            dst[(size_t)i * dst_row_elems + col] = tile[threadIdx.x][r];
        }
    }
}

// 4-bit codes.  src: [d_out][d_in/2] bytes, even i in the low nibble.  A packed row is a sequence
// of chunks of 128 codes (64 bytes): local element e of a chunk is nibble (e >> 4) of the 32-bit
// word w = e & 15, and the 16 words are stored in the order 0, 8, 1, 9, ..., 7, 15 (so that the
// eight bytes at offset 8 g hold words g and g + 8: one lane's share of eight 16 x 16 MMA tiles).
// mode 0 (down): chunk c holds outputs 128 c + e.  mode 1 (gate) / 2 (up): chunk c holds gate
// outputs 64 c + e for e < 64 and up outputs 64 c + (e - 64) for e >= 64.
// One thread writes one destination byte: nibbles m and m + 1 (m even) of a word, i.e. two
// outputs 16 apart of the same source matrix.
__global__ void pack_int4_kernel(const uint8_t *__restrict__ src, uint8_t *__restrict__ dst,
                                 int d_out, int d_in, int dst_row_bytes, int mode)
{
    const int per_chunk = mode == 0 ? 64 : 32;                    // destination bytes of this matrix per chunk
    const int out_per_chunk = mode == 0 ? 128 : 64;
    const int chunks = d_out / out_per_chunk;
    const size_t n = (size_t)d_in * chunks * per_chunk;
    for (size_t tt = blockIdx.x * (size_t)blockDim.x + threadIdx.x; tt < n; tt += (size_t)gridDim.x * blockDim.x) {
        const int i = (int)(tt / ((size_t)chunks * per_chunk));
        const int rem = (int)(tt % ((size_t)chunks * per_chunk));
        const int c = rem / per_chunk, b = rem % per_chunk;
        const int bytes_per_word = mode == 0 ? 4 : 2;             // of this matrix
        const int wp = b / bytes_per_word, bl = b % bytes_per_word;
        const int w = (wp >> 1) + 8 * (wp & 1);                   // word stored at position wp
        const int j = c * out_per_chunk + 32 * bl + w;            // output in the low nibble; j + 16 in the high one
        const int sh = 4 * (i & 1);
        const uint8_t lo = (src[(size_t)j * (d_in / 2) + (i >> 1)] >> sh) & 15;
        const uint8_t hi = (src[(size_t)(j + 16) * (d_in / 2) + (i >> 1)] >> sh) & 15;
        const int byte_in_word = mode == 2 ? 2 + bl : bl;
        dst[(size_t)i * dst_row_bytes + (size_t)c * 64 + wp * 4 + byte_in_word] = (uint8_t)(lo | (hi << 4));
    }
}

// binary16 scales [groups][d_out] -> rows laid out element for element like the code chunks, with
// local element e of a chunk at position (e & 15) * 8 + (e >> 4): eight consecutive scales are the
// eight tiles of one fragment row.
__global__ void pack_scales_kernel(const uint16_t *__restrict__ src, uint16_t *__restrict__ dst,
                                   int groups, int d_out, int dst_row_elems, int mode)
{
    const size_t n = (size_t)groups * d_out;
    for (size_t t = blockIdx.x * (size_t)blockDim.x + threadIdx.x; t < n; t += (size_t)gridDim.x * blockDim.x) {
        const int g = (int)(t / d_out), j = (int)(t % d_out);
        const int c = mode == 0 ? j / 128 : j / 64;
        const int e = mode == 0 ? j % 128 : (j % 64) + (mode == 2 ? 64 : 0);
        dst[(size_t)g * dst_row_elems + (size_t)c * 128 + (e & 15) * 8 + (e >> 4)] = src[t];
    }
}

template <typename T>
void launch_transpose(const void *src, void *dst, int d_out, int d_in, int dst_row_elems, int mode, int C,
                      cudaStream_t stream)
{
    dim3 grid((d_in + 31) / 32, (d_out + 31) / 32), block(32, 8);
    pack_transpose_kernel<T><<<grid, block, 0, stream>>>((const T *)src, (T *)dst, d_out, d_in,
                                                         dst_row_elems, mode, C);
}

}  // namespace

dip_status dip_launch_pack(dip_ctx *ctx, int wtype, int d_model, int d_ff,
                           const void *Wg, const void *Wu, const void *Wd,
                           const void *Sg, const void *Su, const void *Sd,
                           const dip_mlp_weights *out, cudaStream_t stream)
{
    void *gu = const_cast<void *>(out->gate_up), *dn = const_cast<void *>(out->down);
    if (wtype == DIP_W_F32) {
        launch_transpose<uint32_t>(Wg, gu, d_ff, d_model, 2 * d_ff, 1, 4, stream);
        launch_transpose<uint32_t>(Wu, gu, d_ff, d_model, 2 * d_ff, 2, 4, stream);
        launch_transpose<uint32_t>(Wd, dn, d_model, d_ff, d_model, 0, 1, stream);
    } else if (wtype == DIP_W_BF16) {
        launch_transpose<uint16_t>(Wg, gu, d_ff, d_model, 2 * d_ff, 1, 8, stream);
        launch_transpose<uint16_t>(Wu, gu, d_ff, d_model, 2 * d_ff, 2, 8, stream);
        launch_transpose<uint16_t>(Wd, dn, d_model, d_ff, d_model, 0, 1, stream);
    } else {
        void *gus = const_cast<void *>(out->gate_up_scales), *dns = const_cast<void *>(out->down_scales);
        const int blocks = ctx->sm_count * 8;
        pack_int4_kernel<<<blocks, 256, 0, stream>>>((const uint8_t *)Wg, (uint8_t *)gu, d_ff, d_model, d_ff, 1);
        pack_int4_kernel<<<blocks, 256, 0, stream>>>((const uint8_t *)Wu, (uint8_t *)gu, d_ff, d_model, d_ff, 2);
        pack_int4_kernel<<<blocks, 256, 0, stream>>>((const uint8_t *)Wd, (uint8_t *)dn, d_model, d_ff, d_model / 2, 0);
        pack_scales_kernel<<<blocks, 256, 0, stream>>>((const uint16_t *)Sg, (uint16_t *)gus, d_model / DIP_INT4_GROUP,
                                                       d_ff, 2 * d_ff, 1);
        pack_scales_kernel<<<blocks, 256, 0, stream>>>((const uint16_t *)Su, (uint16_t *)gus, d_model / DIP_INT4_GROUP,
                                                       d_ff, 2 * d_ff, 2);
        pack_scales_kernel<<<blocks, 256, 0, stream>>>((const uint16_t *)Sd, (uint16_t *)dns, d_ff / DIP_INT4_GROUP,
                                                       d_model, d_model, 0);
    }
    DIP_CUDA_TRY(ctx, cudaGetLastError());
    return DIP_OK;
}
