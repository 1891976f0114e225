// Expansion of a 4-bit group-quantised expert into the bf16 blob layout the FFN kernels read.
//
// Host store layout of one 4-bit expert (Section 3.2 keeps the experts in 4-bit form; what is
// stored here is plain symmetric group quantisation): for each of W_g [F][d], W_u [F][d],
// W_d [d][F], in this order, the codes [rows][cols / 2] (one byte = two columns, the even column
// in the low nibble) followed by the scales [rows][cols / 64] (bf16).  The weight that the layer
// computes with is bf16( scale * (code - 8) ): the product is exact in fp32 and is rounded to
// nearest even.  The output is the bf16 blob of melinoe_moe_pack_expert: per hidden unit f the rows
// W_g[f] | W_u[f] | W_d[:, f], the 16-byte pieces of every 128-byte group at (piece xor (f mod 8)).
#include "kernels.cuh"

namespace melinoe {

namespace {

__device__ __forceinline__ uint32_t bf16_rne_bits(float v)
{
    uint32_t u = __float_as_uint(v);
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

// A block expands tiles of 64 x 64 weights.  W_g / W_u: 64 rows f x 64 columns, written straight
// through; W_d: 64 rows c x 64 columns f, transposed through shared memory so that the 64 values
// c of one f leave as one 128-byte row piece.
__global__ void __launch_bounds__(256) dequant_q4_kernel(const unsigned char *__restrict__ q, uint16_t *__restrict__ out, int d, int F)
{
    __shared__ uint16_t s_t[64][66];
    const size_t n = (size_t)d * F;
    const size_t sec = n / 2 + n / 32;                 // one matrix's section of the 4-bit blob
    const int tiles_gu = (F / 64) * (d / 64), tiles_d = (d / 64) * (F / 64);
    const int total = 2 * tiles_gu + tiles_d;
    const int tid = threadIdx.x;
    const int r = tid >> 2, part = tid & 3;            // source row of the tile, 16 of its 64 columns
    for (int t = blockIdx.x; t < total; t += gridDim.x) {
        const int m = t < tiles_gu ? 0 : (t < 2 * tiles_gu ? 1 : 2);
        const int tt = t - m * tiles_gu;
        const int cols = m < 2 ? d : F;
        const int tr = tt / (cols / 64), tc = tt % (cols / 64);      // tile of source rows, of source columns
        const unsigned char *codes = q + m * sec;
        const uint16_t *scales = reinterpret_cast<const uint16_t *>(q + m * sec + n / 2);
        const size_t row = (size_t)tr * 64 + r;
        const float sc = __uint_as_float((uint32_t)scales[row * (cols / 64) + tc] << 16);
        const uint2 c8 = *reinterpret_cast<const uint2 *>(codes + (row * cols + (size_t)tc * 64 + part * 16) / 2);
        uint32_t o[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t word = i < 4 ? c8.x : c8.y;
            const uint32_t byte = (word >> (8 * (i & 3))) & 0xffu;
            const float lo = __fmul_rn(sc, (float)((int)(byte & 15u) - 8));
            const float hi = __fmul_rn(sc, (float)((int)(byte >> 4) - 8));
            o[i] = bf16_rne_bits(lo) | (bf16_rne_bits(hi) << 16);
        }
        if (m < 2) {
            // row f = row, columns tc * 64 + part * 16 ..: two 16-byte pieces of the 128-byte group tc
            const int f = (int)row;
            uint16_t *dst = out + ((size_t)f * 3 + m) * d + (size_t)tc * 64;
            const int p0 = (part * 2) ^ (f & 7), p1 = (part * 2 + 1) ^ (f & 7);
            *reinterpret_cast<uint4 *>(dst + p0 * 8) = make_uint4(o[0], o[1], o[2], o[3]);
            *reinterpret_cast<uint4 *>(dst + p1 * 8) = make_uint4(o[4], o[5], o[6], o[7]);
        } else {
            // source row c = row, source columns f = tc * 64 + part * 16 ..: transpose
            __syncthreads();
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                s_t[part * 16 + 2 * i][r] = (uint16_t)(o[i] & 0xffffu);
                s_t[part * 16 + 2 * i + 1][r] = (uint16_t)(o[i] >> 16);
            }
            __syncthreads();
            // thread: f = tc * 64 + r, 16 of the 64 values c = tr * 64 + part * 16 ..
            const int f = tc * 64 + r;
            uint32_t w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
                w[i] = (uint32_t)s_t[r][part * 16 + 2 * i] | ((uint32_t)s_t[r][part * 16 + 2 * i + 1] << 16);
            uint16_t *dst = out + ((size_t)f * 3 + 2) * d + (size_t)tr * 64;
            const int p0 = (part * 2) ^ (f & 7), p1 = (part * 2 + 1) ^ (f & 7);
            *reinterpret_cast<uint4 *>(dst + p0 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4 *>(dst + p1 * 8) = make_uint4(w[4], w[5], w[6], w[7]);
        }
    }
}

}  // namespace

// Copy of a few KB from device-mapped page-locked host memory into device memory by the SMs
// themselves: for decode-sized inputs this takes the stream less time than a copy-engine operation.
__global__ void __launch_bounds__(256) stage_in_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int n16)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");      // dst may still be read by the kernel ahead in the stream
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += gridDim.x * blockDim.x)
        dst[i] = src[i];
}

cudaError_t launch_stage_in(cudaStream_t stream, const void *src_mapped, void *dst, size_t bytes)
{
    const int n16 = (int)(bytes / 16);
    const int blocks = (n16 + 255) / 256 < 32 ? (n16 + 255) / 256 : 32;
    stage_in_kernel<<<blocks, 256, 0, stream>>>(static_cast<const uint4 *>(src_mapped), static_cast<uint4 *>(dst), n16);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_dequant_q4(cudaStream_t stream, const void *q4_blob, void *slot, int d, int F, int n_sms)
{
    dequant_q4_kernel<<<n_sms * 8, 256, 0, stream>>>(static_cast<const unsigned char *>(q4_blob), static_cast<uint16_t *>(slot), d, F);
    count_launch();
    return cudaGetLastError();
}

}  // namespace melinoe
