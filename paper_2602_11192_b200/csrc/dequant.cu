// Expansion of a 4-bit group-quantised expert into the bf16 slot layout the FFN kernels read.
//
// Host store layout of one 4-bit expert (Section 3.2 keeps the experts in 4-bit form; what is
// stored here is plain symmetric group quantisation): for each of W_g [F][d], W_u [F][d],
// W_d [d][F], in this order, the codes [rows][cols / 2] (one byte = two columns, the even column
// in the low nibble) followed by the scales [rows][cols / 64] (bf16).  The weight that the layer
// computes with is bf16( scale * (code - 8) ): the product is exact in fp32 and is rounded to
// nearest even.  The kernel is a pure stream: 1.6 bytes in, 6 bytes out per three weights.
#include "kernels.cuh"

namespace melinoe {

namespace {

__device__ __forceinline__ uint32_t bf16_rne_bits(float v)
{
    uint32_t u = __float_as_uint(v);
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

// One thread expands 16 consecutive weights of one row (8 code bytes in, 32 bytes out).
__global__ void __launch_bounds__(256) dequant_q4_kernel(const unsigned char *__restrict__ q, uint16_t *__restrict__ out, int d, int F)
{
    const size_t per_gu = (size_t)F * d, per_d = (size_t)d * F;       // weights per matrix
    const size_t units = (2 * per_gu + per_d) / 16;
    for (size_t u = (size_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (size_t)gridDim.x * blockDim.x) {
        size_t w0 = u * 16;                 // first weight of the unit, counted over the three matrices
        int m = 0;
        if (w0 >= per_gu) {
            w0 -= per_gu;
            m = 1;
            if (w0 >= per_gu) {
                w0 -= per_gu;
                m = 2;
            }
        }
        const size_t n_w = m < 2 ? per_gu : per_d;
        const int cols = m < 2 ? d : F;
        // the matrix's section of the 4-bit blob: codes, then scales
        const size_t sec = (size_t)m * (per_gu / 2 + per_gu / 32);     // W_g and W_u sections have the same size
        const unsigned char *codes = q + sec;
        const uint16_t *scales = reinterpret_cast<const uint16_t *>(q + sec + n_w / 2);
        const size_t row = w0 / cols, col = w0 % cols;
        const float s = __uint_as_float((uint32_t)scales[row * (cols / 64) + col / 64] << 16);
        const uint2 c8 = *reinterpret_cast<const uint2 *>(codes + w0 / 2);
        uint32_t o[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t word = i < 4 ? c8.x : c8.y;
            const uint32_t byte = (word >> (8 * (i & 3))) & 0xffu;
            const float lo = __fmul_rn(s, (float)((int)(byte & 15u) - 8));
            const float hi = __fmul_rn(s, (float)((int)(byte >> 4) - 8));
            o[i] = bf16_rne_bits(lo) | (bf16_rne_bits(hi) << 16);
        }
        uint4 *dst = reinterpret_cast<uint4 *>(out + (size_t)m * per_gu + w0);
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
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
