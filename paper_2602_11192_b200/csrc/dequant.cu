// Expansion of a 4-bit group-quantised expert into the bf16 blob layout the FFN kernels read.
//
// Both blobs are organised per hidden unit f (see melinoe_moe_pack_expert / _pack_expert_q4): the
// 4-bit unit holds the codes of W_g[f], W_u[f], W_d[:, f] (d / 2 bytes each, the even element in the
// low nibble, the 16-byte pieces of every 128-byte group at (piece xor (f mod 8)); in W_d[:, f] the
// code at position p of a group of 64 is element 8 (p mod 8) + p / 8 of the group), then their
// scales (d / 64 bf16 each).  The weight that the layer computes with is bf16(scale * (code - 8)):
// the product is exact in fp32 and is rounded to nearest even.  The bf16 unit holds the three
// vectors of d bf16 values with the same kind of permutation on its own 16-byte pieces.
#include "kernels.cuh"

namespace melinoe {

namespace {

__device__ __forceinline__ uint32_t bf16_rne_bits(float v)
{
    uint32_t u = __float_as_uint(v);
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

// One thread expands one 16-byte piece of codes (32 weights) into four 16-byte pieces of bf16.
__global__ void __launch_bounds__(256) dequant_q4_kernel(const unsigned char *__restrict__ q, uint16_t *__restrict__ out, int d, int F,
                                                         int unit_bytes)
{
    const int pieces = d / 32;                        // code pieces of one vector
    const size_t total = (size_t)F * 3 * pieces;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int f = (int)(i / (3 * pieces)), rest = (int)(i % (3 * pieces));
        const int m = rest / pieces, piece = rest % pieces;            // vector (g, u, d) and logical code piece
        const unsigned char *unit = q + (size_t)f * unit_bytes;
        const int x = f & 7;
        const int ppiece = (piece & ~7) | ((piece ^ x) & 7);
        const uint4 c = *reinterpret_cast<const uint4 *>(unit + (size_t)m * (d / 2) + (size_t)ppiece * 16);
        const uint16_t *scales = reinterpret_cast<const uint16_t *>(unit + 3 * (size_t)(d / 2)) + m * (d / 64);
        const float sc = __uint_as_float((uint32_t)scales[piece / 2] << 16);
        const uint32_t words[4] = {c.x, c.y, c.z, c.w};
        uint16_t *row = out + ((size_t)f * 3 + m) * d;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            uint32_t o[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const uint32_t byte = (words[w] >> (8 * b)) & 0xffu;
                const float lo = __fmul_rn(sc, (float)((int)(byte & 15u) - 8));
                const float hi = __fmul_rn(sc, (float)((int)(byte >> 4) - 8));
                o[b] = bf16_rne_bits(lo) | (bf16_rne_bits(hi) << 16);
            }
            if (m < 2) {
                // these 8 weights are elements piece * 32 + w * 8 .. of the vector: bf16 piece 4 * piece + w
                const int bp = 4 * piece + w;
                const int pbp = (bp & ~7) | ((bp ^ x) & 7);
                *reinterpret_cast<uint4 *>(row + (size_t)pbp * 8) = make_uint4(o[0], o[1], o[2], o[3]);
            } else {
                // W_d[:, f]: code position pos of a group of 64 holds element 8 * (pos mod 8) + pos / 8; these are
                // positions (piece mod 2) * 32 + w * 8 + j, j = 0 .. 7, that is element 8 j + (piece mod 2) * 4 + w
                const int grp = piece / 2, e0 = (piece & 1) * 4 + w;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int el = grp * 64 + 8 * j + e0;
                    const int bp = el / 8, pbp = (bp & ~7) | ((bp ^ x) & 7);
                    row[(size_t)pbp * 8 + el % 8] = (uint16_t)(j & 1 ? o[j / 2] >> 16 : o[j / 2] & 0xffffu);
                }
            }
        }
    }
}

}  // namespace

// Copy of a few KB from device-mapped page-locked host memory into device memory by the SMs
// themselves: for decode-sized inputs this takes the stream less time than a copy-engine operation.
// Launched with programmatic stream serialisation: it is scheduled while the kernel ahead in the stream
// drains and lets the router behind it be scheduled at once; it touches memory only after the kernel ahead
// has finished (dst may still be read by it, and src may be what it wrote: a caller may chain layers
// through host buffers on one stream).
__global__ void __launch_bounds__(256) stage_in_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int n16)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += gridDim.x * blockDim.x)
        dst[i] = src[i];
}

cudaError_t launch_stage_in(cudaStream_t stream, const void *src_mapped, void *dst, size_t bytes)
{
    const int n16 = (int)(bytes / 16);
    const int blocks = (n16 + 255) / 256 < 32 ? (n16 + 255) / 256 : 32;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(blocks);
    lc.blockDim = dim3(256);
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = pdl_enabled() ? 1 : 0;
    const cudaError_t e = cudaLaunchKernelEx(&lc, stage_in_kernel, static_cast<const uint4 *>(src_mapped), static_cast<uint4 *>(dst), n16);
    count_launch();
    return e;
}

cudaError_t launch_dequant_q4(cudaStream_t stream, const void *q4_blob, void *slot, int d, int F, int n_sms)
{
    const int unit_bytes = (3 * (d / 2) + 3 * (d / 64) * 2 + 15) / 16 * 16;
    dequant_q4_kernel<<<n_sms * 8, 256, 0, stream>>>(static_cast<const unsigned char *>(q4_blob), static_cast<uint16_t *>(slot), d, F,
                                                      unit_bytes);
    count_launch();
    return cudaGetLastError();
}

}  // namespace melinoe
