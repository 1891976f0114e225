// Router: logits, top-k with lowest-index tie-breaking, renormalised gates (Eq. 1).
//
// The selected indices are an integer result that must agree bit for bit with a CPU
// evaluation, so the fp32 logit is summed in one fixed order: element j belongs to lane
// (j mod 256) / 8; every lane adds its elements in increasing j into one accumulator
// (products of two bf16 values are exact in fp32, so fused or unfused multiply-add give the
// same bits); the 32 lane sums are folded by xor-butterflies with strides 16, 8, 4, 2, 1; the
// bias is added last.  That is exactly one 16-byte load per lane per 256 columns.
#include "kernels.cuh"

namespace melinoe {

namespace {

__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

constexpr int kRouterWarps = 8;
constexpr int kMaxExpertsPerWarp = kMaxExperts / kRouterWarps;  // 8

// One block handles TT consecutive tokens.  Warp w computes experts w, w+8, ...
template <int TT>
__global__ void __launch_bounds__(kRouterWarps * 32)
router_topk_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ w_r,
                   const float *__restrict__ bias, const int32_t *__restrict__ token_seq,
                   int T, int d, int E, int k, int32_t *__restrict__ idx,
                   float *__restrict__ gate, float *__restrict__ logits_out)
{
    __shared__ __align__(16) float s_logit[TT][kMaxExperts];
    __shared__ float s_sel[TT][32];
    __shared__ int32_t s_sel_idx[TT][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t0 = blockIdx.x * TT;

    float acc[kMaxExpertsPerWarp][TT];
#pragma unroll
    for (int i = 0; i < kMaxExpertsPerWarp; ++i)
#pragma unroll
        for (int t = 0; t < TT; ++t)
            acc[i][t] = 0.0f;

    const int n_chunks = d >> 8;
#pragma unroll 2
    for (int c = 0; c < n_chunks; ++c) {
        const int col = (c << 8) + (lane << 3);
        // all of this step's loads go out before any arithmetic
        uint4 xv[TT], wvs[kMaxExpertsPerWarp];
#pragma unroll
        for (int t = 0; t < TT; ++t) {
            const int tt = min(t0 + t, T - 1);
            xv[t] = *reinterpret_cast<const uint4 *>(x + (size_t)tt * d + col);
        }
#pragma unroll
        for (int i = 0; i < kMaxExpertsPerWarp; ++i) {
            const int e = warp + i * kRouterWarps;
            wvs[i] = e < E ? __ldg(reinterpret_cast<const uint4 *>(w_r + (size_t)e * d + col)) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int i = 0; i < kMaxExpertsPerWarp; ++i) {
            const int e = warp + i * kRouterWarps;
            if (e < E) {
                const uint4 wv = wvs[i];
#pragma unroll
                for (int t = 0; t < TT; ++t) {
                    float a = acc[i][t];
                    a = __fmaf_rn(bf16lo(xv[t].x), bf16lo(wv.x), a);
                    a = __fmaf_rn(bf16hi(xv[t].x), bf16hi(wv.x), a);
                    a = __fmaf_rn(bf16lo(xv[t].y), bf16lo(wv.y), a);
                    a = __fmaf_rn(bf16hi(xv[t].y), bf16hi(wv.y), a);
                    a = __fmaf_rn(bf16lo(xv[t].z), bf16lo(wv.z), a);
                    a = __fmaf_rn(bf16hi(xv[t].z), bf16hi(wv.z), a);
                    a = __fmaf_rn(bf16lo(xv[t].w), bf16lo(wv.w), a);
                    a = __fmaf_rn(bf16hi(xv[t].w), bf16hi(wv.w), a);
                    acc[i][t] = a;
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kMaxExpertsPerWarp; ++i) {
        const int e = warp + i * kRouterWarps;
#pragma unroll
        for (int t = 0; t < TT; ++t) {
            float a = acc[i][t];
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1)
                a = __fadd_rn(a, __shfl_xor_sync(0xffffffffu, a, m));
            if (lane == 0 && e < E && t0 + t < T) {
                if (bias) {
                    const int q = token_seq ? token_seq[t0 + t] : 0;
                    a = __fadd_rn(a, bias[(size_t)q * E + e]);
                }
                s_logit[t][e] = a;
                if (logits_out)
                    logits_out[(size_t)(t0 + t) * E + e] = a;
            }
        }
    }
    __syncthreads();

    // top-k: warp t of the block serves token t0 + t.  Lane l holds experts l and l + 32.
    if (warp < TT && t0 + warp < T) {
        const int t = t0 + warp;
        const float NEG = -__int_as_float(0x7f800000);  // -inf
        // an element's rank is the number of elements that beat it (greater, or equal with a lower
        // index); the k elements of rank below k are the selection, in order
        const float v0 = lane < E ? s_logit[warp][lane] : NEG;
        const float v1 = lane + 32 < E ? s_logit[warp][lane + 32] : NEG;
        int r0 = 0, r1 = 0;
        const float4 *row = reinterpret_cast<const float4 *>(s_logit[warp]);
#pragma unroll
        for (int i = 0; i < kMaxExperts / 4; ++i) {
            const float4 o4 = row[i];
            const float ov[4] = {o4.x, o4.y, o4.z, o4.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int e = 4 * i + c;
                const float o = e < E ? ov[c] : NEG;     // the row's tail beyond E was never written
                r0 += (o > v0) || (o == v0 && e < lane);
                r1 += (o > v1) || (o == v1 && e < lane + 32);
            }
        }
        if (lane < E && r0 < k) {
            s_sel[warp][r0] = v0;
            s_sel_idx[warp][r0] = lane;
        }
        if (lane + 32 < E && r1 < k) {
            s_sel[warp][r1] = v1;
            s_sel_idx[warp][r1] = lane + 32;
        }
        __syncwarp();
        const float top = s_sel[warp][0];
        const float my_sel = lane < k ? s_sel[warp][lane] : 0.0f;
        const int my_idx = lane < k ? s_sel_idx[warp][lane] : 0;
        float ev = lane < k ? expf(my_sel - top) : 0.0f;
        float sum = ev;
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1)
            sum += __shfl_xor_sync(0xffffffffu, sum, m);
        if (lane < k) {
            idx[(size_t)t * k + lane] = my_idx;
            gate[(size_t)t * k + lane] = ev / sum;
        }
    }
}

}  // namespace

cudaError_t launch_router(cudaStream_t stream, const uint16_t *x, const uint16_t *w_r,
                          const float *bias, const int32_t *token_seq, int T, int d, int E, int k,
                          int32_t *idx, float *gate, float *logits_out)
{
    // one token per block while that still fills the GPU no more than twice over
    if (T <= 296) {
        router_topk_kernel<1><<<T, kRouterWarps * 32, 0, stream>>>(x, w_r, bias, token_seq, T, d, E, k,
                                                                    idx, gate, logits_out);
    } else {
        router_topk_kernel<4><<<(T + 3) / 4, kRouterWarps * 32, 0, stream>>>(x, w_r, bias, token_seq, T, d,
                                                                              E, k, idx, gate, logits_out);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace melinoe
