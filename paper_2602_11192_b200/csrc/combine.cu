// Gate-weighted combine (Eq. 2): y_t = sum_j gate[t][j] * z[t][j] (+ shared experts, gate 1),
// accumulated in fp32 in rank order and rounded once to bf16.
//
// The streaming FFN kernel leaves, for every virtual request, one partial row set per CTA
// that covered a piece of it; the partials of a request sit in consecutive row sets and are
// added here in ascending CTA order, so the result does not depend on scheduling.
#include "kernels.cuh"

namespace melinoe {

namespace {

__device__ __forceinline__ uint32_t bf16_rne(float v)
{
    uint32_t u = __float_as_uint(v);
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

__global__ void __launch_bounds__(256) combine_kernel(CombineParams p)
{
    const int t = blockIdx.y;
    const int col = (blockIdx.x * 256 + threadIdx.x) * 4;
    if (col >= p.d)
        return;
    const DevPlan *plan = p.plan;
    float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
    if (plan->status == MELINOE_OK) {
        for (int j = 0; j < p.k + p.n_shared; ++j) {
            int e, pos;
            float gw;
            if (j < p.k) {
                const int pair = t * p.k + j;
                e = p.idx[pair];
                gw = p.gate[pair];
                pos = p.inv_pos[pair];
            } else {
                e = p.E + (j - p.k);
                gw = 1.0f;
                pos = p.T * p.k + (j - p.k) * p.T + t;
            }
            const ReqRec rec = plan->req[plan->req_of_expert[e]];
            const int ie = pos - rec.tok_off;
            const int vr = rec.vr_start + ie / kTokPerVr;
            const int tpos = ie % kTokPerVr;
            const int vb = plan->group_vr_begin[rec.group];
            const long long nu = (long long)(plan->group_vr_begin[rec.group + 1] - vb) * p.units_per_vr;
            const long long ua = (long long)(vr - vb) * p.units_per_vr;
            const long long geff = nu < p.grid ? nu : (long long)p.grid;  // CTAs the launch really used
            const int c0 = cta_of_unit(ua, nu, geff);
            const int c1 = cta_of_unit(ua + p.units_per_vr - 1, nu, geff);
            float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int c = c0; c <= c1; ++c) {
                const long long row = ((long long)rec.group * p.grid + c + vr) * kTokPerVr + tpos;
                const float4 v = *reinterpret_cast<const float4 *>(p.part + row * p.d + col);
                z.x += v.x;
                z.y += v.y;
                z.z += v.z;
                z.w += v.w;
            }
            y.x = fmaf(gw, z.x, y.x);
            y.y = fmaf(gw, z.y, y.y);
            y.z = fmaf(gw, z.z, y.z);
            y.w = fmaf(gw, z.w, y.w);
        }
    }
    uint2 o;
    o.x = bf16_rne(y.x) | (bf16_rne(y.y) << 16);
    o.y = bf16_rne(y.z) | (bf16_rne(y.w) << 16);
    *reinterpret_cast<uint2 *>(p.out + (size_t)t * p.d + col) = o;
}

}  // namespace

cudaError_t launch_combine(cudaStream_t stream, const CombineParams &p)
{
    dim3 grid((p.d / 4 + 255) / 256, p.T);
    combine_kernel<<<grid, 256, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace melinoe
