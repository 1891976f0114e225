// Forward-only evaluation of the paper's cache-miss proxies over a recorded routing trace
// (Section 3.1: the soft cache state of the cache simulation loss L_cs; Definition C.1: the hard
// gamma-discounted Top-C cache, whose misses are the transfers of Appendix C.1).  One warp per
// configuration (layer, cache size, gamma) walks the layer's tokens in order; lane l owns experts
// l and l + 32.  Everything is fp64 and in the order the definitions state, so the hard misses
// (an integer result) are exact and the soft proxy differs from a straightforward evaluation only
// by the order of a 64-term sum.
//
//   soft:  c starts at 0 and follows c <- gamma c + r while its L1 norm stays below C; the first
//          update that reaches C is rescaled to norm C and starts the normaliser Z = 1; from then
//          on c <- (gamma Z c + r) / Z', Z' = gamma Z + K / C.  proxy_t = sum_i r_i (1 - c_i).
//   hard:  count starts at 0, count <- gamma count + r; the cache holds the up to C experts of
//          largest non-zero count (lower index first among equals); miss_t = requested experts
//          outside it.
#include "kernels.cuh"

namespace melinoe {

namespace {

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1)
        v += __shfl_xor_sync(0xffffffffu, v, m);
    return v;
}

__global__ void __launch_bounds__(32) miss_proxy_kernel(const int32_t *__restrict__ idx, int n_layers, int T, int K, int E,
                                                        const melinoe_proxy_config *__restrict__ cfgs, int n_cfg,
                                                        double *__restrict__ soft_mean, long long *__restrict__ hard_total)
{
    __shared__ double s_count[kMaxExperts];
    const int lane = threadIdx.x;
    const int ci = blockIdx.x;
    if (ci >= n_cfg)
        return;
    const melinoe_proxy_config cfg = cfgs[ci];
    const int C = cfg.cache_slots;
    const double gamma = cfg.gamma;
    if (cfg.layer < 0 || cfg.layer >= n_layers || C < 1 || C > E || !(gamma >= 0.0 && gamma <= 1.0)) {
        if (lane == 0) {       // a configuration that names nothing: marked, not evaluated
            soft_mean[ci] = __longlong_as_double(0x7ff8000000000000ll);
            hard_total[ci] = -1;
        }
        return;
    }
    const int32_t *trace = idx + (size_t)cfg.layer * T * K;
    const int e0 = lane, e1 = lane + 32;
    double c0 = 0.0, c1 = 0.0, n0 = 0.0, n1 = 0.0, Z = 1.0;
    bool filled = false;
    double soft = 0.0;
    long long hard = 0;
    for (int t = 0; t < T; ++t) {
        // request vector of the token
        bool r0 = false, r1 = false;
        for (int j = 0; j < K; ++j) {
            const int e = trace[(size_t)t * K + j];
            r0 |= e == e0;
            r1 |= e == e1;
        }
        const double q0 = r0 ? 1.0 : 0.0, q1 = r1 ? 1.0 : 0.0;
        soft += warp_sum(q0 * (1.0 - c0) + q1 * (1.0 - c1));
        // hard cache: rank of this lane's experts among the non-zero counts
        s_count[e0] = n0;
        s_count[e1] = n1;
        __syncwarp();
        int k0 = 0, k1 = 0;
        for (int e = 0; e < E; ++e) {
            const double o = s_count[e];
            k0 += (o > n0) || (o == n0 && e < e0);
            k1 += (o > n1) || (o == n1 && e < e1);
        }
        __syncwarp();
        const bool in0 = e0 < E && n0 > 0.0 && k0 < C, in1 = e1 < E && n1 > 0.0 && k1 < C;
        hard += __popc(__ballot_sync(0xffffffffu, r0 && !in0)) + __popc(__ballot_sync(0xffffffffu, r1 && !in1));
        // updates
        if (!filled) {
            double a0 = gamma * c0 + q0, a1 = gamma * c1 + q1;
            const double norm = warp_sum(a0 + a1);
            if (norm >= (double)C) {
                a0 *= (double)C / norm;
                a1 *= (double)C / norm;
                filled = true;
                Z = 1.0;
            }
            c0 = a0;
            c1 = a1;
        } else {
            const double Zn = gamma * Z + (double)K / (double)C;
            c0 = (gamma * Z * c0 + q0) / Zn;
            c1 = (gamma * Z * c1 + q1) / Zn;
            Z = Zn;
        }
        // product rounded before the sum (no contraction): the hard cache's decisions hang on these bits
        n0 = __dadd_rn(__dmul_rn(gamma, n0), q0);
        n1 = __dadd_rn(__dmul_rn(gamma, n1), q1);
    }
    if (lane == 0) {
        soft_mean[ci] = T > 0 ? soft / (double)T : 0.0;
        hard_total[ci] = hard;
    }
}

}  // namespace

cudaError_t launch_miss_proxies(cudaStream_t stream, const int32_t *idx, int n_layers, int T, int K, int E,
                                const melinoe_proxy_config *cfgs, int n_cfg, double *soft_mean, long long *hard_total)
{
    miss_proxy_kernel<<<n_cfg, 32, 0, stream>>>(idx, n_layers, T, K, E, cfgs, n_cfg, soft_mean, hard_total);
    count_launch();
    return cudaGetLastError();
}

}  // namespace melinoe
