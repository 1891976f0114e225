// Launch interfaces of the library's kernels (all sm_100a, all launched by api.cu).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/melinoe_moe.h"
#include "moe_types.cuh"

namespace melinoe {

void count_launch();
// Programmatic stream serialisation for the decode kernels (on unless MELINOE_MOE_NO_PDL is set in the environment).
bool pdl_enabled();

// ---- router (Eq. 1): logits, top-k, gates
cudaError_t launch_router(cudaStream_t stream, const uint16_t *x, const uint16_t *w_r,
                          const float *bias, const int32_t *token_seq, int T, int d, int E, int k,
                          int32_t *idx, float *gate, float *logits_out);

// ---- planning: gather lists, LRU slot lookup, miss queue, statistics
struct PlanParams {
    const int32_t *idx;
    int T, k, E, C, n_shared;
    DevCache *cache;
    DevPlan *plan;
    VrRec *vrs;
    const char *slots;        // device cache (slot s at slots + s * slot_stride), for the vrs' blob pointers
    size_t slot_stride;
    const char *const *shared_blobs;
    int32_t *perm, *inv_pos, *tok_of_sorted;
    HostPlan *hplan;          // page-locked host memory (device-visible address)
    unsigned *sync;           // grid-barrier counters of the FFN launches, zeroed here
    uint32_t gmax;            // compute groups the caller has room for
    uint32_t call_seq;        // written to the miss queue's seq word when the record is complete
    int policy;               // MELINOE_POLICY_LRU or MELINOE_POLICY_COUNT
    float gamma;              // decay of the count policy
    melinoe_moe_stats *stats; // may be null
    size_t expert_bytes;
    int vr_capacity;
};
cudaError_t launch_plan(cudaStream_t stream, const PlanParams &p);

// ---- router and planning in one kernel (one thread-block cluster), for calls of at most 8 tokens
bool route_plan_small_supported(int T, int k, int d);
cudaError_t launch_route_plan_small(cudaStream_t stream, const uint16_t *x, const uint16_t *w_r, const float *bias,
                                    const int32_t *token_seq, int d, int32_t *idx, float *gate, float *logits_out,
                                    const PlanParams &p);

// ---- streaming expert FFN (Eq. 3) with the gate-weighted combine (Eq. 2) fused in
struct FfnParams {
    const DevPlan *plan;
    const VrRec *vrs;
    const uint16_t *x;               // hidden [T][d] bf16
    const float *gate;               // [T][k]
    uint16_t *hbuf;                  // h = SiLU(g) * u: [virtual request][8 token slots][Fpad] bf16
    float *zbuf;                     // expert outputs: [T*k routed pairs, then n_shared*T][d] fp32
    uint16_t *out;                   // [T][d] bf16
    unsigned *sync;                  // grid-barrier counters, one per compute group (zero at launch)
    int *err;                        // device error word (0 = ok)
    unsigned long long *trace;       // null, or 8 clock stamps per CTA of the most recent launch
    int d, F, Fpad, E, k, T, n_shared;
    int group;
};
struct FfnLaunchCfg {
    int grid;                        // one CTA per SM
    size_t max_smem;                 // dynamic shared memory the kernel may use
    bool pdl;                        // launch with programmatic stream serialisation
};
// Shape of the shared-memory ring for one call.
struct FfnGeometry {
    int n_op_rows;                   // operand rows per stage: min(T, 8)
    int n_stages, stage_bytes;       // the ring
    int pitch, chunk_bytes;          // gate/up phase: row pitch in a stage, bytes per row piece (rows of 2*d bytes)
    int pitch2, chunk_bytes2;        // down phase (rows of 2*d_ff bytes)
    int sub2, sub_bytes2;            // down phase: sub-stages per ring slot and their size
    int rows2;                       // down phase: weight rows of a sub-stage, min(16, ceil(d / grid)); the h rows follow
    size_t ring_bytes, smem_bytes;
};
cudaError_t ffn_stream_configure(int n_sms, size_t max_smem, FfnLaunchCfg *cfg);
cudaError_t ffn_stream_geometry(const FfnLaunchCfg &cfg, int d, int F, int T, FfnGeometry *geo);
cudaError_t launch_ffn_stream(cudaStream_t stream, const FfnLaunchCfg &cfg, const FfnGeometry &geo,
                              const FfnParams &p);

// ---- grouped GEMM expert FFN on tcgen05 for calls with many tokens per expert (prefill)
// Tensor maps in device memory, in this order:
enum {
    kMapXs = 0, kMapHs = 1, kMapSlotsD = 2, kMapSlotsF = 3,          // boxes of 128, 128, 128 and 256 rows
    kMapShared0 = 4,                                                 // per shared expert: rows of d (128), rows of F (256)
    kMapSlotsF128 = kMapShared0 + 2 * kMaxShared,                    // rows of F in boxes of 128 rows (CTA-pair kernel)
    kMapSharedF128 = kMapSlotsF128 + 1,                              // the same per shared expert
    kMapCount = kMapSharedF128 + kMaxShared
};
struct GemmParams {
    const DevPlan *plan;
    const CUtensorMap *maps;         // device array of kMapCount tensor maps
    uint16_t *hs;                    // h, [sorted rows][F] bf16
    float *zs;                       // expert outputs, [sorted rows][d] fp32
    int *err;
    int group, d, F, E, n_shared;
};
bool ffn_gemm_supported(int d, int F);
cudaError_t ffn_gemm_configure();
cudaError_t launch_gather_rows(cudaStream_t stream, const DevPlan *plan, const uint16_t *x, const int32_t *tok_of_sorted,
                               uint16_t *xs, int d, int n_sorted, int n_sms);
cudaError_t launch_ffn_gemm(cudaStream_t stream, int phase, int n_sms, const GemmParams &p);
// the same two GEMMs on CTA pairs (tcgen05.mma.cta_group::2), for calls with many tokens per expert
cudaError_t ffn_gemm_pair_configure();
cudaError_t launch_ffn_gemm_pair(cudaStream_t stream, int phase, int n_sms, const GemmParams &p);
cudaError_t launch_combine_rows(cudaStream_t stream, const DevPlan *plan, const float *gate, const int32_t *inv_pos,
                                const float *zs, uint16_t *out, int T, int d, int k, int n_shared, int n_sms);

// ---- cache-miss proxies of a recorded routing trace (Section 3.1, Definition C.1)
cudaError_t launch_miss_proxies(cudaStream_t stream, const int32_t *idx, int n_layers, int T, int K, int E,
                                const melinoe_proxy_config *cfgs, int n_cfg, double *soft_mean, long long *hard_total);

// ---- 4-bit host store: expand one 4-bit expert (layout in dequant.cu) into a bf16 slot
// ---- decode-sized input from device-mapped host memory into device memory (bytes % 16 == 0)
cudaError_t launch_stage_in(cudaStream_t stream, const void *src_mapped, void *dst, size_t bytes);
cudaError_t launch_dequant_q4(cudaStream_t stream, const void *q4_blob, void *slot, int d, int F, int n_sms);

}  // namespace melinoe
