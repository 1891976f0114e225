// Launch interfaces of the library's kernels (all sm_100a, all launched by api.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/melinoe_moe.h"
#include "moe_types.cuh"

namespace melinoe {

void count_launch();

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
    int32_t *perm, *inv_pos, *tok_of_sorted;
    HostPlan *hplan;          // page-locked host memory (device-visible address)
    uint32_t gmax;            // compute groups the caller has room for
    uint32_t call_seq;        // written to the miss queue's seq word when the record is complete
    melinoe_moe_stats *stats; // may be null
    size_t expert_bytes;
    int vr_capacity;
};
cudaError_t launch_plan(cudaStream_t stream, const PlanParams &p);

// ---- streaming expert FFN (Eq. 3) for calls with few tokens per expert
struct FfnParams {
    const char *slots;               // device cache: slot s at slots + s * slot_stride
    size_t slot_stride;
    const char *const *shared_blobs; // device array of shared-expert blobs, or null
    const DevPlan *plan;
    const VrRec *vrs;
    const int32_t *tok_of_sorted;
    const uint16_t *x;               // hidden [T][d] bf16
    float *part;                     // partial outputs, rows of d floats
    int *err;                        // device error word (0 = ok)
    int d, F, E;
    int group;
};
struct FfnLaunchCfg {
    int grid, rows_per_entry, n_stages;
    size_t smem_bytes;
};
bool ffn_stream_supported(int d);
cudaError_t ffn_stream_configure(int d, int n_sms, size_t max_smem, FfnLaunchCfg *cfg);
cudaError_t launch_ffn_stream(cudaStream_t stream, const FfnLaunchCfg &cfg, const FfnParams &p);

// ---- gate-weighted combine (Eq. 2) over the streaming kernel's partial outputs
struct CombineParams {
    const DevPlan *plan;
    const int32_t *idx;
    const float *gate;
    const int32_t *inv_pos;
    const float *part;
    uint16_t *out;                   // [T][d] bf16
    int T, d, k, E, n_shared, grid, units_per_vr;
};
cudaError_t launch_combine(cudaStream_t stream, const CombineParams &p);

}  // namespace melinoe
