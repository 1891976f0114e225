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
    const char *slots;        // device cache (slot s at slots + s * slot_stride)
    size_t slot_stride;
    const char *const *shared_blobs;
    const char *const *host_blobs;   // device array [E]: every expert's blob in the host store as the device
                                     // sees it (null entries, or a null array: the store cannot be read from kernels)
    int32_t *perm, *inv_pos, *tok_of_sorted;
    HostPlan *hplan;          // page-locked host memory (device-visible address)
    uint32_t gmax;            // compute groups the caller has room for
    uint32_t call_seq;        // written to the miss queue's seq word when the record is complete
    int policy;               // MELINOE_POLICY_LRU or MELINOE_POLICY_COUNT
    float gamma;              // decay of the count policy
    melinoe_moe_stats *stats; // may be null
    size_t expert_bytes;
    // request trace (melinoe_moe_set_trace): this call's record, or null; see trace_layout()
    char *trace_rec;
    int trace_max_tokens;
    const float *gate;        // [T][k], for the trace record of calls planned by the general kernel
};
// Layout of one request-trace record for a layer of n_experts experts and top_k, max_tokens tokens.
struct TraceLayout {
    size_t req_off, idx_off, gate_off, bytes;
};
__host__ __device__ inline TraceLayout trace_layout(int n_experts, int top_k, int max_tokens)
{
    TraceLayout t;
    t.req_off = sizeof(melinoe_moe_trace_header);
    t.idx_off = t.req_off + (size_t)n_experts * sizeof(melinoe_moe_request);
    t.gate_off = t.idx_off + (size_t)max_tokens * top_k * sizeof(int32_t);
    t.bytes = (t.gate_off + (size_t)max_tokens * top_k * sizeof(float) + 15) / 16 * 16;
    return t;
}
cudaError_t launch_plan(cudaStream_t stream, const PlanParams &p);

// ---- router and planning in one kernel (one thread-block cluster), for calls of at most 8 tokens
bool route_plan_small_supported(int T, int k, int d);
cudaError_t launch_route_plan_small(cudaStream_t stream, const uint16_t *x, const uint16_t *w_r, const float *bias,
                                    const int32_t *token_seq, int d, int32_t *idx, float *gate, float *logits_out,
                                    const PlanParams &p);

// ---- decode expert FFN (Eq. 3) with the gate-weighted combine (Eq. 2) fused in, for up to 8 tokens per launch
struct DecParams {
    const DevPlan *plan;
    const uint16_t *x;               // hidden [T][d] bf16
    const int32_t *idx;              // [T][k]
    const float *gate;               // [T][k]
    long long *yacc;                 // [8][d] output accumulator words of the launch; all zero between launches
    float *ybuf;                     // [T][d] fp32: sum over the earlier launches of the same tokens (group mode)
    uint16_t *out;                   // [T][d] bf16
    unsigned *sync;                  // the handle's counter for the rare launches whose CTAs have to know who is last (zero between launches)
    uint32_t call_seq;               // the call's sequence number: the plan is ready when plan->ready_seq equals it
    int *err;                        // device error word (0 = ok)
    unsigned long long *trace;       // null, or 8 clock stamps per CTA of the most recent launch
    int d, F, E, k, T, n_shared;
    int group;                       // -1: every request of the call in this one launch, the missed experts read
                                     // straight from the host store; g >= 0: compute group g only, from the slots
    int chunk, n_chunks;             // tokens [8 * chunk, 8 * chunk + 8) of the call; launches the call is made in
    int write_back;                  // group -1: store the fetched experts that stay resident into their slots
    int wait_prior;                  // the kernel ahead in the stream is another launch of the same call (it uses the
                                     // same accumulator): wait for that grid to finish before anything else
    int fmt;                         // 0: bf16 blobs, 1: 4-bit blobs
};
struct DecLaunchCfg {
    int grid;                        // one CTA per SM
    size_t max_smem;                 // dynamic shared memory the kernel may use
    bool pdl;                        // launch with programmatic stream serialisation
};
// Shape of the shared-memory ring for one launch.
struct DecGeometry {
    int n_warps;                     // consumer warps (16)
    int tile_rows;                   // f rows per tile = ring stage: at most 8
    int n_stages;
    int row_bytes;                   // bytes of one f row of the blob (its W_g, W_u and W_d^T rows)
    int stage_bytes;
    int x_pitch;                     // bytes between token rows of the staged hidden states
    int tokens;                      // tokens of the launch (1..8)
    int x_tmem;                      // 1: the hidden states' operand fragments live in tensor memory, not in shared memory
    size_t smem_bytes;
};
cudaError_t ffn_decode_configure(int n_sms, size_t max_smem, DecLaunchCfg *cfg);
bool ffn_decode_supported(int d, int F);
bool ffn_decode_supported_q4(int d, int F);
cudaError_t ffn_decode_geometry(const DecLaunchCfg &cfg, int d, int F, int tokens, int fmt, DecGeometry *geo);
cudaError_t launch_ffn_decode(cudaStream_t stream, const DecLaunchCfg &cfg, const DecGeometry &geo,
                              const DecParams &p);

// ---- grouped GEMM expert FFN on tcgen05 for calls with many tokens per expert (prefill)
// Tensor maps in device memory, in this order:
enum {
    kMapXs = 0, kMapHs = 1,                                          // activations: boxes of 128 rows x 64 columns
    kMapSlotsG = 2, kMapSlotsU = 3, kMapSlotsD = 4,                  // W_g, W_u rows (128-row boxes), W_d^T rows (64-row boxes) of all slots
    kMapShared0 = 5,                                                 // per shared expert: the same three views
    kMapCount = kMapShared0 + 3 * kMaxShared
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
cudaError_t launch_ffn_gemm(cudaStream_t stream, int phase, int n_sms, bool pairs, const GemmParams &p);
cudaError_t launch_combine_rows(cudaStream_t stream, const DevPlan *plan, const float *gate, const int32_t *inv_pos,
                                const float *zs, uint16_t *out, int T, int d, int k, int n_shared, int n_sms);

// ---- preload (Eq. 5): cache requests of a list of experts, and the copy of the missing ones into their slots
struct PreloadParams {
    DevCache *cache;
    PreloadList *list;               // device
    PreloadList *host_list;          // page-locked host memory as the device sees it, or null
    int32_t ids[kMaxExperts];
    int n, C, policy;
    uint32_t seq;
};
struct FetchParams {
    const PreloadList *list;
    const char *const *host_blobs;   // device array: the host store as the device sees it
    char *slots;
    size_t slot_stride;
    int rows, row_bytes;             // rows of one expert blob (d_ff) and their size
    int rows_per_piece, piece_bytes; // rows copied at a time (at most 48 KB)
    int *err;
};
cudaError_t launch_preload_plan(cudaStream_t stream, const PreloadParams &p);
cudaError_t launch_fetch_experts(cudaStream_t stream, int n_sms, const FetchParams &p);

// ---- cache-miss proxies of a recorded routing trace (Section 3.1, Definition C.1)
cudaError_t launch_miss_proxies(cudaStream_t stream, const int32_t *idx, int n_layers, int T, int K, int E,
                                const melinoe_proxy_config *cfgs, int n_cfg, double *soft_mean, long long *hard_total);

// ---- 4-bit host store: expand one 4-bit expert (layout in dequant.cu) into a bf16 slot
// ---- decode-sized input from device-mapped host memory into device memory (bytes % 16 == 0)
cudaError_t launch_stage_in(cudaStream_t stream, const void *src_mapped, void *dst, size_t bytes);
cudaError_t launch_dequant_q4(cudaStream_t stream, const void *q4_blob, void *slot, int d, int F, int n_sms);

}  // namespace melinoe
