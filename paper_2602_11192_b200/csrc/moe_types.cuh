// Shared host/device structures of the cached-MoE-layer library (sm_100a).
//
// Nothing here is seen by the CPU oracle; the two implementations share no code.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace melinoe {

constexpr int kMaxExperts = 64;          // routed experts per layer (need-set is one 64-bit mask)
constexpr int kMaxShared = 8;            // always-resident shared experts
constexpr int kMaxReq = kMaxExperts + kMaxShared;
constexpr int kMaxGroups = kMaxExperts + 2;  // 1 + ceil(E / C) with C >= 1
constexpr int kTokPerVr = 8;             // tokens per virtual request of the streaming FFN kernel
constexpr int kUnitRows = 8;             // d_ff must be a multiple of this (one phase-1 tile of the FFN kernel)

// Persistent cache state of one layer (device memory).  The reading of "LRU" used here:
// every request takes stamp = ++counter; a hit re-stamps its slot; a miss takes the lowest
// empty slot, else the slot with the smallest stamp.
struct DevCache {
    int32_t expert_of_slot[kMaxExperts];   // -1 = empty
    int32_t slot_of_expert[kMaxExperts];   // -1 = not resident
    uint64_t stamp[kMaxExperts];
    uint64_t counter;
    uint64_t tot_hits, tot_misses, tot_evictions;
    uint64_t call_no;
    uint64_t tot_vr;                        // virtual requests handed to the FFN kernels so far
    // gamma-discounted request count of every expert (Definition C.1), kept for the count policy:
    // one step per forward call, count <- gamma * count + (requested ? 1 : 0), fp32, the product
    // rounded before the sum
    float count[kMaxExperts];
};

// One cache request of a call plus what the compute kernels need to serve it.
struct ReqRec {
    int32_t expert;    // routed: 0..E-1; shared: E + s
    int32_t slot;      // cache slot, or -1 for a shared expert
    int32_t hit;
    int32_t evicted;   // expert displaced by this request, or -1
    int32_t tok_off;   // first entry of this expert's token list in the sorted arrays
    int32_t n_tok;     // tokens routed to it
    int32_t vr_start;  // first virtual request (global index within the call)
    int32_t group;     // compute group: 0 = resident at call entry, g >= 1 = g-th miss wave
};

// A virtual request: up to kTokPerVr tokens of one expert, with everything the FFN kernel
// needs to serve it in one 80-byte record (one dependent load instead of a chain of them).
struct __align__(16) VrRec {
    const char *blob;            // the expert's weights: its cache slot, or a shared expert's blob
    int32_t n_tok;               // 1..kTokPerVr
    int32_t group;
    int32_t tok[kTokPerVr];      // token (row of hidden) of each slot, -1 beyond n_tok
    int32_t pair[kTokPerVr];     // row of the z buffer: t * k + j for routed pairs, T*k + s*T + t for shared
};

// Per-call plan written by the planning kernel, read by the FFN and combine kernels.
struct DevPlan {
    int32_t n_tokens, n_req, n_hits, n_miss, n_evict, n_groups, n_vr, status;
    int32_t group_vr_begin[kMaxGroups + 1];
    int32_t counts[kMaxReq];
    int32_t offsets[kMaxReq + 1];
    int32_t req_of_expert[kMaxReq];        // -1 = expert not requested by this call
    ReqRec req[kMaxReq];
};

// The miss queue of a call: what the host needs in order to issue the transfers, written by
// the planning kernel into page-locked host memory.  Every 16-byte record carries the call's
// sequence number and is written with one 16-byte store, so a record is valid exactly when its
// seq field matches and no fence is needed between records (a system-wide fence costs several
// microseconds over the host link).
struct __align__(16) HostMiss {
    int32_t expert, slot;
    int16_t group, dep_group;    // dep_group: compute group that must finish first, or -1
    uint32_t seq;
};
struct __align__(16) HostPlanHeader {
    int32_t n_miss, n_groups, status;
    uint32_t seq;
};
struct __align__(16) HostPlan {
    HostPlanHeader hdr;
    HostMiss miss[kMaxExperts];
};

// Device side: publish the miss queue of call `seq` (one 16-byte store per record).
__device__ inline void store16_host(void *dst, const void *rec)
{
    const int4 v = *reinterpret_cast<const int4 *>(rec);
    asm volatile("st.volatile.global.v4.s32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
__device__ inline void publish_miss_queue(HostPlan *hp, const HostMiss *miss, int n_miss, int n_groups, int status,
                                          uint32_t seq)
{
    for (int i = 0; i < n_miss; ++i) {
        HostMiss m = miss[i];
        m.seq = seq;
        store16_host(&hp->miss[i], &m);
    }
    HostPlanHeader h{n_miss, n_groups, status, seq};
    store16_host(&hp->hdr, &h);
}

}  // namespace melinoe
