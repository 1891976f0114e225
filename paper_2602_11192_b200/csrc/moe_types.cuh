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
constexpr int kTokPerVr = 8;             // tokens one launch of the decode FFN kernel serves (its mma N dimension)
constexpr int kUnitRows = 8;             // d_ff must be a multiple of this (the row swizzle of the expert blob has period 8)

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
    uint64_t reserved0;
    // gamma-discounted request count of every expert (Definition C.1), kept for the count policy:
    // one step per forward call, count <- gamma * count + (requested ? 1 : 0), fp32, the product
    // rounded before the sum
    float count[kMaxExperts];
};

// One cache request of a call plus what the compute kernels need to serve it.
struct __align__(16) ReqRec {
    int32_t expert;    // routed: 0..E-1; shared: E + s
    int32_t slot;      // cache slot, or -1 for a shared expert
    int32_t hit;
    int32_t evicted;   // expert displaced by this request, or -1
    int32_t vr_start;  // its entry of DevPlan::dreq
    int32_t group;     // compute group: 0 = resident at call entry, g >= 1 = g-th miss wave
    int32_t tok_off;   // first entry of this expert's token list in the sorted arrays
    int32_t n_tok;     // tokens routed to it
};

// What the decode FFN kernel needs to serve one request (one distinct expert of the call, or a
// shared expert): where its weights are and what has to happen to them.  One 32-byte record, read
// with one load.
struct __align__(32) DecReq {
    const char *blob;            // the expert's cache slot, or a shared expert's blob (device memory)
    const char *host;            // the expert's blob in the page-locked host store as the device sees it, or null
    int32_t expert;              // routed: 0..E-1; shared: E + s
    int32_t flags;               // kDecMiss | kDecStays | kDecHazard
    int32_t group;               // compute group (0 = resident at call entry or shared, g >= 1 = g-th miss wave)
    int32_t reserved;
};
constexpr int kDecMiss = 1;      // not resident at call entry: the weights come from the host store
constexpr int kDecStays = 2;     // a miss that still occupies its slot when the call ends: written into the slot
constexpr int kDecHazard = 4;    // ... whose slot held, at call entry, an expert that this call also computes with

// Per-call plan written by the planning kernel, read by the FFN and combine kernels.
struct DevPlan {
    int32_t n_tokens, n_req, n_hits, n_miss, n_evict, n_groups, n_dreq, status;
    // Sequence number of the call whose plan this is, written last (after a device-wide fence) by the
    // planning kernel: the decode FFN kernel, which may have been scheduled while the planner was still
    // running, waits for it instead of waiting for the planner's grid to drain.
    uint32_t ready_seq;
    uint32_t pad_[3];
    int32_t group_vr_begin[kMaxGroups + 1];   // first entry of dreq[] of every compute group
    int32_t counts[kMaxReq];
    int32_t offsets[kMaxReq + 1];
    int32_t req_of_expert[kMaxReq];        // -1 = expert not requested by this call
    ReqRec req[kMaxReq];
    DecReq dreq[kMaxReq];                     // group 0 (hits, then shared experts), then the misses by wave
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

// What a preload has to fetch, written by its planning kernel: device copy for the fetch kernel,
// and a copy in page-locked host memory (seq written last) where the host issues the copies.
struct PreloadList {
    int32_t n;
    uint32_t seq;
    int32_t expert[kMaxExperts];
    int32_t slot[kMaxExperts];
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
