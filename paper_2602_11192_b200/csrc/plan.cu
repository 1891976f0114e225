// Planning kernel: token-to-expert gather, slot lookup with LRU eviction, miss queue.
//
// One block per call.  It turns the router's indices into
//   (a) per-expert token lists (stable counting sort of the (token, rank) pairs),
//   (b) the call's cache requests: one per distinct expert, experts resident at call entry
//       first (ascending id), then the missing ones (ascending id); a miss takes the lowest
//       empty slot, else the least recently stamped slot (Section 3.2: experts are fetched on
//       demand, "evicting cached experts as dictated by the cache policy"; the policy is LRU),
//   (c) compute groups: group 0 = resident experts (+ shared experts); the misses follow in
//       waves, a new wave starting whenever a miss would overwrite an expert of the current
//       wave, so every wave's transfers can be in flight while earlier groups compute,
//   (d) the miss queue, in page-locked host memory, from which the host issues the transfers, and
//   (e) the call's statistics (hard miss count of Appendix C.1).
#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kPlanThreads = 1024;
constexpr int kPlanWarps = kPlanThreads / 32;

__global__ void __launch_bounds__(kPlanThreads) plan_kernel(PlanParams p)
{
    __shared__ int32_t s_counts[kMaxReq];
    __shared__ int32_t s_offsets[kMaxReq + 1];
    __shared__ int32_t s_running[kMaxExperts];
    __shared__ int32_t s_warp_cnt[kPlanWarps][kMaxExperts];
    __shared__ DevCache s_cache;
    __shared__ int32_t s_group_of_expert[kMaxExperts];
    __shared__ int32_t s_req_of_expert[kMaxReq];
    __shared__ ReqRec s_req[kMaxReq];
    __shared__ HostMiss s_miss[kMaxExperts];
    __shared__ int32_t s_group_vr_begin[kMaxGroups + 1];
    __shared__ unsigned long long s_key[kMaxExperts];            // victim-order key of a slot
    __shared__ int32_t s_victim[kMaxExperts];                    // V: slots in victim order
    __shared__ int32_t s_miss_expert[kMaxExperts];               // expert of miss number i
    __shared__ int32_t s_entry_occ[kMaxExperts];                 // occupant of a slot at call entry
    __shared__ int32_t s_miss_flags[kMaxExperts];                // kDecStays / kDecHazard of miss number i
    __shared__ int32_t s_misc[8];  // 0 n_req(routed) 1 n_hits 2 n_miss 3 n_evict 4 n_groups 5 n_dreq 6 status 7 n_req_total

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_pairs = p.T * p.k;
    const int E = p.E, C = p.C;

    // ---- load persistent cache state, clear tables
    {
        const uint32_t *src = reinterpret_cast<const uint32_t *>(p.cache);
        uint32_t *dst = reinterpret_cast<uint32_t *>(&s_cache);
        for (int i = tid; i < (int)(sizeof(DevCache) / 4); i += kPlanThreads)
            dst[i] = src[i];
    }
    for (int i = tid; i < kMaxReq; i += kPlanThreads) {
        s_counts[i] = 0;
        s_req_of_expert[i] = -1;
    }
    if (tid < 8)
        s_misc[tid] = 0;
    __syncthreads();

    // ---- (a) histogram
    for (int q = tid; q < n_pairs; q += kPlanThreads) {
        const int e = p.idx[q];
        if (e >= 0 && e < E)
            atomicAdd(&s_counts[e], 1);
        else
            s_misc[6] = MELINOE_ERR_INVALID;
    }
    __syncthreads();
    // count policy (Definition C.1): one time step per call, count <- gamma * count + request
    if (p.policy == MELINOE_POLICY_COUNT && tid < E)
        s_cache.count[tid] = __fadd_rn(__fmul_rn(p.gamma, s_cache.count[tid]), s_counts[tid] > 0 ? 1.0f : 0.0f);
    if (tid == 0) {
        int run = 0;
        for (int e = 0; e < E; ++e) {
            s_offsets[e] = run;
            s_running[e] = run;
            run += s_counts[e];
        }
        for (int s = 0; s < p.n_shared; ++s) {
            s_counts[E + s] = p.T;
            s_offsets[E + s] = run;
            run += p.T;
        }
        s_offsets[E + p.n_shared] = run;
    }
    __syncthreads();

    // ---- stable scatter, kPlanThreads pairs per pass, in pair order
    for (int base = 0; base < n_pairs; base += kPlanThreads) {
        for (int i = tid; i < kPlanWarps * kMaxExperts; i += kPlanThreads)
            (&s_warp_cnt[0][0])[i] = 0;
        __syncthreads();
        const int q = base + tid;
        int e = q < n_pairs ? p.idx[q] : kMaxExperts;
        if (e < 0 || e >= E)
            e = kMaxExperts;  // invalid or padding: takes no part
        const unsigned same = __match_any_sync(0xffffffffu, e);
        const int rank = __popc(same & ((1u << lane) - 1u));
        if (e < kMaxExperts && rank == 0)
            s_warp_cnt[warp][e] = __popc(same);
        __syncthreads();
        if (tid < E) {
            int run = 0;
            for (int w = 0; w < kPlanWarps; ++w) {
                const int c = s_warp_cnt[w][tid];
                s_warp_cnt[w][tid] = run;
                run += c;
            }
            s_group_of_expert[tid] = run;  // scratch: this pass's total for expert tid
        }
        __syncthreads();
        if (e < kMaxExperts) {
            const int pos = s_running[e] + s_warp_cnt[warp][e] + rank;
            p.perm[pos] = q;
            p.inv_pos[q] = pos;
            p.tok_of_sorted[pos] = q / p.k;
        }
        __syncthreads();
        if (tid < E)
            s_running[tid] += s_group_of_expert[tid];
        __syncthreads();
    }
    for (int i = tid; i < p.n_shared * p.T; i += kPlanThreads)
        p.tok_of_sorted[n_pairs + i] = i % p.T;

    // ---- (b), (c): cache requests, by warp 0; lane owns experts lane and lane + 32 and slots lane and
    // lane + 32.  The sequential rules (hits in ascending id, then misses in ascending id, a miss
    // takes the lowest empty slot, else the least recently stamped one; a new wave starts when a
    // miss would overwrite an expert of the current wave) have a closed form:
    //   - hit number r (ascending id) stamps its slot with counter + r + 1;
    //   - let V be the slots ordered by (empty first, by index), then by stamp after the hits were
    //     stamped; miss number i (ascending id) takes V[i mod C], because every slot it could prefer
    //     has either been taken by an earlier miss (and stamped newer) or comes later in V;
    //   - the expert it displaces is V[i]'s occupant at call entry for i < C, and miss i - C otherwise;
    //   - miss i belongs to wave 1 + i / C; it must wait for group i / C (i >= C), for group 0 if it
    //     displaces one of the call's hits, for nothing otherwise.
    if (warp == 0) {
        const int e0 = lane, e1 = lane + 32;
        const int c0 = e0 < E ? s_counts[e0] : 0, c1 = e1 < E ? s_counts[e1] : 0;
        const int soe0 = e0 < E ? s_cache.slot_of_expert[e0] : -1, soe1 = e1 < E ? s_cache.slot_of_expert[e1] : -1;
        const int eos0 = lane < C ? s_cache.expert_of_slot[lane] : -1, eos1 = lane + 32 < C ? s_cache.expert_of_slot[lane + 32] : -1;
        const uint64_t st0 = lane < C ? s_cache.stamp[lane] : 0ull, st1 = lane + 32 < C ? s_cache.stamp[lane + 32] : 0ull;
        uint64_t counter = s_cache.counter;
        auto ballot64 = [](bool lo, bool hi) {
            return (uint64_t)__ballot_sync(0xffffffffu, lo) | ((uint64_t)__ballot_sync(0xffffffffu, hi) << 32);
        };
        auto rank_below = [](uint64_t mask, int bit) { return __popcll(mask & ((1ull << bit) - 1ull)); };
        const uint64_t need = ballot64(c0 > 0, c1 > 0);
        const uint64_t resident = ballot64(soe0 >= 0, soe1 >= 0);
        const uint64_t hit_mask = need & resident, miss_mask = need & ~resident;
        const int n_hits = __popcll(hit_mask), n_miss = __popcll(miss_mask), n_req = n_hits + n_miss;
        __syncwarp();
        s_key[lane] = lane < C ? (eos0 < 0 ? (uint64_t)lane : ((1ull << 63) | st0)) : ~0ull;
        s_key[lane + 32] = lane + 32 < C ? (eos1 < 0 ? (uint64_t)(lane + 32) : ((1ull << 63) | st1)) : ~0ull;
        s_entry_occ[lane] = eos0;
        s_entry_occ[lane + 32] = eos1;
        __syncwarp();
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int e = h ? e1 : e0, soe = h ? soe1 : soe0;
            if ((hit_mask >> e) & 1ull) {
                const int r = rank_below(hit_mask, e);
                const uint64_t st = counter + (uint64_t)r + 1ull;
                s_key[soe] = (1ull << 63) | st;
                s_cache.stamp[soe] = st;
                s_req[r] = ReqRec{e, soe, 1, -1, 0, 0, s_offsets[e], s_counts[e]};
                s_req_of_expert[e] = r;
                s_group_of_expert[e] = 0;
            }
            if ((miss_mask >> e) & 1ull)
                s_miss_expert[rank_below(miss_mask, e)] = e;
        }
        __syncwarp();
        // V: rank of each slot among the keys (keys are distinct); only misses under LRU take victims from it
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int sl = lane + 32 * h;
            if (sl < C && n_miss > 0 && p.policy != MELINOE_POLICY_COUNT) {
                const uint64_t mine = s_key[sl];
                int r = 0;
#pragma unroll 8
                for (int s2 = 0; s2 < C; ++s2)
                    r += s_key[s2] < mine;
                s_victim[r] = sl;
            }
        }
        __syncwarp();
        bool ev_flag[2] = {false, false};
        int n_groups = n_miss ? 1 + (n_miss + C - 1) / C : 1;
        int n_evict_seq = 0;
        if (p.policy == MELINOE_POLICY_COUNT) {
            // The count policy has no closed form (a victim depends on the counts of what the
            // earlier misses of the call brought in): one search per miss, in ascending expert id.
            // Victim: lowest empty slot, else the smallest (count of the occupant, stamp).
            int cur_group = 1, i = 0;
            for (uint64_t m = miss_mask; m; m &= m - 1, ++i) {
                const int e = __ffsll((long long)m) - 1;
                uint64_t khi = ~0ull, klo = ~0ull;
                int slot = -1;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int sl = lane + 32 * h;
                    if (sl < C) {
                        const int occ = s_cache.expert_of_slot[sl];
                        const uint64_t hi = occ < 0 ? 0ull : ((1ull << 32) | (uint64_t)__float_as_uint(s_cache.count[occ]));
                        const uint64_t lo = occ < 0 ? (uint64_t)sl : s_cache.stamp[sl];
                        if (hi < khi || (hi == khi && lo < klo)) {
                            khi = hi;
                            klo = lo;
                            slot = sl;
                        }
                    }
                }
#pragma unroll
                for (int mm = 16; mm >= 1; mm >>= 1) {
                    const uint64_t ohi = __shfl_xor_sync(0xffffffffu, khi, mm);
                    const uint64_t olo = __shfl_xor_sync(0xffffffffu, klo, mm);
                    const int os = __shfl_xor_sync(0xffffffffu, slot, mm);
                    if (ohi < khi || (ohi == khi && olo < klo)) {
                        khi = ohi;
                        klo = olo;
                        slot = os;
                    }
                }
                const int ev = s_cache.expert_of_slot[slot];
                int dep = -1;
                if (ev >= 0) {
                    ++n_evict_seq;
                    if ((need >> ev) & 1ull)
                        dep = s_group_of_expert[ev];
                }
                if (dep == cur_group)
                    ++cur_group;      // it would overwrite an expert of the current wave: next wave
                __syncwarp();
                if (lane == 0) {
                    if (ev >= 0)
                        s_cache.slot_of_expert[ev] = -1;
                    s_cache.expert_of_slot[slot] = e;
                    s_cache.slot_of_expert[e] = slot;
                    s_cache.stamp[slot] = counter + (uint64_t)(n_hits + i) + 1ull;
                    s_req[n_hits + i] = ReqRec{e, slot, 0, ev, 0, cur_group, s_offsets[e], s_counts[e]};
                    s_req_of_expert[e] = n_hits + i;
                    s_group_of_expert[e] = cur_group;
                    s_miss[i] = HostMiss{e, slot, (int16_t)cur_group, (int16_t)dep, 0u};
                }
                __syncwarp();
            }
            n_groups = n_miss ? cur_group + 1 : 1;
            // a miss stays if it still occupies its slot when the call ends; storing it there has to
            // wait for the call's compute if the slot held one of the call's hits at entry
            for (int j = lane; j < n_miss; j += 32) {
                const int e = s_miss[j].expert, slot = s_miss[j].slot, occ = s_entry_occ[slot];
                const bool stays = s_cache.expert_of_slot[slot] == e;
                const bool hazard = stays && occ >= 0 && ((need >> occ) & 1ull);
                s_miss_flags[j] = (stays ? kDecStays : 0) | (hazard ? kDecHazard : 0);
            }
        } else
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int e = h ? e1 : e0;
            if ((miss_mask >> e) & 1ull) {
                const int i = rank_below(miss_mask, e);
                const int slot = s_victim[i % C];
                const int ev = i < C ? s_entry_occ[slot] : s_miss_expert[i - C];
                const int group = 1 + i / C;
                int dep = -1;
                if (i >= C)
                    dep = i / C;
                else if (ev >= 0 && ((need >> ev) & 1ull))
                    dep = 0;
                ev_flag[h] = ev >= 0;
                s_req[n_hits + i] = ReqRec{e, slot, 0, ev, 0, group, s_offsets[e], s_counts[e]};
                s_req_of_expert[e] = n_hits + i;
                s_miss[i] = HostMiss{e, slot, (int16_t)group, (int16_t)dep, 0u};
                // cache update: the last miss that lands in a slot keeps it
                const bool stays = i + C >= n_miss;
                {
                    const int occ = s_entry_occ[slot];
                    const bool hazard = stays && occ >= 0 && ((need >> occ) & 1ull);
                    s_miss_flags[i] = (stays ? kDecStays : 0) | (hazard ? kDecHazard : 0);
                }
                s_cache.slot_of_expert[e] = stays ? slot : -1;
                if (stays) {
                    s_cache.expert_of_slot[slot] = e;
                    s_cache.stamp[slot] = counter + (uint64_t)(n_hits + i) + 1ull;
                }
                if (i < C && ev >= 0)
                    s_cache.slot_of_expert[ev] = -1;
            }
        }
        const int n_evict = p.policy == MELINOE_POLICY_COUNT ? n_evict_seq : __popcll(ballot64(ev_flag[0], ev_flag[1]));
        counter += (uint64_t)n_req;
        __syncwarp();
        if (lane == 0) {
            int n_req_total = n_req;
            for (int s = 0; s < p.n_shared; ++s) {
                s_req[n_req_total] = ReqRec{E + s, -1, 1, -1, 0, 0, s_offsets[E + s], p.T};
                s_req_of_expert[E + s] = n_req_total;
                ++n_req_total;
            }
            // records for the compute kernels, grouped: group 0 = hits then shared experts, then the
            // miss waves in order
            int ndr = 0;
            s_group_vr_begin[0] = 0;
            for (int r = 0; r < n_hits; ++r)
                s_req[r].vr_start = ndr++;
            for (int r = n_req; r < n_req_total; ++r)
                s_req[r].vr_start = ndr++;
            int g = 0;
            for (int r = n_hits; r < n_req; ++r) {
                while (g < s_req[r].group)
                    s_group_vr_begin[++g] = ndr;
                s_req[r].vr_start = ndr++;
            }
            while (g < kMaxGroups)
                s_group_vr_begin[++g] = ndr;
            int status = s_misc[6];
            if (n_groups > (int)p.gmax)
                status = MELINOE_ERR_STATE;
            if (status != MELINOE_OK) {
                // leave nothing for the compute kernels to do
                for (int i = 0; i <= kMaxGroups; ++i)
                    s_group_vr_begin[i] = 0;
                ndr = 0;
            }
            s_cache.counter = counter;
            s_cache.tot_hits += (uint64_t)n_hits;
            s_cache.tot_misses += (uint64_t)n_miss;
            s_cache.tot_evictions += (uint64_t)n_evict;
            s_cache.call_no += 1;
            s_misc[0] = n_req;
            s_misc[1] = n_hits;
            s_misc[2] = n_miss;
            s_misc[3] = n_evict;
            s_misc[4] = n_groups;
            s_misc[5] = ndr;
            s_misc[6] = status;
            s_misc[7] = n_req_total;
        }
    }
    __syncthreads();

    // ---- write the plan, the virtual requests and the cache state back
    const int n_req_total = s_misc[7];
    const bool ok = s_misc[6] == MELINOE_OK;
    DevPlan *plan = p.plan;
    if (tid == 0) {
        plan->n_tokens = p.T;
        plan->n_req = s_misc[0];
        plan->n_hits = s_misc[1];
        plan->n_miss = s_misc[2];
        plan->n_evict = s_misc[3];
        plan->n_groups = s_misc[4];
        plan->n_dreq = s_misc[5];
        plan->status = s_misc[6];
    }
    for (int i = tid; i <= kMaxGroups; i += kPlanThreads)
        plan->group_vr_begin[i] = s_group_vr_begin[i];
    for (int i = tid; i < kMaxReq; i += kPlanThreads) {
        plan->counts[i] = s_counts[i];
        plan->req_of_expert[i] = s_req_of_expert[i];
    }
    for (int i = tid; i <= kMaxReq; i += kPlanThreads)
        plan->offsets[i] = i <= E + p.n_shared ? s_offsets[i] : 0;
    for (int i = tid; i < n_req_total; i += kPlanThreads)
        plan->req[i] = s_req[i];
    if (ok) {
        const int n_hits = s_misc[1];
        for (int r = tid; r < n_req_total; r += kPlanThreads) {
            const ReqRec rec = s_req[r];
            DecReq q;
            q.blob = rec.slot >= 0 ? p.slots + (size_t)rec.slot * p.slot_stride : p.shared_blobs[rec.expert - E];
            q.host = nullptr;
            q.expert = rec.expert;
            q.flags = 0;
            q.group = rec.group;
            q.reserved = 0;
            if (!rec.hit) {
                q.host = p.host_blobs ? p.host_blobs[rec.expert] : nullptr;
                q.flags = kDecMiss | s_miss_flags[r - n_hits];
            }
            plan->dreq[rec.vr_start] = q;
        }
    }
    {
        uint32_t *dst = reinterpret_cast<uint32_t *>(p.cache);
        const uint32_t *src = reinterpret_cast<const uint32_t *>(&s_cache);
        for (int i = tid; i < (int)(sizeof(DevCache) / 4); i += kPlanThreads)
            dst[i] = src[i];
    }

    // ---- (d) miss queue for the host service, (e) statistics
    if (tid == 0) {
        const int n_miss = s_misc[2];
        if (p.stats) {
            melinoe_moe_stats st;
            st.status = s_misc[6];
            st.n_tokens = p.T;
            st.n_distinct = s_misc[0];
            st.hits = s_misc[1];
            st.misses = n_miss;
            st.evictions = s_misc[3];
            st.groups = s_misc[4];
            st.reserved = 0;
            st.bytes_h2d = (uint64_t)n_miss * (uint64_t)p.expert_bytes;
            st.call_no = s_cache.call_no;
            *p.stats = st;
        }
        publish_miss_queue(p.hplan, s_miss, n_miss, s_misc[4], s_misc[6], p.call_seq);
    }
    // the call's request-trace record, if one is being kept
    if (p.trace_rec) {
        const TraceLayout tl = trace_layout(E, p.k, p.trace_max_tokens);
        melinoe_moe_request *rq = reinterpret_cast<melinoe_moe_request *>(p.trace_rec + tl.req_off);
        for (int i = tid; i < s_misc[0]; i += kPlanThreads)
            rq[i] = melinoe_moe_request{s_req[i].expert, s_req[i].slot, s_req[i].hit, s_req[i].evicted};
        const int nt = p.T < p.trace_max_tokens ? p.T : p.trace_max_tokens;
        for (int i = tid; i < nt * p.k; i += kPlanThreads) {
            reinterpret_cast<int32_t *>(p.trace_rec + tl.idx_off)[i] = p.idx[i];
            reinterpret_cast<float *>(p.trace_rec + tl.gate_off)[i] = p.gate ? p.gate[i] : 0.0f;
        }
        if (tid == 0) {
            melinoe_moe_trace_header th;
            th.call_no = s_cache.call_no;
            th.n_tokens = p.T;
            th.n_requests = s_misc[0];
            th.hits = s_misc[1];
            th.misses = s_misc[2];
            th.status = s_misc[6];
            th.reserved = 0;
            *reinterpret_cast<melinoe_moe_trace_header *>(p.trace_rec) = th;
        }
    }
    // the plan is complete: announce it (see DevPlan::ready_seq)
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(&plan->ready_seq), "r"(p.call_seq) : "memory");
    }
}

}  // namespace

cudaError_t launch_plan(cudaStream_t stream, const PlanParams &p)
{
    plan_kernel<<<1, kPlanThreads, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace melinoe
