// Router (Eq. 1) and planning fused into one kernel for calls of at most 8 tokens (decode):
// logits, top-k with lowest-index tie-breaking, renormalised gates, token-to-expert lists, slot
// lookup with LRU eviction, compute groups, miss queue and statistics.
//
// At this size every step is latency, not throughput, so the kernel is organised to take as
// few dependent memory round trips as possible:
//   - logits: one warp per expert, spread over a thread-block cluster of 8 CTAs x 8 warps (a single
//     SM pulling the whole router matrix takes ~9 us; eight take ~2); each lane has all its loads in
//     flight at once, the router row already before the kernel ahead in the stream has finished;
//   - the logits go straight into the shared memory of the cluster's first CTA and the cluster
//     barrier tells it when they are all there: no fence, no device counter, no second launch;
//   - top-k is a rank count (an element's rank is the number of elements that beat it) shared by
//     the eight warps, instead of k rounds of a warp-wide maximum; the gates are computed by the
//     other warps while the first one plans;
//   - planning is written for one warp with lane = expert / slot / request: ranks come from
//     ballots and population counts, prefix sums from shuffles, and the LRU victims of a call are
//     taken from one sorted list instead of one search per miss.
//
// The results are exactly those of the general router and planning kernels.  The logit sum uses
// the same fixed order (element j belongs to lane (j mod 256) / 8, lanes add their elements in
// increasing j, xor-butterfly 16, 8, 4, 2, 1, bias last).  The cache requests follow the same
// rules (hits in ascending expert id, then misses in ascending id; a miss takes the lowest empty
// slot, else the least recently stamped one), restated in closed form:
//   - hit number r (ascending id) stamps its slot with counter + r + 1;
//   - let V be the slots ordered by (empty first, by index), then by stamp after the hits were
//     stamped.  Miss number i (ascending id) takes V[i mod C], because every slot it could prefer
//     has either been taken by an earlier miss (and stamped newer) or comes later in V;
//   - the expert it displaces is V[i]'s occupant at call entry for i < C, and miss i - C otherwise;
//   - miss i belongs to compute group 1 + i / C: a new wave starts exactly when a miss would
//     overwrite an expert of the current wave, which is every C misses; it must wait for group
//     i / C (i >= C), for group 0 if it displaces one of the call's hits, for nothing otherwise.
#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;
constexpr int kCluster = kMaxExperts / kWarpsPerBlock;   // 8 CTAs: a warp for each of up to 64 experts
constexpr int kMaxT = kTokPerVr;                 // 8 tokens
constexpr int kMaxPairs = kMaxExperts;           // T * k <= 64 is required by the launcher

__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ int warp_excl_scan(int v, int lane, int &total)
{
    int inc = v;
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, inc, m);
        if (lane >= m)
            inc += o;
    }
    total = __shfl_sync(0xffffffffu, inc, 31);
    return inc - v;
}

__device__ __forceinline__ uint64_t ballot64(bool lo, bool hi)
{
    return (uint64_t)__ballot_sync(0xffffffffu, lo) | ((uint64_t)__ballot_sync(0xffffffffu, hi) << 32);
}

__device__ __forceinline__ int rank_below(uint64_t mask, int bit) { return __popcll(mask & ((1ull << bit) - 1ull)); }

// The cache half of a request record (the gather warp writes tok_off / n_tok, the other two words).
__device__ __forceinline__ void write_req(ReqRec *r, int expert, int slot, int hit, int evicted, int at, int group,
                                          char *trace_req = nullptr)
{
    *reinterpret_cast<int4 *>(&r->expert) = make_int4(expert, slot, hit, evicted);
    *reinterpret_cast<int2 *>(&r->vr_start) = make_int2(at, group);
    if (trace_req)      // the same four words into the call's request-trace record
        *reinterpret_cast<int4 *>(trace_req) = make_int4(expert, slot, hit, evicted);
}

__global__ void __launch_bounds__(kThreads, 1)
route_plan_small_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ w_r,
                        const float *__restrict__ bias, const int32_t *__restrict__ token_seq, int d,
                        int32_t *__restrict__ idx_out, float *__restrict__ gate_out, float *logits_out,
                        PlanParams p)
{
    __shared__ __align__(16) float s_logit[kMaxT][kMaxExperts];
    __shared__ int32_t s_cnt[2][kMaxExperts];                    // pairs of an expert among pairs 0..31 / 32..63
    __shared__ int32_t s_tok[kMaxPairs];                         // token of a pair
    __shared__ int32_t s_rank[kMaxT][kMaxExperts];               // rank of an expert among a token's logits
    // count policy only: live slot table during the call's misses, counts, groups
    __shared__ int32_t s_live_occ[kMaxExperts];
    __shared__ unsigned long long s_live_stamp[kMaxExperts];
    __shared__ float s_cntf[kMaxExperts];
    __shared__ int32_t s_grp_of[kMaxExperts];
    __shared__ int32_t s_grp_first[kMaxGroups + 1];              // first miss of a wave
    __shared__ int32_t s_idx[kMaxPairs];
    __shared__ unsigned long long s_key[kMaxExperts];            // victim-order key of a slot
    __shared__ int32_t s_victim[kMaxExperts];                    // V: slots in victim order
    __shared__ int32_t s_miss_expert[kMaxExperts];               // expert of miss number i
    __shared__ int32_t s_needflags[2][kMaxExperts];              // per planning warp: 1 = some pair of the call names this expert
    __shared__ HostMiss s_hm[kMaxExperts];                       // the call's miss queue, sent to the host last
    __shared__ int32_t s_miss_slot[kMaxExperts];                 // count policy: its slot and wave
    __shared__ int32_t s_miss_group[kMaxExperts];
    __shared__ int32_t s_entry_occ[kMaxExperts];                 // occupant of a slot at call entry
    __shared__ float s_sel[kMaxT][kMaxExperts];                  // a token's selected logits, by rank

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int T = p.T, k = p.k, E = p.E, C = p.C;
    const int n_pairs = T * k;
    unsigned cta_rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(cta_rank));

    // ================================================================ logits: one warp per expert
    const int e_mine = (int)cta_rank * kWarpsPerBlock + warp;
    const int n_chunks = d >> 8;
    // The router matrix does not change while calls are queued, so the first eight pieces of the
    // row go out before anything else.
    uint4 wv0[8];
    if (e_mine < E) {
        const uint4 *wrow = reinterpret_cast<const uint4 *>(w_r + (size_t)e_mine * d) + lane;
#pragma unroll
        for (int i = 0; i < 8; ++i)
            wv0[i] = i < n_chunks ? __ldg(wrow + i * 32) : make_uint4(0, 0, 0, 0);
    }
    // The launch may have been made with programmatic stream serialisation: this block can then be
    // running before the kernel ahead of it in the stream has finished.  Nothing before this point
    // reads what that kernel may have written; wait for it here (returns at once in an ordinary
    // launch).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // lane t holds token t's bias (two dependent loads, in flight under the dot products)
    float my_bias = 0.0f;
    if (e_mine < E && bias && lane < T) {
        const int q = token_seq ? token_seq[lane] : 0;
        my_bias = bias[(size_t)q * E + e_mine];
    }

    // the planner's view of the cache: its loads overlap the logits
    DevCache *cache = p.cache;
    int soe0 = -1, soe1 = -1, eos0 = -1, eos1 = -1;
    unsigned long long st0 = 0ull, st1 = 0ull, counter = 0ull, call_no = 0ull;
    float cnt0 = 0.0f, cnt1 = 0.0f;
    const bool by_count = p.policy == MELINOE_POLICY_COUNT;
    if (cta_rank == 0 && warp == 1) {
        // the gather warp only needs to know which experts are resident
        if (lane < E)
            soe0 = cache->slot_of_expert[lane];
        if (lane + 32 < E)
            soe1 = cache->slot_of_expert[lane + 32];
    }
    if (cta_rank == 0 && warp == 0) {
        if (by_count) {
            if (lane < E)
                cnt0 = cache->count[lane];
            if (lane + 32 < E)
                cnt1 = cache->count[lane + 32];
        }
        if (lane < E)
            soe0 = cache->slot_of_expert[lane];
        if (lane + 32 < E)
            soe1 = cache->slot_of_expert[lane + 32];
        if (lane < C) {
            eos0 = cache->expert_of_slot[lane];
            st0 = cache->stamp[lane];
        }
        if (lane + 32 < C) {
            eos1 = cache->expert_of_slot[lane + 32];
            st1 = cache->stamp[lane + 32];
        }
        counter = cache->counter;
        call_no = cache->call_no + 1ull;
    }
    if (e_mine < E) {
        const uint4 *wrow = reinterpret_cast<const uint4 *>(w_r + (size_t)e_mine * d) + lane;
        float my_logit = 0.0f;
        for (int t = 0; t < T; ++t) {
            const uint4 *xrow = reinterpret_cast<const uint4 *>(x + (size_t)t * d) + lane;
            float a = 0.0f;
            for (int c0 = 0; c0 < n_chunks; c0 += 8) {
                // all of a lane's loads for these 8 pieces go out before any arithmetic
                uint4 wv[8], xv[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const bool on = c0 + i < n_chunks;
                    xv[i] = on ? __ldcg(xrow + (c0 + i) * 32) : make_uint4(0, 0, 0, 0);
                }
                if (c0 == 0) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        wv[i] = wv0[i];
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        wv[i] = c0 + i < n_chunks ? __ldg(wrow + (c0 + i) * 32) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (c0 + i < n_chunks) {
                        a = __fmaf_rn(bf16lo(xv[i].x), bf16lo(wv[i].x), a);
                        a = __fmaf_rn(bf16hi(xv[i].x), bf16hi(wv[i].x), a);
                        a = __fmaf_rn(bf16lo(xv[i].y), bf16lo(wv[i].y), a);
                        a = __fmaf_rn(bf16hi(xv[i].y), bf16hi(wv[i].y), a);
                        a = __fmaf_rn(bf16lo(xv[i].z), bf16lo(wv[i].z), a);
                        a = __fmaf_rn(bf16hi(xv[i].z), bf16hi(wv[i].z), a);
                        a = __fmaf_rn(bf16lo(xv[i].w), bf16lo(wv[i].w), a);
                        a = __fmaf_rn(bf16hi(xv[i].w), bf16hi(wv[i].w), a);
                    }
                }
            }
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1)
                a = __fadd_rn(a, __shfl_xor_sync(0xffffffffu, a, m));
            if (lane == t)
                my_logit = bias ? __fadd_rn(a, my_bias) : a;
        }
        if (lane < T) {
            // into the first CTA's shared memory, and to global memory for the inspection calls
            uint32_t remote;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
                         : "=r"(remote)
                         : "r"((uint32_t)__cvta_generic_to_shared(&s_logit[lane][e_mine])), "r"(0));
            asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(my_logit) : "memory");
            logits_out[(size_t)lane * E + e_mine] = my_logit;
        }
    }
    // ---- the cluster's first CTA carries on when every logit has arrived
    if (cta_rank == 0)
        for (int i = tid; i < kMaxT * kMaxExperts; i += kThreads)
            (&s_rank[0][0])[i] = 0;
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    if (cta_rank != 0)
        return;
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");

    // ================================================================ top-k
    // An element's rank is the number of elements that beat it (greater, or equal with a lower
    // index).  The eight warps share the count (warp w compares against elements 8w .. 8w + 7 of
    // every token) and add their parts up in shared memory; then warp t writes token t's selection.
    // Only the indices are on the way to the planner: the gates are left to the other warps.
    {
        const float NEG = -__int_as_float(0x7f800000);  // -inf
        for (int t = 0; t < T; ++t) {
            const float v0 = lane < E ? s_logit[t][lane] : NEG;
            const float v1 = lane + 32 < E ? s_logit[t][lane + 32] : NEG;
            int r0 = 0, r1 = 0;
            const float4 *row = reinterpret_cast<const float4 *>(s_logit[t]) + 2 * warp;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const float4 o4 = row[i];
                const float ov[4] = {o4.x, o4.y, o4.z, o4.w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int e = 8 * warp + 4 * i + c;
                    const float o = e < E ? ov[c] : NEG;     // the row's tail beyond E was never written
                    r0 += (o > v0) || (o == v0 && e < lane);
                    r1 += (o > v1) || (o == v1 && e < lane + 32);
                }
            }
            if (r0)
                atomicAdd(&s_rank[t][lane], r0);
            if (r1)
                atomicAdd(&s_rank[t][lane + 32], r1);
        }
        __syncthreads();
        if (warp < T) {
            const int t = warp;
            const int r0 = s_rank[t][lane], r1 = s_rank[t][lane + 32];
            if (lane < E && r0 < k) {
                s_sel[t][r0] = s_logit[t][lane];
                s_idx[t * k + r0] = lane;
            }
            if (lane + 32 < E && r1 < k) {
                s_sel[t][r1] = s_logit[t][lane + 32];
                s_idx[t * k + r1] = lane + 32;
            }
        }
        __syncthreads();
    }
    if (warp >= 2) {
        // ============================================================ gates (Eq. 1), off the planner's path
        for (int t = warp - 2; t < T; t += kWarpsPerBlock - 2) {
            const float top = s_sel[t][0];
            const float ev = lane < k ? expf(s_sel[t][lane] - top) : 0.0f;
            float sum = ev;
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1)
                sum += __shfl_xor_sync(0xffffffffu, sum, m);
            if (lane < k) {
                idx_out[(size_t)t * k + lane] = s_idx[t * k + lane];
                gate_out[(size_t)t * k + lane] = ev / sum;
                if (p.trace_rec && t < p.trace_max_tokens) {
                    const TraceLayout tl = trace_layout(E, k, p.trace_max_tokens);
                    reinterpret_cast<int32_t *>(p.trace_rec + tl.idx_off)[t * k + lane] = s_idx[t * k + lane];
                    reinterpret_cast<float *>(p.trace_rec + tl.gate_off)[t * k + lane] = ev / sum;
                }
            }
        }
        // these warps' results are written before the planning warp announces the plan
        asm volatile("bar.arrive 2, %0;" ::"n"(kThreads) : "memory");
        return;
    }

    // ================================================================ planning, by two warps side by side
    // Warp 1 builds the token lists (what the gather and the inspection calls need), warp 0 the cache
    // requests (what the compute kernel waits for).  Both know which experts are needed and which of
    // those are resident, so both can tell a request's place in the call's request order.
    // lane owns experts lane and lane + 32, slots lane and lane + 32, pairs lane and lane + 32
    // (the cache state of this lane's experts and slots was loaded before the logits)
    DevPlan *plan = p.plan;
    const int e0 = lane, e1 = lane + 32;
    // which experts the call's pairs name
    int32_t *s_needflag = s_needflags[warp];
    s_needflag[lane] = 0;
    s_needflag[lane + 32] = 0;
    __syncwarp();
    if (lane < n_pairs)
        s_needflag[s_idx[lane]] = 1;
    if (lane + 32 < n_pairs)
        s_needflag[s_idx[lane + 32]] = 1;
    __syncwarp();
    const uint64_t need = ballot64(s_needflag[lane] != 0, s_needflag[lane + 32] != 0);
    const uint64_t resident = ballot64(soe0 >= 0, soe1 >= 0);
    const uint64_t hit_mask = need & resident, miss_mask = need & ~resident;
    const int n_hits = __popcll(hit_mask), n_miss = __popcll(miss_mask), n_req = n_hits + n_miss;

    if (warp == 1) {
        // ---- token lists: counts, offsets, stable positions (pairs in increasing flat index)
        // Lane q also stands for pairs q and q + 32: the lanes whose pair names the same expert find
        // one another with a match, so an expert's count and a pair's place among its expert's pairs
        // are population counts.
        const int qe[2] = {lane < n_pairs ? s_idx[lane] : -1 - lane, lane + 32 < n_pairs ? s_idx[lane + 32] : -1 - lane};
        const unsigned lt = (1u << lane) - 1u;
        const unsigned same[2] = {__match_any_sync(0xffffffffu, qe[0]), __match_any_sync(0xffffffffu, qe[1])};
        s_cnt[0][lane] = s_cnt[0][lane + 32] = s_cnt[1][lane] = s_cnt[1][lane + 32] = 0;
        s_tok[lane] = lane / k;
        s_tok[lane + 32] = (lane + 32) / k;
        __syncwarp();
#pragma unroll
        for (int h = 0; h < 2; ++h)
            if (qe[h] >= 0 && (same[h] & lt) == 0u)
                s_cnt[h][qe[h]] = __popc(same[h]);
        __syncwarp();
        const int c0 = s_cnt[0][e0] + s_cnt[1][e0], c1 = s_cnt[0][e1] + s_cnt[1][e1];
        int tot0, tot1;
        const int off0 = warp_excl_scan(c0, lane, tot0);
        const int off1 = tot0 + warp_excl_scan(c1, lane, tot1);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int q = lane + 32 * h;
            const int e = qe[h] >= 0 ? qe[h] : 0;
            const int r = __popc(same[h] & lt) + (h ? s_cnt[0][e] : 0);
            const int o0 = __shfl_sync(0xffffffffu, off0, e & 31), o1 = __shfl_sync(0xffffffffu, off1, e & 31);
            if (q < n_pairs) {
                const int pos = (e < 32 ? o0 : o1) + r;
                p.perm[pos] = q;
                p.inv_pos[q] = pos;
                p.tok_of_sorted[pos] = s_tok[q];
            }
        }
        for (int i = lane; i < p.n_shared * T; i += 32)
            p.tok_of_sorted[n_pairs + i] = i % T;
        // every request's token list: its record's place follows from the masks (hits in ascending
        // id, then the misses in ascending id, then the shared experts)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int e = h ? e1 : e0, cnt = h ? c1 : c0, off = h ? off1 : off0;
            if ((need >> e) & 1ull) {
                const int r = ((hit_mask >> e) & 1ull) ? rank_below(hit_mask, e) : n_hits + rank_below(miss_mask, e);
                *reinterpret_cast<int2 *>(&plan->req[r].tok_off) = make_int2(off, cnt);
            }
        }
        for (int sh = lane; sh < p.n_shared; sh += 32)
            *reinterpret_cast<int2 *>(&plan->req[n_req + sh].tok_off) = make_int2(n_pairs + sh * T, T);
        if (e0 < E) {
            plan->counts[e0] = c0;
            plan->offsets[e0] = off0;
        }
        if (e1 < E) {
            plan->counts[e1] = c1;
            plan->offsets[e1] = off1;
        }
        if (lane <= p.n_shared) {
            if (lane < p.n_shared)
                plan->counts[E + lane] = T;
            plan->offsets[E + lane] = n_pairs + lane * T;
        }
        asm volatile("bar.arrive 2, %0;" ::"n"(kThreads) : "memory");
        return;
    }

    // ---- the cache requests (warp 0)
    char *tr_req = p.trace_rec ? p.trace_rec + trace_layout(E, k, p.trace_max_tokens).req_off : nullptr;
    const bool req0 = (need >> e0) & 1ull, req1 = (need >> e1) & 1ull;
    // compute groups: closed form under LRU; under the count policy known only after the misses
    // have been walked, one wave per miss at most
    int n_groups = n_miss ? 1 + (by_count ? n_miss : (n_miss + C - 1) / C) : 1;
    const int ndr = n_req + p.n_shared;             // records for the compute kernels: hits, shared experts, misses
    const int status = n_groups > (int)p.gmax ? MELINOE_ERR_STATE : MELINOE_OK;
    const bool ok = status == MELINOE_OK;
    if (by_count) {
        // Definition C.1: one time step per call, count <- gamma * count + request
        const float n0 = __fadd_rn(__fmul_rn(p.gamma, cnt0), req0 ? 1.0f : 0.0f);
        const float n1 = __fadd_rn(__fmul_rn(p.gamma, cnt1), req1 ? 1.0f : 0.0f);
        s_cntf[lane] = n0;
        s_cntf[lane + 32] = n1;
        if (e0 < E)
            cache->count[e0] = n0;
        if (e1 < E)
            cache->count[e1] = n1;
    }

    // victim-order key of every slot: empty slots by index, then occupied ones by stamp, with the
    // stamps this call's hits receive
    s_key[lane] = lane < C ? (eos0 < 0 ? (unsigned long long)lane : ((1ull << 63) | st0)) : ~0ull;
    s_key[lane + 32] = lane + 32 < C ? (eos1 < 0 ? (unsigned long long)(lane + 32) : ((1ull << 63) | st1)) : ~0ull;
    s_entry_occ[lane] = eos0;
    s_entry_occ[lane + 32] = eos1;
    __syncwarp();
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int e = h ? e1 : e0, soe = h ? soe1 : soe0;
        if ((hit_mask >> e) & 1ull) {
            const int r = rank_below(hit_mask, e);
            const unsigned long long st = counter + (unsigned long long)r + 1ull;
            s_key[soe] = (1ull << 63) | st;
            cache->stamp[soe] = st;
            write_req(&plan->req[r], e, soe, 1, -1, r, 0, tr_req ? tr_req + 16 * r : nullptr);
            s_grp_of[e] = 0;
            plan->dreq[r] = DecReq{p.slots + (size_t)soe * p.slot_stride, nullptr, e, 0, 0, 0};
        }
        if ((miss_mask >> e) & 1ull)
            s_miss_expert[rank_below(miss_mask, e)] = e;
    }
    __syncwarp();
    // V: rank of each slot among the keys (keys are distinct); only misses take victims
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int s = lane + 32 * h;
        if (s < C && n_miss > 0 && !by_count) {
            const unsigned long long mine = s_key[s];
            int r = 0;
#pragma unroll 8
            for (int s2 = 0; s2 < C; ++s2)
                r += s_key[s2] < mine;
            s_victim[r] = s;
        }
    }
    __syncwarp();
    bool ev_flag[2] = {false, false};
    int n_evict_seq = 0;
    if (by_count) {
        // The count policy has no closed form (a victim depends on the counts of what the earlier
        // misses of the call brought in): one search per miss, in ascending expert id, over a live
        // copy of the slot table.  Victim: lowest empty slot, else the smallest (count of the
        // occupant, stamp).  A new wave starts when a miss would overwrite an expert of the
        // current wave.
        s_live_occ[lane] = eos0;
        s_live_occ[lane + 32] = eos1;
        s_live_stamp[lane] = s_key[lane] & ~(1ull << 63);
        s_live_stamp[lane + 32] = s_key[lane + 32] & ~(1ull << 63);
        if (lane == 0)
            s_grp_first[1] = 0;
        __syncwarp();
        int cur_group = 1, i = 0;
        for (uint64_t m = miss_mask; m; m &= m - 1, ++i) {
            const int e = __ffsll((long long)m) - 1;
            unsigned long long khi = ~0ull, klo = ~0ull;
            int slot = -1;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int sl = lane + 32 * h;
                if (sl < C) {
                    const int occ = s_live_occ[sl];
                    const unsigned long long hi = occ < 0 ? 0ull : ((1ull << 32) | (unsigned long long)__float_as_uint(s_cntf[occ]));
                    const unsigned long long lo = occ < 0 ? (unsigned long long)sl : s_live_stamp[sl];
                    if (hi < khi || (hi == khi && lo < klo)) {
                        khi = hi;
                        klo = lo;
                        slot = sl;
                    }
                }
            }
#pragma unroll
            for (int mm = 16; mm >= 1; mm >>= 1) {
                const unsigned long long ohi = __shfl_xor_sync(0xffffffffu, khi, mm);
                const unsigned long long olo = __shfl_xor_sync(0xffffffffu, klo, mm);
                const int os = __shfl_xor_sync(0xffffffffu, slot, mm);
                if (ohi < khi || (ohi == khi && olo < klo)) {
                    khi = ohi;
                    klo = olo;
                    slot = os;
                }
            }
            const int ev = s_live_occ[slot];
            int dep = -1;
            if (ev >= 0) {
                ++n_evict_seq;
                if ((need >> ev) & 1ull)
                    dep = s_grp_of[ev];
            }
            if (dep == cur_group) {
                ++cur_group;
                if (lane == 0)
                    s_grp_first[cur_group] = i;
            }
            __syncwarp();
            if (lane == 0) {
                const unsigned long long st = counter + (unsigned long long)(n_hits + i) + 1ull;
                const int vr_at = n_hits + p.n_shared + i;
                if (ev >= 0)
                    cache->slot_of_expert[ev] = -1;
                cache->expert_of_slot[slot] = e;
                cache->slot_of_expert[e] = slot;
                cache->stamp[slot] = st;
                s_live_occ[slot] = e;
                s_live_stamp[slot] = st;
                s_grp_of[e] = cur_group;
                write_req(&plan->req[n_hits + i], e, slot, 0, ev, vr_at, cur_group, tr_req ? tr_req + 16 * (n_hits + i) : nullptr);
                s_miss_expert[i] = e;
                s_miss_slot[i] = slot;
                s_miss_group[i] = cur_group;
                s_hm[i] = HostMiss{e, slot, (int16_t)cur_group, (int16_t)dep, p.call_seq};
            }
            __syncwarp();
        }
        n_groups = n_miss ? cur_group + 1 : 1;
        // a miss stays if it still occupies its slot when the call ends; writing it there must wait
        // for the end of the call's compute if the slot held one of the call's hits at entry
        for (int j = lane; j < n_miss; j += 32) {
            const int e = s_miss_expert[j], slot = s_miss_slot[j], occ = s_entry_occ[slot];
            const bool stays = s_live_occ[slot] == e;
            const bool hazard = stays && occ >= 0 && ((need >> occ) & 1ull);
            plan->dreq[n_hits + p.n_shared + j] =
                DecReq{p.slots + (size_t)slot * p.slot_stride, p.host_blobs ? p.host_blobs[e] : nullptr, e,
                       kDecMiss | (stays ? kDecStays : 0) | (hazard ? kDecHazard : 0), s_miss_group[j], 0};
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
            const int vr_at = n_hits + p.n_shared + i;
            write_req(&plan->req[n_hits + i], e, slot, 0, ev, vr_at, group, tr_req ? tr_req + 16 * (n_hits + i) : nullptr);
            // cache update: the last miss that lands in a slot keeps it
            const bool stays = i + C >= n_miss;
            {
                const int occ = s_entry_occ[slot];
                const bool hazard = stays && occ >= 0 && ((need >> occ) & 1ull);
                plan->dreq[vr_at] = DecReq{p.slots + (size_t)slot * p.slot_stride, p.host_blobs ? p.host_blobs[e] : nullptr, e,
                                           kDecMiss | (stays ? kDecStays : 0) | (hazard ? kDecHazard : 0), group, 0};
            }
            cache->slot_of_expert[e] = stays ? slot : -1;
            if (stays) {
                cache->expert_of_slot[slot] = e;
                cache->stamp[slot] = counter + (unsigned long long)(n_hits + i) + 1ull;
            }
            if (i < C && ev >= 0)
                cache->slot_of_expert[ev] = -1;
            s_hm[i] = HostMiss{e, slot, (int16_t)group, (int16_t)dep, p.call_seq};
        }
    }
    const int n_evict = by_count ? n_evict_seq : __popcll(ballot64(ev_flag[0], ev_flag[1]));
    // shared experts: always resident, group 0, behind the hits
    for (int s = lane; s < p.n_shared; s += 32) {
        write_req(&plan->req[n_req + s], E + s, -1, 1, -1, n_hits + s, 0);
        plan->dreq[n_hits + s] = DecReq{p.shared_blobs[s], nullptr, E + s, 0, 0, 0};
    }
    // group boundaries, counts and offsets (what the FFN launches and the inspection calls read)
    for (int g = lane; g <= kMaxGroups; g += 32) {
        int b = 0;
        if (ok && g >= 1) {
            // misses served before wave g: (g - 1) * C under LRU, the wave's recorded first miss otherwise
            const int done = by_count ? (g < n_groups ? s_grp_first[g] : n_miss) : (g - 1) * C;
            b = n_hits + p.n_shared + (done < n_miss ? done : n_miss);
        }
        plan->group_vr_begin[g] = b;
    }
    if (lane == 0) {
        plan->n_tokens = T;
        plan->n_req = n_req;
        plan->n_hits = n_hits;
        plan->n_miss = n_miss;
        plan->n_evict = n_evict;
        plan->n_groups = n_groups;
        plan->n_dreq = ok ? ndr : 0;
        plan->status = status;
        cache->counter = counter + (unsigned long long)n_req;
        cache->tot_hits += (unsigned long long)n_hits;
        cache->tot_misses += (unsigned long long)n_miss;
        cache->tot_evictions += (unsigned long long)n_evict;
        cache->call_no = call_no;
    }
    // The plan is complete: announce it.  The decode FFN kernel behind this one in the stream may
    // already be running (programmatic launch) and waits for this word, not for this grid to drain.
    // (The barrier orders the other warps' and lanes' writes before lane 0's release, which is cumulative:
    // whoever acquires the word sees them all.)
    asm volatile("bar.sync 2, %0;" ::"n"(kThreads) : "memory");
    if (lane == 0)
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(&plan->ready_seq), "r"(p.call_seq) : "memory");
    // What may live in host memory goes out last, so that no fence above has to wait for the host link:
    // the statistics, and the miss queue for calls whose transfers the host issues.
    for (int i = lane; i < n_miss; i += 32)
        store16_host(&p.hplan->miss[i], &s_hm[i]);
    __syncwarp();
    if (lane == 0) {
        if (p.stats) {
            melinoe_moe_stats st;
            st.status = status;
            st.n_tokens = T;
            st.n_distinct = n_req;
            st.hits = n_hits;
            st.misses = n_miss;
            st.evictions = n_evict;
            st.groups = n_groups;
            st.reserved = 0;
            st.bytes_h2d = (uint64_t)n_miss * (uint64_t)p.expert_bytes;
            st.call_no = call_no;
            *p.stats = st;
        }
        const HostPlanHeader hdr{n_miss, n_groups, status, p.call_seq};
        store16_host(&p.hplan->hdr, &hdr);
        if (p.trace_rec) {
            melinoe_moe_trace_header th;
            th.call_no = call_no;
            th.n_tokens = T;
            th.n_requests = n_req;
            th.hits = n_hits;
            th.misses = n_miss;
            th.status = status;
            th.reserved = 0;
            *reinterpret_cast<melinoe_moe_trace_header *>(p.trace_rec) = th;
        }
    }
}

}  // namespace

bool route_plan_small_supported(int T, int k, int d)
{
    (void)d;
    return T >= 1 && T <= kMaxT && T * k <= kMaxPairs;
}

cudaError_t launch_route_plan_small(cudaStream_t stream, const uint16_t *x, const uint16_t *w_r, const float *bias,
                                    const int32_t *token_seq, int d, int32_t *idx, float *gate, float *logits_out,
                                    const PlanParams &p)
{
    // one cluster of 8 CTAs; programmatic stream serialisation: the blocks may be scheduled while the
    // kernel ahead in the stream is still draining; the kernel itself waits for that kernel before it
    // reads anything that kernel may have written
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kCluster);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, route_plan_small_kernel, x, w_r, bias, token_seq, d, idx, gate, logits_out, p);
    count_launch();
    return e;
}

}  // namespace melinoe
