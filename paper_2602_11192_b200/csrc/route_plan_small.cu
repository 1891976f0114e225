// Router (Eq. 1) and planning fused into one single-block kernel for calls of at most 8 tokens
// (decode): logits, top-k with lowest-index tie-breaking, renormalised gates, token-to-expert
// lists, slot lookup with LRU eviction, compute groups, miss queue and statistics.
//
// At this size every step is latency, not throughput: the router matrix (E x d bf16, a few
// hundred KB) is pulled by one SM with all 32 warps loading at once, and everything after it
// works on at most 64 (token, rank) pairs, so one kernel without any device-wide hand-over
// replaces two launches.  The results are exactly those of the general router and planning
// kernels: the logit sum uses the same fixed order (element j belongs to lane (j mod 256) / 8,
// lanes add their elements in increasing j, xor-butterfly 16, 8, 4, 2, 1, bias last), and the
// cache requests follow the same rules (hits in ascending expert id, then misses in ascending
// id; a miss takes the lowest empty slot, else the least recently stamped one).
#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxT = kTokPerVr;                 // 8 tokens
constexpr int kMaxPairs = kMaxExperts;           // T * k <= 64 is required by the launcher

__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__global__ void __launch_bounds__(kThreads, 1)
route_plan_small_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ w_r,
                        const float *__restrict__ bias, const int32_t *__restrict__ token_seq, int d,
                        int32_t *__restrict__ idx_out, float *__restrict__ gate_out,
                        float *__restrict__ logits_out, PlanParams p)
{
    extern __shared__ __align__(16) unsigned char dyn[];
    uint4 *xs = reinterpret_cast<uint4 *>(dyn);                  // [T][d / 8]
    __shared__ float s_logit[kMaxT][kMaxExperts];
    __shared__ int32_t s_idx[kMaxPairs];
    __shared__ int32_t s_pos[kMaxPairs];                         // sorted position of pair q
    __shared__ int32_t s_pair_at[kMaxPairs];                     // pair at sorted position
    __shared__ int32_t s_counts[kMaxReq];
    __shared__ int32_t s_offsets[kMaxReq + 1];
    __shared__ __align__(16) DevCache s_cache;
    __shared__ int32_t s_group_of_expert[kMaxExperts];
    __shared__ int32_t s_req_of_expert[kMaxReq];
    __shared__ ReqRec s_req[kMaxReq];
    __shared__ HostMiss s_miss[kMaxExperts];
    __shared__ int32_t s_group_vr_begin[kMaxGroups + 1];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int T = p.T, k = p.k, E = p.E, C = p.C;
    const int n_pairs = T * k;
    const int dv = d >> 3;                                       // uint4 per row

    // ---- stage the hidden rows; warp 0 fetches the cache state meanwhile
    for (int i = tid; i < T * dv; i += kThreads)
        xs[i] = reinterpret_cast<const uint4 *>(x)[i];
    if (warp == 1) {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.cache);
        uint4 *dst = reinterpret_cast<uint4 *>(&s_cache);
        for (int i = lane; i < (int)(sizeof(DevCache) / 16); i += 32)
            dst[i] = src[i];
    }
    for (int i = tid; i < 2 * (kMaxGroups + 1); i += kThreads)
        p.sync[i] = 0u;
    __syncthreads();

    // ---- logits: warp w computes experts w and w + 32 for every token.  The weight row pieces
    // of a lane are fetched eight at a time before any arithmetic, so that a row costs one
    // memory latency instead of one per piece.
    const int n_chunks = d >> 8;
    for (int e = warp; e < E; e += kWarps) {
        float acc[kMaxT];
#pragma unroll
        for (int t = 0; t < kMaxT; ++t)
            acc[t] = 0.0f;
        const uint4 *wrow = reinterpret_cast<const uint4 *>(w_r + (size_t)e * d) + lane;
        for (int c0 = 0; c0 < n_chunks; c0 += 8) {
            uint4 wv[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
                wv[i] = c0 + i < n_chunks ? __ldg(wrow + (c0 + i) * 32) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (c0 + i < n_chunks) {
#pragma unroll
                    for (int t = 0; t < kMaxT; ++t) {
                        if (t < T) {
                            const uint4 xv = xs[t * dv + (c0 + i) * 32 + lane];
                            float a = acc[t];
                            a = __fmaf_rn(bf16lo(xv.x), bf16lo(wv[i].x), a);
                            a = __fmaf_rn(bf16hi(xv.x), bf16hi(wv[i].x), a);
                            a = __fmaf_rn(bf16lo(xv.y), bf16lo(wv[i].y), a);
                            a = __fmaf_rn(bf16hi(xv.y), bf16hi(wv[i].y), a);
                            a = __fmaf_rn(bf16lo(xv.z), bf16lo(wv[i].z), a);
                            a = __fmaf_rn(bf16hi(xv.z), bf16hi(wv[i].z), a);
                            a = __fmaf_rn(bf16lo(xv.w), bf16lo(wv[i].w), a);
                            a = __fmaf_rn(bf16hi(xv.w), bf16hi(wv[i].w), a);
                            acc[t] = a;
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int t = 0; t < kMaxT; ++t) {
            if (t < T) {
                float a = acc[t];
#pragma unroll
                for (int m = 16; m >= 1; m >>= 1)
                    a = __fadd_rn(a, __shfl_xor_sync(0xffffffffu, a, m));
                if (lane == 0) {
                    if (bias) {
                        const int q = token_seq ? token_seq[t] : 0;
                        a = __fadd_rn(a, bias[(size_t)q * E + e]);
                    }
                    s_logit[t][e] = a;
                    if (logits_out)
                        logits_out[(size_t)t * E + e] = a;
                }
            }
        }
    }
    __syncthreads();

    // ---- top-k and gates: warp t serves token t.  Lane l holds experts l and l + 32.
    if (warp < T) {
        const int t = warp;
        const float NEG = -__int_as_float(0x7f800000);  // -inf
        const float v0 = lane < E ? s_logit[t][lane] : NEG;
        const float v1 = lane + 32 < E ? s_logit[t][lane + 32] : NEG;
        bool taken0 = !(lane < E), taken1 = !(lane + 32 < E);
        float my_sel = 0.0f, top = 0.0f;
        int my_idx = 0;
        for (int j = 0; j < k; ++j) {
            float bv;
            int bi;
            if (!taken0 && (taken1 || v0 >= v1)) {
                bv = v0;
                bi = lane;
            } else if (!taken1) {
                bv = v1;
                bi = lane + 32;
            } else {
                bv = NEG;
                bi = 1 << 20;
            }
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, m);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, m);
                if (ov > bv || (ov == bv && oi < bi)) {
                    bv = ov;
                    bi = oi;
                }
            }
            if (bi == lane)
                taken0 = true;
            if (bi == lane + 32)
                taken1 = true;
            if (j == 0)
                top = bv;
            if (lane == j) {
                my_sel = bv;
                my_idx = bi;
            }
        }
        const float ev = lane < k ? expf(my_sel - top) : 0.0f;
        float sum = ev;
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1)
            sum += __shfl_xor_sync(0xffffffffu, sum, m);
        if (lane < k) {
            s_idx[t * k + lane] = my_idx;
            idx_out[(size_t)t * k + lane] = my_idx;
            gate_out[(size_t)t * k + lane] = ev / sum;
        }
    }
    __syncthreads();
    if (warp != 0)
        return;

    // ================================================================ planning, by warp 0
    // ---- token lists: counts, offsets, stable positions (pairs in increasing flat index)
    for (int e = lane; e < kMaxReq; e += 32) {
        int c = 0;
        if (e < E)
            for (int q = 0; q < n_pairs; ++q)
                c += s_idx[q] == e;
        else if (e < E + p.n_shared)
            c = T;
        s_counts[e] = c;
        s_req_of_expert[e] = -1;
    }
    __syncwarp();
    if (lane == 0) {
        int run = 0;
        for (int e = 0; e < E + p.n_shared; ++e) {
            s_offsets[e] = run;
            run += s_counts[e];
        }
        s_offsets[E + p.n_shared] = run;
    }
    __syncwarp();
    for (int q = lane; q < n_pairs; q += 32) {
        const int e = s_idx[q];
        int r = 0;
        for (int q2 = 0; q2 < q; ++q2)
            r += s_idx[q2] == e;
        const int pos = s_offsets[e] + r;
        s_pos[q] = pos;
        s_pair_at[pos] = q;
        p.perm[pos] = q;
        p.inv_pos[q] = pos;
        p.tok_of_sorted[pos] = q / k;
    }
    for (int i = lane; i < p.n_shared * T; i += 32)
        p.tok_of_sorted[n_pairs + i] = i % T;
    __syncwarp();

    // ---- cache requests: hits in ascending expert id, then misses in ascending id
    uint64_t need = 0, resident = 0;
    {
        const bool n0 = lane < E && s_counts[lane] > 0;
        const bool n1 = lane + 32 < E && s_counts[lane + 32] > 0;
        const bool r0 = lane < E && s_cache.slot_of_expert[lane] >= 0;
        const bool r1 = lane + 32 < E && s_cache.slot_of_expert[lane + 32] >= 0;
        need = (uint64_t)__ballot_sync(0xffffffffu, n0) | ((uint64_t)__ballot_sync(0xffffffffu, n1) << 32);
        resident = (uint64_t)__ballot_sync(0xffffffffu, r0) | ((uint64_t)__ballot_sync(0xffffffffu, r1) << 32);
    }
    int n_req = 0, n_hits = 0, n_miss = 0, n_evict = 0;
    uint64_t counter = s_cache.counter;
    for (uint64_t m = need & resident; m; m &= m - 1) {
        const int e = __ffsll((long long)m) - 1;
        if (lane == 0) {
            const int s = s_cache.slot_of_expert[e];
            s_cache.stamp[s] = ++counter;
            s_req[n_req] = ReqRec{e, s, 1, -1, s_offsets[e], s_counts[e], 0, 0};
            s_req_of_expert[e] = n_req;
            s_group_of_expert[e] = 0;
        }
        ++n_req;
        ++n_hits;
    }
    counter = __shfl_sync(0xffffffffu, counter, 0);
    __syncwarp();
    int cur_group = 1;
    for (uint64_t m = need & ~resident; m; m &= m - 1) {
        const int e = __ffsll((long long)m) - 1;
        // victim: lowest empty slot, else smallest stamp (stamps are unique)
        uint64_t key = ~0ull;
        int slot = -1;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int s = lane + 32 * h;
            if (s < C) {
                const uint64_t ks = s_cache.expert_of_slot[s] < 0 ? (uint64_t)s : ((1ull << 63) | s_cache.stamp[s]);
                if (ks < key) {
                    key = ks;
                    slot = s;
                }
            }
        }
#pragma unroll
        for (int mm = 16; mm >= 1; mm >>= 1) {
            const uint64_t ok = __shfl_xor_sync(0xffffffffu, key, mm);
            const int os = __shfl_xor_sync(0xffffffffu, slot, mm);
            if (ok < key) {
                key = ok;
                slot = os;
            }
        }
        const int ev = s_cache.expert_of_slot[slot];
        int dep = -1;
        if (ev >= 0) {
            ++n_evict;
            if ((need >> ev) & 1ull)
                dep = s_group_of_expert[ev];
        }
        if (dep == cur_group)
            ++cur_group;
        __syncwarp();
        if (lane == 0) {
            ++counter;
            if (ev >= 0)
                s_cache.slot_of_expert[ev] = -1;
            s_cache.expert_of_slot[slot] = e;
            s_cache.slot_of_expert[e] = slot;
            s_cache.stamp[slot] = counter;
            s_req[n_req] = ReqRec{e, slot, 0, ev, s_offsets[e], s_counts[e], 0, cur_group};
            s_req_of_expert[e] = n_req;
            s_group_of_expert[e] = cur_group;
            s_miss[n_miss] = HostMiss{e, slot, (int16_t)cur_group, (int16_t)dep, 0u};
        }
        counter = __shfl_sync(0xffffffffu, counter, 0);
        ++n_req;
        ++n_miss;
        __syncwarp();
    }
    const int n_groups = n_miss ? cur_group + 1 : 1;
    int n_req_total = n_req;
    int nvr = 0;
    int status = MELINOE_OK;
    if (lane == 0) {
        for (int s = 0; s < p.n_shared; ++s) {
            s_req[n_req_total] = ReqRec{E + s, -1, 1, -1, s_offsets[E + s], T, 0, 0};
            s_req_of_expert[E + s] = n_req_total;
            ++n_req_total;
        }
        // virtual requests (one per request here: at most 8 tokens), grouped: group 0 = hits then
        // shared, then the miss waves in order
        s_group_vr_begin[0] = 0;
        for (int r = 0; r < n_hits; ++r)
            s_req[r].vr_start = nvr++;
        for (int r = n_req; r < n_req_total; ++r)
            s_req[r].vr_start = nvr++;
        int g = 0;
        for (int r = n_hits; r < n_req; ++r) {
            while (g < s_req[r].group)
                s_group_vr_begin[++g] = nvr;
            s_req[r].vr_start = nvr++;
        }
        while (g < kMaxGroups)
            s_group_vr_begin[++g] = nvr;
        if (nvr > p.vr_capacity || n_groups > (int)p.gmax)
            status = MELINOE_ERR_STATE;
        if (status != MELINOE_OK) {
            for (int i = 0; i <= kMaxGroups; ++i)
                s_group_vr_begin[i] = 0;
            nvr = 0;
        }
        s_cache.counter = counter;
        s_cache.tot_hits += (uint64_t)n_hits;
        s_cache.tot_misses += (uint64_t)n_miss;
        s_cache.tot_evictions += (uint64_t)n_evict;
        s_cache.call_no += 1;
        s_cache.tot_vr += (uint64_t)nvr;
    }
    n_req_total = __shfl_sync(0xffffffffu, n_req_total, 0);
    nvr = __shfl_sync(0xffffffffu, nvr, 0);
    status = __shfl_sync(0xffffffffu, status, 0);
    __syncwarp();

    // ---- write the plan, the virtual requests and the cache state back
    DevPlan *plan = p.plan;
    if (lane == 0) {
        plan->n_tokens = T;
        plan->n_req = n_req;
        plan->n_hits = n_hits;
        plan->n_miss = n_miss;
        plan->n_evict = n_evict;
        plan->n_groups = n_groups;
        plan->n_vr = nvr;
        plan->status = status;
    }
    for (int i = lane; i <= kMaxGroups; i += 32)
        plan->group_vr_begin[i] = s_group_vr_begin[i];
    for (int i = lane; i < kMaxReq; i += 32) {
        plan->counts[i] = s_counts[i];
        plan->req_of_expert[i] = s_req_of_expert[i];
    }
    for (int i = lane; i <= kMaxReq; i += 32)
        plan->offsets[i] = i <= E + p.n_shared ? s_offsets[i] : 0;
    for (int r = lane; r < n_req_total; r += 32) {
        const ReqRec rec = s_req[r];
        plan->req[r] = rec;
        if (status == MELINOE_OK) {
            VrRec vr;
            vr.blob = rec.slot >= 0 ? p.slots + (size_t)rec.slot * p.slot_stride : p.shared_blobs[rec.expert - E];
            vr.n_tok = rec.n_tok;
            vr.group = rec.group;
            for (int i = 0; i < kTokPerVr; ++i) {
                const int pos = rec.tok_off + i;
                const bool on = i < rec.n_tok;
                const bool routed = pos < n_pairs;
                vr.tok[i] = on ? (routed ? s_pair_at[pos] / k : (pos - n_pairs) % T) : -1;
                vr.pair[i] = on ? (routed ? s_pair_at[pos] : pos) : -1;
            }
            p.vrs[rec.vr_start] = vr;
        }
    }
    {
        uint4 *dst = reinterpret_cast<uint4 *>(p.cache);
        const uint4 *src = reinterpret_cast<const uint4 *>(&s_cache);
        for (int i = lane; i < (int)(sizeof(DevCache) / 16); i += 32)
            dst[i] = src[i];
    }

    // ---- statistics and the miss queue for the host
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
            st.call_no = s_cache.call_no;
            *p.stats = st;
        }
        publish_miss_queue(p.hplan, s_miss, n_miss, n_groups, status, p.call_seq);
    }
}

}  // namespace

bool route_plan_small_supported(int T, int k, int d)
{
    return T >= 1 && T <= kMaxT && T * k <= kMaxPairs && (size_t)T * d * 2 <= 160 * 1024;
}

cudaError_t launch_route_plan_small(cudaStream_t stream, const uint16_t *x, const uint16_t *w_r, const float *bias,
                                    const int32_t *token_seq, int d, int32_t *idx, float *gate, float *logits_out,
                                    const PlanParams &p)
{
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(route_plan_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             160 * 1024);
        if (e != cudaSuccess)
            return e;
        attr_set = true;
    }
    const size_t smem = (size_t)p.T * d * 2;
    route_plan_small_kernel<<<1, kThreads, smem, stream>>>(x, w_r, bias, token_seq, d, idx, gate, logits_out, p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace melinoe
