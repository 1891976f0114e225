// Filling the cache ahead of the first token (Section 3.2, Eq. 5: the experts of the predicted
// prefetch set are loaded before generation begins), without the host in the loop.
//
//   preload_plan_kernel   one warp walks the caller's list: every id is one cache request of its own
//                         (a resident expert is re-stamped, a missing one takes the lowest empty slot,
//                         else the policy's victim), exactly as the planning kernels treat a miss, and
//                         writes the list of (expert, slot) pairs that have to be fetched.
//   fetch_experts_kernel  every CTA copies its share of the rows of each listed expert from the
//                         page-locked host store (read over the host link by the SMs themselves) into
//                         the expert's slot: bulk copy global -> shared -> global, two buffers in turn.
//
// Both run on the handle's copy stream; the first forward call afterwards waits for their event.
// Where the device cannot read the host store (or the store is 4-bit), the host issues the copies
// from the list instead.
#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr long long kWaitLimitCycles = 4000000000ll;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

__global__ void __launch_bounds__(32) preload_plan_kernel(PreloadParams p)
{
    const int lane = threadIdx.x;
    DevCache *c = p.cache;
    PreloadList *out = p.list;
    int n_fetch = 0;
    // one request per id, in order; lane = slot for the victim search
    for (int i = 0; i < p.n; ++i) {
        const int e = p.ids[i];
        unsigned long long st = 0;
        int slot = -1;
        if (lane == 0) {
            st = ++c->counter;
            if (p.policy == MELINOE_POLICY_COUNT)
                c->count[e] += 1.0f;           // no decay step: the definition's initial count vector
            slot = c->slot_of_expert[e];
        }
        st = __shfl_sync(0xffffffffu, st, 0);
        slot = __shfl_sync(0xffffffffu, slot, 0);
        if (slot >= 0) {
            if (lane == 0) {
                c->stamp[slot] = st;
                c->tot_hits += 1;
            }
            __syncwarp();
            continue;
        }
        // victim: lowest empty slot, else the smallest (count of the occupant under the count policy, stamp)
        unsigned long long khi = ~0ull, klo = ~0ull;
        int best = -1;
        for (int s = lane; s < p.C; s += 32) {
            const int occ = c->expert_of_slot[s];
            unsigned long long hi, lo;
            if (occ < 0) {
                hi = 0ull;
                lo = (unsigned long long)s;
            } else {
                hi = p.policy == MELINOE_POLICY_COUNT ? ((1ull << 32) | (unsigned long long)__float_as_uint(c->count[occ])) : (1ull << 32);
                lo = c->stamp[s];
            }
            if (hi < khi || (hi == khi && lo < klo)) {
                khi = hi;
                klo = lo;
                best = s;
            }
        }
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) {
            const unsigned long long ohi = __shfl_xor_sync(0xffffffffu, khi, m);
            const unsigned long long olo = __shfl_xor_sync(0xffffffffu, klo, m);
            const int ob = __shfl_xor_sync(0xffffffffu, best, m);
            if (ohi < khi || (ohi == khi && olo < klo)) {
                khi = ohi;
                klo = olo;
                best = ob;
            }
        }
        if (lane == 0) {
            const int ev = c->expert_of_slot[best];
            if (ev >= 0) {
                c->slot_of_expert[ev] = -1;
                c->tot_evictions += 1;
            }
            c->expert_of_slot[best] = e;
            c->slot_of_expert[e] = best;
            c->stamp[best] = st;
            c->tot_misses += 1;
            out->expert[n_fetch] = e;
            out->slot[n_fetch] = best;
            if (p.host_list) {
                p.host_list->expert[n_fetch] = e;
                p.host_list->slot[n_fetch] = best;
            }
        }
        ++n_fetch;
        __syncwarp();
    }
    if (lane == 0) {
        out->n = n_fetch;
        if (p.host_list) {
            __threadfence_system();
            p.host_list->n = n_fetch;
            *reinterpret_cast<volatile uint32_t *>(&p.host_list->seq) = p.seq;
        }
    }
}

// Copies listed experts host store -> slot.  A later entry may name a slot an earlier one filled
// (a list longer than the free slots): entries are processed in order by every CTA, and two entries
// that share a slot touch the same row range in the same CTA, one after the other.
__global__ void __launch_bounds__(64, 1) fetch_experts_kernel(FetchParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t s_bar[2];
    if (threadIdx.x != 0)
        return;
    int s_bad = 0;                       // 1: a wait ran out, 2: the list names an expert the device cannot read
    const uint32_t bar0 = smem_u32(s_bar), buf0 = smem_u32(smem);
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0), "r"(1));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0 + 8), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const int n = p.list->n;
    const long long rows_lo = (long long)blockIdx.x * p.rows / gridDim.x, rows_hi = (long long)(blockIdx.x + 1) * p.rows / gridDim.x;
    uint32_t k = 0;                      // pieces issued so far: piece k uses buffer k & 1
    for (int i = 0; i < n && !s_bad; ++i) {
        const int e = p.list->expert[i], slot = p.list->slot[i];
        if (e < 0 || e >= kMaxExperts || slot < 0 || slot >= kMaxExperts) {
            s_bad = 2;
            break;
        }
        const char *src = p.host_blobs[e];
        char *dst = p.slots + (size_t)slot * p.slot_stride;
        if (src == nullptr) {
            s_bad = 2;
            break;
        }
        for (long long r = rows_lo; r < rows_hi; r += p.rows_per_piece, ++k) {
            const long long nr = rows_hi - r < p.rows_per_piece ? rows_hi - r : p.rows_per_piece;
            const uint32_t bytes = (uint32_t)(nr * p.row_bytes);
            const uint32_t b = k & 1u, bar = bar0 + 8 * b, buf = buf0 + b * p.piece_bytes;
            if (k >= 2)
                asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the store that last read this buffer
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(buf), "l"(src + (size_t)r * p.row_bytes), "r"(bytes), "r"(bar)
                         : "memory");
            const long long t0 = clock64();
            while (!mbar_try(bar, (k >> 1) & 1u)) {
                if (clock64() - t0 > kWaitLimitCycles) {
                    s_bad = 1;
                    break;
                }
            }
            if (s_bad)
                break;
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         ::"l"(dst + (size_t)r * p.row_bytes), "r"(buf), "r"(bytes)
                         : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (s_bad)
        atomicExch(p.err, s_bad == 2 ? MELINOE_ERR_STATE : MELINOE_ERR_TIMEOUT);
}

}  // namespace

cudaError_t launch_preload_plan(cudaStream_t stream, const PreloadParams &p)
{
    preload_plan_kernel<<<1, 32, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_fetch_experts(cudaStream_t stream, int n_sms, const FetchParams &p)
{
    static bool configured = false;
    if (!configured) {
        const cudaError_t e = cudaFuncSetAttribute(fetch_experts_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 49152);
        if (e != cudaSuccess)
            return e;
        configured = true;
    }
    fetch_experts_kernel<<<n_sms, 64, 2 * p.piece_bytes, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace melinoe
