// Grouped GEMM of the expert FFN (Eq. 3) for prompts with many tokens per expert, on CTA pairs:
// the same two GEMMs as ffn_gemm.cu, but one MMA spans two SMs (tcgen05.mma.cta_group::2,
// M = 256 tokens x N = 256), so a 256-row B tile is staged once for 256 token rows instead of
// once for 128: each CTA of the pair stages its own 128 token rows of A and HALF of the B tile.
// A single CTA stages 48 KB of operands for 128 x 256 x 64 multiply-adds (85 flop per byte); at
// the full tensor rate that is more than shared memory can be fed with from L2.  The pair stages
// 2 x 32 KB for twice the work: 128 flop per byte.
//
//   cluster of 2 CTAs, item = (request, n-tile, 256-token m-tile); CTA r of the pair owns token
//   rows row0 + 128 r .. + 127 and B rows 128 r .. 128 r + 127 of the tile (GEMM 1: CTA 0 the
//   W_g rows, CTA 1 the W_u rows, so the accumulator still holds g in columns 0..127 and u in
//   128..255; GEMM 2: the two halves of 256 W_d rows).
//   warp 0  TMA producer in BOTH CTAs; every load signals the "full" barrier of the pair's first
//           CTA (the .cta_group::2 form of the load routes the completion there; no load is
//           broadcast to more than one CTA).
//   warp 1  MMA issuer, first CTA only: waits for a stage's bytes from both CTAs, issues four
//           K = 16 MMAs, commits to the stage's "empty" barrier in both CTAs; after the last
//           stage of an item commits to the accumulator's "full" barrier in both CTAs.
//   warps 2..5  epilogue in both CTAs, each on its own 128 accumulator rows in its own tensor
//           memory; they release the accumulator by arriving on the first CTA's barrier.
//
// Ragged M as in the one-CTA kernel: rows past the expert's last are computed and not stored
// (past the end of the buffer the loads return zeros).  Every wait is bounded.  The pair meets at
// a cluster barrier before tensor memory is freed, so neither CTA leaves while the other may
// still read its shared memory or signal its barriers.
#include <cuda.h>

#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kPairThreads = 192;          // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int kPM = 128;                   // token rows per CTA (256 per pair)
constexpr int kPK = 64;                    // K elements per stage (128 bytes)
constexpr int kPN = 256;                   // accumulator columns
constexpr int kPStages = 6;
constexpr int kPABytes = kPM * kPK * 2, kPBBytes = (kPN / 2) * kPK * 2, kPStageBytes = kPABytes + kPBBytes;   // 16 + 16 KB
constexpr long long kPairWaitCycles = 4000000000ll;
constexpr uint32_t kLeaderMask = 0xFEFFFFFFu;   // clears the CTA-rank bit of a shared::cluster address of the pair

__device__ __forceinline__ uint32_t p_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool p_mbar_try(uint32_t bar, uint32_t parity)
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

__device__ __forceinline__ bool p_mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (p_mbar_try(bar, parity))
        return true;
    if (*abort_flag)
        return false;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (p_mbar_try(bar, parity))
                return true;
        if (*abort_flag)
            return false;
        if (clock64() - t0 > kPairWaitCycles) {
            *abort_flag = 1;
            return false;
        }
    }
}

__device__ __forceinline__ void p_mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void p_mbar_expect(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// arrive on a barrier that may live in the other CTA of the pair (a shared::cluster address)
__device__ __forceinline__ void p_mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// shared::cluster address of this CTA's shared-memory location `addr` in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t p_map_to_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}

// 2-D tiled TMA load into this CTA's shared memory; the completion goes to the barrier at the same
// offset in the pair's first CTA.
__device__ __forceinline__ void p_tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar & kLeaderMask)
        : "memory");
}

// K-major operand, 128-byte swizzle, rows of 128 bytes, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t p_smem_desc_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// bf16 x bf16 -> fp32, both operands K-major.
__device__ __forceinline__ uint32_t p_instr_desc_bf16(int m, int n)
{
    uint32_t d = 0;
    d |= 1u << 4;
    d |= 1u << 7;
    d |= 1u << 10;
    d |= (uint32_t)(n >> 3) << 17;
    d |= (uint32_t)(m >> 4) << 24;
    return d;
}

__device__ __forceinline__ void p_umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The barrier (a shared::cluster address, this CTA's or the peer's) receives one arrival when all
// MMAs issued so far by this thread have completed.
__device__ __forceinline__ void p_umma_commit(uint32_t cluster_bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_bar) : "memory");
}

__device__ __forceinline__ void p_tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}

__device__ __forceinline__ uint32_t p_bf16_rne(float v)
{
    uint32_t u = __float_as_uint(v);
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

struct PairItem {
    int row0;      // first sorted row of THIS CTA's 128 token rows
    int row_end;   // one past the expert's last sorted row
    int b_row;     // first row of THIS CTA's half of the B tile in its tensor map
    int n0;        // first output column of the tile (f for GEMM 1, output column for GEMM 2)
    int shared;    // B comes from a shared expert's tensor map: index of that expert, else -1
};

template <int PHASE>
__global__ void __launch_bounds__(kPairThreads, 1) ffn_gemm_pair_kernel(GemmParams p)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[2 * kPStages + 4];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ int s_req[kMaxReq], s_tile0[kMaxReq + 1], s_nreq;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const DevPlan *plan = p.plan;
    if (plan->status != MELINOE_OK)
        return;
    unsigned char *ring = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t ring_s = p_smem_u32(ring);
    const uint32_t full0 = p_smem_u32(s_bars), empty0 = full0 + 8 * kPStages;
    const uint32_t tfull0 = empty0 + 8 * kPStages, tempty0 = tfull0 + 16;
    volatile int *abort_flag = &s_abort;

    const int K = PHASE == 1 ? p.d : p.F;
    const int n_tiles_n = PHASE == 1 ? p.F / 128 : p.d / kPN;
    if (tid == 0) {
        s_abort = 0;
        int n = 0, tiles = 0;
        const int n_req_total = plan->n_req + p.n_shared;
        for (int r = 0; r < n_req_total; ++r) {
            const ReqRec rec = plan->req[r];
            if (rec.group == p.group && rec.n_tok > 0) {
                s_req[n] = r;
                s_tile0[n] = tiles;
                tiles += (rec.n_tok + 2 * kPM - 1) / (2 * kPM) * n_tiles_n;
                ++n;
            }
        }
        s_tile0[n] = tiles;
        s_nreq = n;
        for (int i = 0; i < kPStages; ++i) {
            p_mbar_init(full0 + 8 * i, 1);      // the first CTA's: its producer's expect-arrival; both CTAs' bytes land here
            p_mbar_init(empty0 + 8 * i, 1);     // one commit per use, in each CTA
        }
        p_mbar_init(tfull0, 1);
        p_mbar_init(tfull0 + 8, 1);
        p_mbar_init(tempty0, 8);                // the first CTA's: four epilogue warps of each CTA
        p_mbar_init(tempty0 + 8, 8);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int n_reqs = s_nreq;
    const int total_items = s_tile0[n_reqs];
    if (total_items == 0)
        return;                                 // both CTAs of the pair see the same plan

    // both CTAs' barriers exist before either is signalled from the other side
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");

    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(p_smem_u32(&s_tmem_base)),
                     "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = s_tmem_base;

    auto item_of = [&](int w) -> PairItem {
        int q = 0;
        while (q + 1 < n_reqs && s_tile0[q + 1] <= w)
            ++q;
        const ReqRec rec = plan->req[s_req[q]];
        const int local = w - s_tile0[q];
        const int mtiles = (rec.n_tok + 2 * kPM - 1) / (2 * kPM);
        const int nt = local / mtiles, mt = local % mtiles;
        PairItem it;
        it.row0 = rec.tok_off + mt * 2 * kPM + (int)rank * kPM;
        it.row_end = rec.tok_off + rec.n_tok;
        it.shared = rec.slot >= 0 ? -1 : rec.expert - p.E;
        const int base_expert = rec.slot >= 0 ? rec.slot : 0;
        if (PHASE == 1) {
            it.n0 = nt * 128;
            it.b_row = base_expert * 3 * p.F + it.n0 + (int)rank * p.F;               // CTA 0: W_g rows, CTA 1: W_u rows
        } else {
            it.n0 = nt * kPN;
            it.b_row = base_expert * 3 * p.d + 2 * p.d + it.n0 + (int)rank * (kPN / 2);
        }
        return it;
    };
    const int kblocks = K / kPK;

    if (warp == 0) {
        // ============================================================ TMA producer (both CTAs)
        if (lane == 0) {
            const CUtensorMap *map_a = p.maps + (PHASE == 1 ? kMapXs : kMapHs);
            uint32_t n = 0;
            for (int w = pair; w < total_items && !*abort_flag; w += n_pairs) {
                const PairItem it = item_of(w);
                const CUtensorMap *map_b =
                    PHASE == 1 ? (it.shared < 0 ? p.maps + kMapSlotsD : p.maps + kMapShared0 + 2 * it.shared)
                               : (it.shared < 0 ? p.maps + kMapSlotsF128 : p.maps + kMapSharedF128 + it.shared);
                for (int kb = 0; kb < kblocks; ++kb, ++n) {
                    const uint32_t s = n % kPStages;
                    if (n >= (uint32_t)kPStages && !p_mbar_wait(empty0 + 8 * s, ((n / kPStages) - 1u) & 1u, abort_flag))
                        break;
                    const uint32_t bar = full0 + 8 * s;
                    const uint32_t a_dst = ring_s + s * kPStageBytes, b_dst = a_dst + kPABytes;
                    if (rank == 0)
                        p_mbar_expect(bar, 2 * kPStageBytes);       // this CTA's bytes and the peer's
                    p_tma_load_2d(a_dst, map_a, kb * kPK, it.row0, bar);
                    p_tma_load_2d(b_dst, map_b, kb * kPK, it.b_row, bar);
                }
            }
        }
    } else if (warp == 1) {
        // ============================================================ MMA issuer (first CTA of the pair)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = p_instr_desc_bf16(2 * kPM, kPN);
            const uint32_t peer_empty0 = p_map_to_rank(empty0, 1), peer_tfull0 = p_map_to_rank(tfull0, 1);
            uint32_t n = 0, item = 0;
            for (int w = pair; w < total_items && !*abort_flag; w += n_pairs, ++item) {
                const uint32_t acc = item & 1u;
                if (item >= 2 && !p_mbar_wait(tempty0 + 8 * acc, ((item >> 1) - 1u) & 1u, abort_flag))
                    break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + acc * kPN;
                bool ok = true;
                for (int kb = 0; kb < kblocks; ++kb, ++n) {
                    const uint32_t s = n % kPStages;
                    if (!p_mbar_wait(full0 + 8 * s, (n / kPStages) & 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = ring_s + s * kPStageBytes, b_addr = a_addr + kPABytes;
                    const uint64_t a_desc = p_smem_desc_sw128(a_addr), b_desc = p_smem_desc_sw128(b_addr);
#pragma unroll
                    for (int ks = 0; ks < kPK / 16; ++ks)
                        p_umma_bf16(d_tmem, a_desc + 2 * ks, b_desc + 2 * ks, idesc, (kb | ks) != 0);
                    p_umma_commit(empty0 + 8 * s);               // the stage is free in this CTA ...
                    p_umma_commit(peer_empty0 + 8 * s);          // ... and in the peer
                }
                if (!ok)
                    break;
                p_umma_commit(tfull0 + 8 * acc);                 // the accumulator is complete, here ...
                p_umma_commit(peer_tfull0 + 8 * acc);            // ... and in the peer's tensor memory
            }
        }
    } else {
        // ============================================================ epilogue (warps 2..5, both CTAs)
        const int quarter = warp & 3;
        const uint32_t lead_tempty0 = p_map_to_rank(tempty0, 0);
        uint32_t item = 0;
        for (int w = pair; w < total_items && !*abort_flag; w += n_pairs, ++item) {
            const PairItem it = item_of(w);
            const uint32_t acc = item & 1u;
            if (!p_mbar_wait(tfull0 + 8 * acc, (item >> 1) & 1u, abort_flag))
                break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int row = it.row0 + quarter * 32 + lane;
            const bool live = row < it.row_end;
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kPN;
            if (PHASE == 1) {
#pragma unroll 1
                for (int c = 0; c < 128; c += 32) {
                    uint32_t g[32], u[32];
                    p_tmem_ld32(t_row + c, g);
                    p_tmem_ld32(t_row + 128 + c, u);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (live) {
                        uint4 *dst = reinterpret_cast<uint4 *>(p.hs + (size_t)row * p.F + it.n0 + c);
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint32_t o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float g0 = __uint_as_float(g[v * 8 + 2 * e]), g1 = __uint_as_float(g[v * 8 + 2 * e + 1]);
                                const float u0 = __uint_as_float(u[v * 8 + 2 * e]), u1 = __uint_as_float(u[v * 8 + 2 * e + 1]);
                                const float h0 = g0 / (1.0f + __expf(-g0)) * u0, h1 = g1 / (1.0f + __expf(-g1)) * u1;
                                o[e] = p_bf16_rne(h0) | (p_bf16_rne(h1) << 16);
                            }
                            dst[v] = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < kPN; c += 32) {
                    uint32_t z[32];
                    p_tmem_ld32(t_row + c, z);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (live) {
                        uint4 *dst = reinterpret_cast<uint4 *>(p.zs + (size_t)row * p.d + it.n0 + c);
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            dst[v] = make_uint4(z[4 * v], z[4 * v + 1], z[4 * v + 2], z[4 * v + 3]);
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0)
                p_mbar_arrive_cluster(lead_tempty0 + 8 * acc);
        }
    }

    // ---- the pair is done with tensor memory and with each other's shared memory: meet, then free
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 2)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
    if (*abort_flag && tid == 0)
        atomicExch(p.err, MELINOE_ERR_TIMEOUT);
}

constexpr size_t kPairSmem = (size_t)kPStages * kPStageBytes + 1024;

}  // namespace

cudaError_t ffn_gemm_pair_configure()
{
    cudaError_t e = cudaFuncSetAttribute(ffn_gemm_pair_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmem);
    if (e != cudaSuccess)
        return e;
    return cudaFuncSetAttribute(ffn_gemm_pair_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmem);
}

cudaError_t launch_ffn_gemm_pair(cudaStream_t stream, int phase, int n_sms, const GemmParams &p)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_sms & ~1));
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = kPairSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = phase == 1 ? cudaLaunchKernelEx(&cfg, ffn_gemm_pair_kernel<1>, p)
                                     : cudaLaunchKernelEx(&cfg, ffn_gemm_pair_kernel<2>, p);
    count_launch();
    return e;
}

}  // namespace melinoe
