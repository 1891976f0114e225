// Expert FFN (Eq. 3) for calls with many tokens per expert (prefill): a grouped GEMM on the
// fifth-generation tensor cores (tcgen05.mma, accumulators in tensor memory, operands staged
// in shared memory by TMA), plus the token gather in front of it and the combine (Eq. 2) behind.
//
//   gather    Xs[pos] = hidden[token of sorted position pos]: the tokens of one expert become
//             consecutive rows, so an expert's activations are one 2-D box for TMA.
//   GEMM 1    per expert: [G | U] = Xs_e (M_e x d) * [W_g ; W_u]^T, tile 128 tokens x 128 f:
//             one MMA of N = 256 whose B tile stacks 128 rows of W_g on 128 rows of W_u, so the
//             accumulator holds g in columns 0..127 and u in 128..255 of the same token row and
//             the epilogue forms h = SiLU(g) * u in registers; h is stored as bf16.
//   GEMM 2    per expert: Z = H_e (M_e x F) * W_d^T, tile 128 tokens x 256 output columns, fp32.
//   combine   y_t = sum_j gate[t][j] * Z[pos(t, j)] (+ shared experts), rank order, one rounding.
//
// The expert blob (see melinoe_moe_pack_expert) holds, per hidden unit f, the rows W_g[f], W_u[f]
// and W_d[:, f], each d elements, with the 16-byte pieces of every 128-byte group stored at
// (piece xor (f mod 8)).  That permutation is exactly what a TMA load with 128-byte swizzle would
// have produced in shared memory from plain rows, as long as a tile starts at a multiple of 8 rows
// and 64 columns; so the weight tiles are fetched by TMA WITHOUT swizzle and the MMA descriptors
// name the 128-byte-swizzled layout.  W_g and W_u rows are "N x K, K contiguous" (K-major, like the
// activations Xs and H, which are plain and fetched with TMA swizzle); the W_d^T rows are
// "K x N, N contiguous": GEMM 2 takes its B operand N-major (four 64-column boxes per stage).
// The experts of all slots are addressed through one tensor map per view (W_g rows, W_u rows,
// W_d^T rows: the same row pitch of 6 d bytes, different offsets), because the slots are contiguous.
//
// One persistent CTA per SM, warp-specialised: warp 0 issues TMA loads into a 4-stage ring,
// warp 1 issues the MMAs (one elected thread) and commits them to mbarriers, warps 2..5 drain
// the accumulator (tcgen05.ld, 32 rows per warp) and write the tile.  Two accumulators of 256
// columns alternate so the epilogue of a tile overlaps the MMAs of the next.  Work items are
// (request, n-tile, m-tile) triples of the launch's compute group, dealt round-robin.
//
// Ragged M: an m-tile may run past its expert's last row; those rows are computed on whatever
// the next rows hold (or zeros past the end of the buffer) and never stored.
//
// CTA pairs (template parameter CG = 2, used where the experts have enough tokens): two CTAs of a
// cluster on neighbouring SMs take two adjacent m-tiles of the same expert and n-tile and run them
// as ONE tensor-core operation of M = 256 (tcgen05.mma.cta_group::2, issued by the even CTA).  Each
// CTA stages its own 128 activation rows but only HALF of the weight tile (128 of its 256 columns);
// the tensor cores of both SMs read both halves.  Per CTA and k-block that is 32 KB instead of 48 KB
// through shared memory for the same arithmetic, which is what limits the single-CTA form, and the
// ring holds 6 stages instead of 4.  Both CTAs' loads complete on the even CTA's barrier; its MMA
// thread frees a stage, and hands over an accumulator, in both CTAs at once (commit with cluster
// multicast); the odd CTA's epilogue warps report to the even CTA's barrier.  Each CTA drains its own
// accumulator rows.
//
// Every wait is bounded; on a timeout the CTA raises its abort flag, every role leaves its
// loops, tensor memory is freed and the error word tells the host.
#include <cuda.h>

#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kGemmThreads = 192;          // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int kBM = 128, kBK = 64;         // tile rows (tokens), K elements per stage (128 bytes)
constexpr int kBN = 256;                   // accumulator columns: 128 g + 128 u, or 256 outputs
constexpr int kABytes = kBM * kBK * 2, kBBytes = kBN * kBK * 2;
// ring stages and bytes of a stage for the single-CTA form (CG = 1) and the CTA-pair form (CG = 2)
__host__ __device__ constexpr int gemm_stages(int cg) { return cg == 2 ? 6 : 4; }
__host__ __device__ constexpr int gemm_stage_bytes(int cg) { return kABytes + kBBytes / cg; }
constexpr long long kGemmWaitCycles = 4000000000ll;

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

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try(bar, parity))
        return true;
    if (*abort_flag)
        return false;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity))
                return true;
        if (*abort_flag)
            return false;
        if (clock64() - t0 > kGemmWaitCycles) {
            *abort_flag = 1;
            return false;
        }
    }
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// 2-D tiled TMA load: box at (x = element column, y = row) of the tensor map into shared memory.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// The same from a CTA of a pair: the completion may be counted on the peer CTA's barrier (bar is an
// address in the cluster's shared window).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// Address of this CTA's shared-memory location `addr` in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t cluster_addr(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, groups
// of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);          // start address
    d |= (uint64_t)(1024u >> 4) << 32;                // stride between 8-row groups
    d |= (uint64_t)1 << 46;                           // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                           // 128-byte swizzle
    return d;
}

// The same for an N-major B operand made of 64-column boxes (64 K rows of 128 bytes each, 8 KB per
// box): the boxes follow one another along N (leading offset), groups of 8 K rows are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128_nmajor(uint32_t addr)
{
    uint64_t d = smem_desc_sw128(addr);
    d |= (uint64_t)(8192u >> 4) << 16;                // between 64-column boxes
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K-major or N-major, M = 128, N = 256.
__device__ __forceinline__ uint32_t instr_desc_bf16(int m, int n, bool b_nmajor)
{
    uint32_t d = 0;
    d |= 1u << 4;                    // D format: fp32
    d |= 1u << 7;                    // A format: bf16
    d |= 1u << 10;                   // B format: bf16
    d |= (b_nmajor ? 1u : 0u) << 16; // B major: 0 = K, 1 = N
    d |= (uint32_t)(n >> 3) << 17;
    d |= (uint32_t)(m >> 4) << 24;
    return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// The pair forms: one operation over both CTAs' tensor cores; the commit arrives on the barrier at this
// offset in both CTAs of the pair.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3)
                 : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
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

__device__ __forceinline__ uint32_t bf16_rne(float v)
{
    uint32_t u = __float_as_uint(v);
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

struct GemmItem {
    int row0;      // first sorted row of the m-tile
    int row_end;   // one past the expert's last sorted row
    int b_row;     // first expert row of its tensor maps (its slot times F, 0 for a shared expert)
    int n0;        // first output column of the tile (f for GEMM 1, output column for GEMM 2)
    int shared;    // B comes from a shared expert's tensor map: index of that expert, else -1
};

// PHASE 1: h = SiLU(Xs W_g^T) * (Xs W_u^T) -> hs (bf16).  PHASE 2: z = hs W_d^T -> zs (fp32).
template <int PHASE, int CG>
__global__ void __launch_bounds__(kGemmThreads, 1) ffn_gemm_kernel(GemmParams p)
{
    constexpr int kStages = gemm_stages(CG), kStageBytes = gemm_stage_bytes(CG);
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ uint64_t s_bars[2 * kStages + 4];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ int s_tile0[kMaxReq + 1], s_nreq;
    __shared__ int4 s_rec[kMaxReq];                          // tok_off, n_tok, slot, expert of the launch's requests

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const DevPlan *plan = p.plan;
    if (plan->status != MELINOE_OK)
        return;
    // 1024-byte aligned ring (the swizzle pattern repeats every 1024 bytes)
    unsigned char *ring = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t ring_s = smem_u32(ring);
    const uint32_t full0 = smem_u32(s_bars), empty0 = full0 + 8 * kStages;
    const uint32_t tfull0 = empty0 + 8 * kStages, tempty0 = tfull0 + 16;
    volatile int *abort_flag = &s_abort;
    // rank within the CTA pair; the even CTA issues the MMAs, owns the "stage full" barriers and counts
    // the drained accumulators of both
    uint32_t rank = 0;
    if (CG == 2)
        asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int n_units = (int)gridDim.x / CG, unit = (int)blockIdx.x / CG;    // CTAs, or CTA pairs, that share out the items

    // ---- the launch's requests and their m-tiles (CG = 2: pairs of m-tiles)
    const int K = PHASE == 1 ? p.d : p.F;                 // reduction length
    const int n_tiles_n = PHASE == 1 ? p.F / 128 : p.d / kBN;
    if (tid == 0) {
        s_abort = 0;
        int n = 0, tiles = 0;
        const int n_req_total = plan->n_req + p.n_shared;
        for (int r = 0; r < n_req_total; ++r) {
            const ReqRec rec = plan->req[r];
            if (rec.group == p.group && rec.n_tok > 0) {
                s_rec[n] = make_int4(rec.tok_off, rec.n_tok, rec.slot, rec.expert);
                s_tile0[n] = tiles;
                tiles += (rec.n_tok + CG * kBM - 1) / (CG * kBM) * n_tiles_n;
                ++n;
            }
        }
        s_tile0[n] = tiles;
        s_nreq = n;
        for (int i = 0; i < kStages; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, 1);
        }
        mbar_init(tfull0, 1);
        mbar_init(tfull0 + 8, 1);
        mbar_init(tempty0, 4 * CG);
        mbar_init(tempty0 + 8, 4 * CG);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int n_reqs = s_nreq;
    const int total_items = s_tile0[n_reqs];
    if (total_items == 0)
        return;

    // (the barriers of both CTAs exist before either signals the other's)
    if (CG == 2)
        cluster_sync_all();
    if (warp == 2) {
        if (CG == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                         "r"(512));
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
        } else {
            // the same warp of both CTAs, the same destination: one allocation over the pair
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                         "r"(512));
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = s_tmem_base;

    // item w -> (request, n-tile, m-tile): within a request the m-tiles of one n-tile are adjacent,
    // so CTAs working side by side share the weight tile in L2
    auto item_of = [&](int w) -> GemmItem {
        int q = 0;
        while (q + 1 < n_reqs && s_tile0[q + 1] <= w)
            ++q;
        const int4 rec = s_rec[q];                                  // tok_off, n_tok, slot, expert
        const int local = w - s_tile0[q];
        const int mtiles = (rec.y + CG * kBM - 1) / (CG * kBM);
        const int nt = local / mtiles, mt = local % mtiles;
        GemmItem it;
        it.row0 = rec.x + (mt * CG + (int)rank) * kBM;              // this CTA's 128 rows of the item
        it.row_end = rec.x + rec.y;
        it.shared = rec.z >= 0 ? -1 : rec.w - p.E;
        it.b_row = (rec.z >= 0 ? rec.z : 0) * p.F;                  // shared experts have maps of their own
        it.n0 = PHASE == 1 ? nt * 128 : nt * kBN;
        return it;
    };
    const int kblocks = K / kBK;

    if (warp == 0) {
        // ============================================================ TMA producer
        if (lane == 0) {
            const CUtensorMap *map_a = p.maps + (PHASE == 1 ? kMapXs : kMapHs);
            uint32_t n = 0;
            for (int w = unit; w < total_items && !*abort_flag; w += n_units) {
                const GemmItem it = item_of(w);
                // W_g rows, W_u rows, W_d^T rows of the slots, or of the shared expert
                const CUtensorMap *map_w = it.shared < 0 ? p.maps + kMapSlotsG : p.maps + kMapShared0 + 3 * it.shared;
                for (int kb = 0; kb < kblocks; ++kb, ++n) {
                    const uint32_t s = n % kStages;
                    if (n >= (uint32_t)kStages && !mbar_wait(empty0 + 8 * s, ((n / kStages) - 1u) & 1u, abort_flag))
                        break;
                    const uint32_t a_dst = ring_s + s * kStageBytes, b_dst = a_dst + kABytes;
                    if (CG == 1) {
                        const uint32_t bar = full0 + 8 * s;
                        mbar_expect(bar, kStageBytes);
                        tma_load_2d(a_dst, map_a, kb * kBK, it.row0, bar);
                        if (PHASE == 1) {
                            tma_load_2d(b_dst, map_w, kb * kBK, it.b_row + it.n0, bar);                   // 128 rows of W_g
                            tma_load_2d(b_dst + kBBytes / 2, map_w + 1, kb * kBK, it.b_row + it.n0, bar); // 128 rows of W_u
                        } else {
                            // 64 rows f of W_d^T, four boxes of 64 output columns
#pragma unroll
                            for (int i = 0; i < kBN / 64; ++i)
                                tma_load_2d(b_dst + i * 8192, map_w + 2, it.n0 + 64 * i, it.b_row + kb * kBK, bar);
                        }
                    } else {
                        // the bytes of both CTAs are expected, once, on the even CTA's barrier
                        const uint32_t bar = cluster_addr(full0 + 8 * s, 0);
                        if (rank == 0)
                            mbar_expect(full0 + 8 * s, 2 * kStageBytes);
                        tma_load_2d_pair(a_dst, map_a, kb * kBK, it.row0, bar);
                        if (PHASE == 1) {
                            // columns 0..127 of the accumulator (g) come from the even CTA's half, 128..255 (u) from the odd one's
                            tma_load_2d_pair(b_dst, map_w + rank, kb * kBK, it.b_row + it.n0, bar);
                        } else {
#pragma unroll
                            for (int i = 0; i < 2; ++i)
                                tma_load_2d_pair(b_dst + i * 8192, map_w + 2, it.n0 + 64 * (2 * (int)rank + i), it.b_row + kb * kBK, bar);
                        }
                    }
                }
            }
            if (CG == 2) {
                // The MMA thread's commits arrive on this CTA's barriers from outside: wait for the last
                // ones so that none is still under way when the CTA ends.
                for (uint32_t j = n > (uint32_t)kStages ? n - kStages : 0; j < n && !*abort_flag; ++j)
                    mbar_wait(empty0 + 8 * (j % kStages), (j / kStages) & 1u, abort_flag);
            }
        }
    } else if (warp == 1) {
        // ============================================================ MMA issuer (of a pair: the even CTA's)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc_bf16(CG * kBM, kBN, PHASE == 2);
            uint32_t n = 0, item = 0;
            for (int w = unit; w < total_items && !*abort_flag; w += n_units, ++item) {
                const uint32_t acc = item & 1u;
                if (item >= 2 && !mbar_wait(tempty0 + 8 * acc, ((item >> 1) - 1u) & 1u, abort_flag))
                    break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + acc * kBN;
                bool ok = true;
                for (int kb = 0; kb < kblocks; ++kb, ++n) {
                    const uint32_t s = n % kStages;
                    if (!mbar_wait(full0 + 8 * s, (n / kStages) & 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = ring_s + s * kStageBytes, b_addr = a_addr + kABytes;
                    const uint64_t a_desc = smem_desc_sw128(a_addr);
                    const uint64_t b_desc = PHASE == 1 ? smem_desc_sw128(b_addr) : smem_desc_sw128_nmajor(b_addr);
                    // 16 K elements: 32 bytes along a K-major row (2 descriptor units), 16 rows of 128 bytes
                    // in an N-major box (128 units)
                    constexpr int kBStep = PHASE == 1 ? 2 : 128;
#pragma unroll
                    for (int ks = 0; ks < kBK / 16; ++ks) {
                        if (CG == 1)
                            umma_bf16(d_tmem, a_desc + 2 * ks, b_desc + kBStep * ks, idesc, (kb | ks) != 0);
                        else
                            umma_bf16_pair(d_tmem, a_desc + 2 * ks, b_desc + kBStep * ks, idesc, (kb | ks) != 0);
                    }
                    // the stage is free once these MMAs have read it
                    if (CG == 1)
                        umma_commit(empty0 + 8 * s);
                    else
                        umma_commit_pair(empty0 + 8 * s);
                }
                if (!ok)
                    break;
                // the accumulator is complete
                if (CG == 1)
                    umma_commit(tfull0 + 8 * acc);
                else
                    umma_commit_pair(tfull0 + 8 * acc);
            }
        }
    } else {
        // ============================================================ epilogue (warps 2..5)
        const int quarter = warp & 3;                        // the 32 accumulator rows this warp may read
        uint32_t item = 0;
        for (int w = unit; w < total_items && !*abort_flag; w += n_units, ++item) {
            const GemmItem it = item_of(w);
            const uint32_t acc = item & 1u;
            if (!mbar_wait(tfull0 + 8 * acc, (item >> 1) & 1u, abort_flag))
                break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int row = it.row0 + quarter * 32 + lane;
            const bool live = row < it.row_end;
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kBN;
            if (PHASE == 1) {
#pragma unroll 1
                for (int c = 0; c < 128; c += 32) {
                    uint32_t g[32], u[32];
                    tmem_ld32(t_row + c, g);
                    tmem_ld32(t_row + 128 + c, u);
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
                                o[e] = bf16_rne(h0) | (bf16_rne(h1) << 16);
                            }
                            dst[v] = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < kBN; c += 32) {
                    uint32_t z[32];
                    tmem_ld32(t_row + c, z);
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
            if (lane == 0) {
                if (CG == 1 || rank == 0)
                    mbar_arrive(tempty0 + 8 * acc);
                else
                    mbar_arrive_cluster(cluster_addr(tempty0 + 8 * acc, 0));
            }
        }
    }

    // ---- everyone is done with tensor memory: free it
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // (a pair: neither CTA goes while the other may still signal it or read its shared memory)
    if (CG == 2)
        cluster_sync_all();
    if (warp == 2) {
        if (CG == 1)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
        else
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
    }
    if (*abort_flag && tid == 0)
        atomicExch(p.err, MELINOE_ERR_TIMEOUT);
}

// Xs[pos] = hidden[tok_of_sorted[pos]], one block per sorted row.
__global__ void __launch_bounds__(256) gather_rows_kernel(const DevPlan *plan, const uint16_t *__restrict__ x,
                                                          const int32_t *__restrict__ tok_of_sorted, uint16_t *xs, int d,
                                                          int n_sorted)
{
    if (plan->status != MELINOE_OK)
        return;
    for (int pos = blockIdx.x; pos < n_sorted; pos += gridDim.x) {
        const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)tok_of_sorted[pos] * d);
        uint4 *dst = reinterpret_cast<uint4 *>(xs + (size_t)pos * d);
        for (int i = threadIdx.x; i < d / 8; i += 256)
            dst[i] = src[i];
    }
}

// y_t = sum_j gate[t][j] * Z[inv_pos[t*k+j]] + sum_s Z[T*k + s*T + t], fp32 in rank order, bf16 out.
__global__ void __launch_bounds__(256) combine_rows_kernel(const DevPlan *plan, const float *__restrict__ gate,
                                                           const int32_t *__restrict__ inv_pos, const float *__restrict__ zs,
                                                           uint16_t *out, int T, int d, int k, int n_shared)
{
    const bool ok = plan->status == MELINOE_OK;
    for (int t = blockIdx.x; t < T; t += gridDim.x) {
        for (int c = threadIdx.x * 4; c < d; c += 256 * 4) {
            float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
            if (ok) {
                for (int j = 0; j < k; ++j) {
                    const float gw = gate[t * k + j];
                    const float4 z = *reinterpret_cast<const float4 *>(zs + (size_t)inv_pos[t * k + j] * d + c);
                    y.x = fmaf(gw, z.x, y.x);
                    y.y = fmaf(gw, z.y, y.y);
                    y.z = fmaf(gw, z.z, y.z);
                    y.w = fmaf(gw, z.w, y.w);
                }
                for (int s = 0; s < n_shared; ++s) {
                    const float4 z = *reinterpret_cast<const float4 *>(zs + ((size_t)T * k + (size_t)s * T + t) * d + c);
                    y.x += z.x;
                    y.y += z.y;
                    y.z += z.z;
                    y.w += z.w;
                }
            }
            uint2 o;
            o.x = bf16_rne(y.x) | (bf16_rne(y.y) << 16);
            o.y = bf16_rne(y.z) | (bf16_rne(y.w) << 16);
            *reinterpret_cast<uint2 *>(out + (size_t)t * d + c) = o;
        }
    }
}

constexpr size_t gemm_smem(int cg) { return (size_t)gemm_stages(cg) * gemm_stage_bytes(cg) + 1024; }

}  // namespace

bool ffn_gemm_supported(int d, int F) { return d % kBN == 0 && F % 128 == 0 && d >= kBN && F >= 128; }

cudaError_t ffn_gemm_configure()
{
    cudaError_t e = cudaFuncSetAttribute(ffn_gemm_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem(1));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(ffn_gemm_kernel<2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem(1));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(ffn_gemm_kernel<1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem(2));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(ffn_gemm_kernel<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem(2));
    return e;
}

cudaError_t launch_gather_rows(cudaStream_t stream, const DevPlan *plan, const uint16_t *x, const int32_t *tok_of_sorted,
                               uint16_t *xs, int d, int n_sorted, int n_sms)
{
    const int grid = n_sorted < n_sms * 16 ? n_sorted : n_sms * 16;
    gather_rows_kernel<<<grid, 256, 0, stream>>>(plan, x, tok_of_sorted, xs, d, n_sorted);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_ffn_gemm(cudaStream_t stream, int phase, int n_sms, bool pairs, const GemmParams &p)
{
    if (!pairs) {
        if (phase == 1)
            ffn_gemm_kernel<1, 1><<<n_sms, kGemmThreads, gemm_smem(1), stream>>>(p);
        else
            ffn_gemm_kernel<2, 1><<<n_sms, kGemmThreads, gemm_smem(1), stream>>>(p);
        count_launch();
        return cudaGetLastError();
    }
    // clusters of two CTAs on neighbouring SMs
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(n_sms / 2 * 2);
    lc.blockDim = dim3(kGemmThreads);
    lc.dynamicSmemBytes = gemm_smem(2);
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    const cudaError_t e = phase == 1 ? cudaLaunchKernelEx(&lc, ffn_gemm_kernel<1, 2>, p) : cudaLaunchKernelEx(&lc, ffn_gemm_kernel<2, 2>, p);
    count_launch();
    return e;
}

cudaError_t launch_combine_rows(cudaStream_t stream, const DevPlan *plan, const float *gate, const int32_t *inv_pos,
                                const float *zs, uint16_t *out, int T, int d, int k, int n_shared, int n_sms)
{
    const int grid = T < n_sms * 8 ? T : n_sms * 8;
    combine_rows_kernel<<<grid, 256, 0, stream>>>(plan, gate, inv_pos, zs, out, T, d, k, n_shared);
    count_launch();
    return cudaGetLastError();
}

}  // namespace melinoe
