// Streaming SwiGLU expert FFN (Eq. 3) with the gate-weighted combine (Eq. 2) fused in, for
// calls with few tokens per expert (decode).  The work is reading every needed expert once
// from HBM, so the kernel is built around keeping the memory system full: measured on B200,
// bulk copies of whole 4 KB rows stream at the full HBM rate while 256-byte pieces reach
// little more than half of it, so the unit of transfer is a whole row (or a 4 KB piece of a
// longer one).
//
// One cooperative launch per compute group, one CTA per SM: one producer warp and eight
// consumer warps.  A "virtual request" is one expert with up to 8 of its tokens.
//
//   phase 1  tile = 8 rows of W_g plus the same 8 rows of W_u of one virtual request.
//            D[16 x 8] = [W_g rows; W_u rows] (16 x d) * x^T (d x 8 tokens) on mma.sync
//            (bf16 in, fp32 accumulate); the eight warps split the columns of a stage and
//            their partial sums meet in shared memory once per tile.  In the accumulator
//            layout a thread holds g_f and u_f of the same f and the same two tokens, so
//            h = SiLU(g) * u is thread-local; h goes to global memory as bf16.
//   barrier  grid-wide, crossed by the producer warps only (bounded spin on a device counter):
//            the consumers never wait for it.  The ring is cut anew for the (usually shorter)
//            W_d rows as soon as the CTA's own phase 1 has drained, and as many W_d stages as
//            fit are in flight before the producer reaches the barrier.
//   phase 2  every CTA owns a contiguous range of the d_model output rows (d/G of them, so the
//            split is even to within one row) for ALL virtual requests of the launch.  Tile =
//            up to 16 of those W_d rows of one virtual request: D[16 x 8] = W_d rows * h^T, a
//            complete dot product over d_ff, so z needs no cross-CTA reduction; it goes to
//            z[pair][d] in fp32.
//   combine  in the call's last compute group every CTA, having finished its rows, sums
//            gate * z over the ranks in rank order (plus shared experts) for those rows and
//            writes them as bf16: it reads only what itself (or an earlier launch) wrote, so
//            no device-wide synchronisation is involved.  The result does not depend on how the
//            experts were split over groups.
//
// A stage of the shared-memory ring holds one piece (at most 4 KB) of each of the tile's 16
// weight rows plus the matching piece of up to 8 operand rows (hidden rows in phase 1, h rows
// in phase 2), each fetched by its own cp.async.bulk (one producer lane per row) completing on
// the stage's mbarrier.  Rows sit at a pitch of 16 bytes more than a multiple of 128, which
// makes the ldmatrix reads and the operand-fragment reads bank-conflict free.
//
// Every wait is bounded: when an mbarrier or the grid barrier does not complete in time the
// warp raises the CTA's abort flag, later waits fall through, the kernel ends normally and the
// error word tells the host.
#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStages = 8;
constexpr int kMaxChunk = 4096;                      // bytes of one row piece
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

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

// Bounded wait.  Returns false (and raises the CTA's abort flag) when the limit runs out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try(bar, parity))
        return true;
    if (*abort_flag)
        return false;
    const unsigned long long t0 = globaltimer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity))
                return true;
        if (*abort_flag)
            return false;
        if (globaltimer_ns() - t0 > kWaitLimitNs) {
            *abort_flag = 1;
            return false;
        }
    }
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_expect(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void consumer_bar()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// D(16x8) += A(16x16) * B(16x8), bf16 in, fp32 accumulate.
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

__device__ __forceinline__ uint16_t bf16_rne(float v)
{
    uint32_t u = __float_as_uint(v);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async;" ::: "memory");
}

__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// What the producer needs to know about a tile.
struct Tile {
    const char *src;     // this lane's source row (weights: lanes 0..15, operand rows: 16..23)
    int n_tok;           // tokens of the virtual request
    int n_rows;          // weight rows in the tile (16 except at the end of a CTA's row range)
};

__global__ void __launch_bounds__(kThreads, 1) ffn_stream_kernel(FfnParams p, FfnGeometry geo)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int d = p.d, F = p.F, Fpad = p.Fpad;
    const DevPlan *plan = p.plan;
    const int G = (int)gridDim.x;
    const int NOP = geo.n_op_rows;
    const int S1 = geo.n_stages, PITCH1 = geo.pitch, CB1 = geo.chunk_bytes, STAGE1 = (16 + NOP) * PITCH1;
    const int S2 = geo.n_stages2, PITCH2 = geo.pitch2, CB2 = geo.chunk_bytes2, STAGE2 = (16 + NOP) * PITCH2;

    // optional timeline: 8 device-clock stamps per CTA (see melinoe_moe_set_trace)
    unsigned long long *trace = p.trace ? p.trace + (size_t)blockIdx.x * 8 : nullptr;
    if (trace && tid == 0)
        trace[0] = globaltimer_ns();

    const int status = plan->status, n_groups = plan->n_groups;
    const int vb = plan->group_vr_begin[p.group];
    const int nv = plan->group_vr_begin[p.group + 1] - vb;
    if (status != MELINOE_OK) {
        // the call was refused on the device: the output is all zeros, the status tells why
        if (p.group == 0)
            for (size_t i = (size_t)blockIdx.x * kThreads + tid; i < (size_t)p.T * d; i += (size_t)G * kThreads)
                p.out[i] = 0;
        return;
    }
    const bool final_group = p.group == n_groups - 1;
    if (nv <= 0 && !final_group)
        return;

    // ring | reduction buffers | barriers (phase 1 full/empty, phase 2 full/empty)
    unsigned char *ring = smem;
    float *red = reinterpret_cast<float *>(smem + geo.ring_bytes);              // [2][8 warps][4][32]
    uint64_t *bars = reinterpret_cast<uint64_t *>(red + 2 * kConsumerWarps * 128);
    const uint32_t ring_s = smem_u32(ring);
    const uint32_t full1 = smem_u32(bars), empty1 = full1 + 8 * kMaxStages;
    const uint32_t full2 = empty1 + 8 * kMaxStages, empty2 = full2 + 8 * kMaxStages;
    volatile int *abort_flag = &s_abort;

    if (tid == 0) {
        s_abort = 0;
        for (int i = 0; i < kMaxStages; ++i) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full1 + 8 * i), "r"(1));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty1 + 8 * i), "r"(kConsumerWarps));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full2 + 8 * i), "r"(1));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty2 + 8 * i), "r"(kConsumerWarps));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (F % 16 != 0) {
        // the last 16-column step of a W_d row is half filled: what the copy leaves untouched
        // must be finite, because it meets the zero padding of the h rows in the product
        uint4 *z = reinterpret_cast<uint4 *>(ring);
        for (int i = tid; i < (int)(geo.ring_bytes / 16); i += kThreads)
            z[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async();
    }
    __syncthreads();
    if (trace && tid == 0)
        trace[1] = globaltimer_ns();

    // ---- phase 1: a contiguous range of (virtual request, 8-row f-block) tiles per CTA
    const int upe1 = F / 8;
    const int rb1 = 2 * d, rb2 = 2 * F;                       // row bytes
    const int nk1 = (rb1 + CB1 - 1) / CB1, nk2 = (rb2 + CB2 - 1) / CB2;
    const long long NT1 = (long long)nv * upe1;
    const int lo1 = (int)(blockIdx.x * NT1 / G), hi1 = (int)((blockIdx.x + 1) * NT1 / G);
    // ---- phase 2: output rows [r_lo, r_hi) of every virtual request, in tiles of up to 16 rows
    const int r_lo = (int)((long long)blockIdx.x * d / G), r_hi = (int)((long long)(blockIdx.x + 1) * d / G);
    const int mt = (r_hi - r_lo + 15) / 16;
    const int hi2 = nv * mt;

    if (warp == kConsumerWarps) {
        // =================================================================== producer
        // Per virtual request (looked up only when the tile sequence moves on to the next one):
        // this lane's source row of block 0 and its stride from one block to the next.
        int cur_vr = -1, cur_ntok = 0;
        const char *lane_base = nullptr;
        size_t lane_step = 0;
        // phase 1: lanes 0..7 W_g rows, 8..15 W_u rows, 16..23 hidden rows of the request's tokens
        auto tile1 = [&](int t) -> Tile {
            const int vr = vb + t / upe1, blk = t % upe1;
            if (vr != cur_vr) {
                const VrRec *v = p.vrs + vr;
                cur_vr = vr;
                cur_ntok = v->n_tok;
                lane_base = nullptr;
                lane_step = 0;
                if (lane < 16) {
                    lane_base = v->blob + (size_t)((lane < 8 ? 0 : F) + (lane & 7)) * rb1;
                    lane_step = (size_t)8 * rb1;
                } else if (lane - 16 < cur_ntok) {
                    lane_base = reinterpret_cast<const char *>(p.x) + (size_t)v->tok[lane - 16] * rb1;
                }
            }
            Tile ti;
            ti.n_tok = cur_ntok;
            ti.n_rows = 16;
            ti.src = lane_base ? lane_base + (size_t)blk * lane_step : nullptr;
            return ti;
        };
        // phase 2: lanes 0..15 W_d rows, 16..23 rows of h
        auto tile2 = [&](int t) -> Tile {
            const int vr = vb + t / mt, blk = t % mt;
            if (vr != cur_vr) {
                const VrRec *v = p.vrs + vr;
                cur_vr = vr;
                cur_ntok = v->n_tok;
                lane_base = nullptr;
                lane_step = 0;
                if (lane < 16) {
                    lane_base = v->blob + (size_t)2 * F * rb1 + (size_t)(r_lo + lane) * rb2;
                    lane_step = (size_t)16 * rb2;
                } else if (lane - 16 < cur_ntok) {
                    lane_base = reinterpret_cast<const char *>(p.hbuf) + ((size_t)vr * kTokPerVr + lane - 16) * Fpad * 2;
                }
            }
            Tile ti;
            ti.n_tok = cur_ntok;
            ti.n_rows = min(16, r_hi - r_lo - 16 * blk);
            ti.src = lane_base ? lane_base + (size_t)blk * lane_step : nullptr;
            if (lane < 16 && lane >= ti.n_rows)
                ti.src = nullptr;
            return ti;
        };
        bool dead = false;
        // One stage of either phase.  parts bit 0: wait for the slot, arm the barrier, fetch the
        // weight rows; bit 1: operand rows.  wbytes / obytes: bytes of each weight / operand piece.
        auto issue = [&](const Tile &ti, uint32_t full0, uint32_t empty0, int S, int STAGE, int PITCH, size_t src_off,
                         int wbytes, int obytes, int parts, uint32_t nn) {
            const uint32_t slot = nn % S;
            const uint32_t bar = full0 + 8 * slot;
            if (parts & 1) {
                if (nn >= (uint32_t)S && !dead)
                    dead = !mbar_wait(empty0 + 8 * slot, ((nn / S) - 1u) & 1u, abort_flag);
                if (lane == 0)
                    mbar_expect(bar, (uint32_t)ti.n_rows * wbytes + (uint32_t)ti.n_tok * obytes);
                __syncwarp();
            }
            if (ti.src && !dead) {
                const bool is_w = lane < 16;
                if (is_w ? (parts & 1) : (parts & 2))
                    bulk_g2s(ring_s + slot * STAGE + lane * PITCH, ti.src + src_off,
                             (uint32_t)(is_w ? wbytes : obytes), bar);
            }
        };
        uint32_t n1 = 0;
        for (int t = lo1; t < hi1; ++t) {
            const Tile ti = tile1(t);
            for (int kc = 0; kc < nk1; ++kc) {
                const int b = min(CB1, rb1 - kc * CB1);
                issue(ti, full1, empty1, S1, STAGE1, PITCH1, (size_t)kc * CB1, b, b, 3, n1++);
            }
        }
        // the ring is cut anew for phase 2: wait until the consumers have let go of every phase-1 stage
        for (uint32_t m = n1 > (uint32_t)S1 ? n1 - S1 : 0u; m < n1 && !dead; ++m)
            dead = !mbar_wait(empty1 + 8 * (m % S1), (m / S1) & 1u, abort_flag);
        // phase 2: the first stages go out with their weight rows only; h is not complete yet
        cur_vr = -1;
        uint32_t n2 = 0;
        int t2 = 0, k2 = 0;
        Tile ti2{};
        if (t2 < hi2)
            ti2 = tile2(t2);
        auto w_bytes2 = [&](int kc) { return min(CB2, rb2 - kc * CB2); };
        auto op_bytes2 = [&](int kc) { return min(CB2, Fpad * 2 - kc * CB2); };
        int pre = 0;
        for (; pre < S2 && t2 < hi2; ++pre) {
            issue(ti2, full2, empty2, S2, STAGE2, PITCH2, (size_t)k2 * CB2, w_bytes2(k2), op_bytes2(k2), 1, n2++);
            if (++k2 == nk2) {
                k2 = 0;
                if (++t2 < hi2)
                    ti2 = tile2(t2);
            }
        }
        // grid barrier: every CTA's consumers have written their part of h
        if (lane == 0) {
            const unsigned target = (unsigned)G;
            volatile unsigned *w = p.sync + p.group;
            if (*w < target && !*abort_flag) {
                const unsigned long long t0 = globaltimer_ns();
                while (*w < target) {
                    if (*abort_flag || globaltimer_ns() - t0 > kWaitLimitNs) {
                        *abort_flag = 1;
                        break;
                    }
                }
            }
            __threadfence();
            if (trace)
                trace[5] = globaltimer_ns();
        }
        __syncwarp();
        fence_proxy_async();
        {
            // the operand rows of the stages already under way: replay the tile sequence from the
            // start of phase 2 with a cache of its own, then restore the main sequence's cache
            const int keep_vr = cur_vr, keep_ntok = cur_ntok;
            const char *keep_base = lane_base;
            const size_t keep_step = lane_step;
            cur_vr = -1;
            int qt = 0, qk = 0;
            Tile qtile{};
            if (pre > 0)
                qtile = tile2(0);
            for (int i = 0; i < pre; ++i) {
                issue(qtile, full2, empty2, S2, STAGE2, PITCH2, (size_t)qk * CB2, 0, op_bytes2(qk), 2, (uint32_t)i);
                if (++qk == nk2) {
                    qk = 0;
                    if (++qt < hi2)
                        qtile = tile2(qt);
                }
            }
            cur_vr = keep_vr;
            cur_ntok = keep_ntok;
            lane_base = keep_base;
            lane_step = keep_step;
        }
        while (t2 < hi2) {
            issue(ti2, full2, empty2, S2, STAGE2, PITCH2, (size_t)k2 * CB2, w_bytes2(k2), op_bytes2(k2), 3, n2++);
            if (++k2 == nk2) {
                k2 = 0;
                if (++t2 < hi2)
                    ti2 = tile2(t2);
            }
        }
        if (*abort_flag && lane == 0) {
            // a wait ran out: give the copies still in flight a bounded time to land before this
            // CTA's shared memory goes away
            const unsigned long long t0 = globaltimer_ns();
            for (uint32_t m = n1 > (uint32_t)S1 ? n1 - S1 : 0u; m < n1; ++m)
                while (!mbar_try(full1 + 8 * (m % S1), (m / S1) & 1u) && globaltimer_ns() - t0 < kWaitLimitNs) {
                }
            for (uint32_t m = n2 > (uint32_t)S2 ? n2 - S2 : 0u; m < n2; ++m)
                while (!mbar_try(full2 + 8 * (m % S2), (m / S2) & 1u) && globaltimer_ns() - t0 < kWaitLimitNs) {
                }
            atomicExch(p.err, MELINOE_ERR_TIMEOUT);
        }
        return;
    }

    // ======================================================================= consumers
    const int g = lane >> 2, tig = lane & 3;
    int n_tiles = 0;       // tiles finished so far (selects the reduction buffer and the epilogue warp)
    float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};

    // this warp's share of one stage: some of the 16-column steps of the piece
    auto compute = [&](uint32_t full0, uint32_t empty0, int S, int STAGE, uint32_t a_off, uint32_t b_off, uint32_t n,
                       int bytes, int n_tok) {
        const uint32_t slot = n % S;
        mbar_wait(full0 + 8 * slot, (n / S) & 1u, abort_flag);
        const uint32_t base = ring_s + slot * STAGE;
        const int ks_total = (bytes + 31) >> 5;
        const int ks_lo = warp * ks_total / kConsumerWarps, ks_hi = (warp + 1) * ks_total / kConsumerWarps;
        const bool has_tok = g < n_tok;
        int ks = ks_lo;
        for (; ks + 1 < ks_hi; ks += 2) {
            uint32_t a0, a1, a2, a3, e0, e1, e2, e3;
            ldmatrix_x4(base + a_off + ks * 32, a0, a1, a2, a3);
            ldmatrix_x4(base + a_off + ks * 32 + 32, e0, e1, e2, e3);
            uint32_t b0 = 0, b1 = 0, f0 = 0, f1 = 0;
            if (has_tok) {
                b0 = lds32(base + b_off + ks * 32);
                b1 = lds32(base + b_off + ks * 32 + 16);
                f0 = lds32(base + b_off + ks * 32 + 32);
                f1 = lds32(base + b_off + ks * 32 + 48);
            }
            mma_16816(c0, a0, a1, a2, a3, b0, b1);
            mma_16816(c1, e0, e1, e2, e3, f0, f1);
        }
        if (ks < ks_hi) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(base + a_off + ks * 32, a0, a1, a2, a3);
            uint32_t b0 = 0, b1 = 0;
            if (has_tok) {
                b0 = lds32(base + b_off + ks * 32);
                b1 = lds32(base + b_off + ks * 32 + 16);
            }
            mma_16816(c0, a0, a1, a2, a3, b0, b1);
        }
        __syncwarp();
        if (lane == 0)
            mbar_arrive(empty0 + 8 * slot);
    };
    // end of a tile: the warps' partial accumulators meet in shared memory; one warp (they take
    // turns) ends up with the complete 16 x 8 tile in the usual accumulator layout
    auto reduce_tile = [&](float (&out)[4]) -> bool {
        float *buf = red + (n_tiles & 1) * (kConsumerWarps * 128);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            buf[warp * 128 + i * 32 + lane] = c0[i] + c1[i];
            c0[i] = c1[i] = 0.f;
        }
        consumer_bar();
        const bool mine = warp == (n_tiles & (kConsumerWarps - 1));
        if (mine) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float s = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w)
                    s += buf[w * 128 + i * 32 + lane];
                out[i] = s;
            }
        }
        ++n_tiles;
        return mine;
    };
    // what a consumer lane needs of a virtual request: its token count and the z rows of the two
    // token slots this lane's accumulators belong to
    struct VrInfo {
        int n_tok, pair0, pair1;
    };
    auto load_vr = [&](int vr) -> VrInfo {
        const VrRec *v = p.vrs + vr;
        VrInfo r;
        r.n_tok = v->n_tok;
        const int2 pr = *reinterpret_cast<const int2 *>(v->pair + tig * 2);
        r.pair0 = pr.x;
        r.pair1 = pr.y;
        return r;
    };

    // ---- phase 1: h = SiLU(W_g x) * (W_u x)
    {
        const uint32_t a_off = ((lane & 7) + ((lane >> 3) & 1) * 8) * PITCH1 + (lane >> 4) * 16;
        const uint32_t b_off = (16 + g) * PITCH1 + tig * 4;
        uint32_t n = 0;
        int cur_vr = -1;
        VrInfo v{};
        for (int t = lo1; t < hi1; ++t) {
            const int vr = vb + t / upe1, blk = t % upe1;
            if (vr != cur_vr) {
                v = load_vr(vr);
                cur_vr = vr;
            }
            for (int kc = 0; kc < nk1; ++kc) {
                compute(full1, empty1, S1, STAGE1, a_off, b_off, n, min(CB1, rb1 - kc * CB1), v.n_tok);
                if (trace && n == 0 && tid == 0)
                    trace[2] = globaltimer_ns();
                ++n;
            }
            float r[4];
            if (reduce_tile(r)) {
                // rows g and g + 8 of the tile are g_f and u_f for f = 8 * blk + g
                uint16_t *hrow = p.hbuf + ((size_t)vr * kTokPerVr) * Fpad + blk * 8 + g;
                if (tig * 2 < v.n_tok)
                    hrow[(size_t)(tig * 2) * Fpad] = bf16_rne(r[0] / (1.0f + __expf(-r[0])) * r[2]);
                if (tig * 2 + 1 < v.n_tok)
                    hrow[(size_t)(tig * 2 + 1) * Fpad] = bf16_rne(r[1] / (1.0f + __expf(-r[1])) * r[3]);
            }
        }
    }
    if (trace && tid == 0)
        trace[3] = globaltimer_ns();
    // this CTA's part of h is complete: tell the grid
    __threadfence();
    fence_proxy_async();       // h was written through the generic proxy, bulk copies will read it
    consumer_bar();
    if (tid == 0) {
        atomicAdd(p.sync + p.group, 1u);
        if (trace)
            trace[4] = globaltimer_ns();
    }

    // ---- phase 2: z = W_d h for this CTA's output rows
    {
        const uint32_t a_off = ((lane & 7) + ((lane >> 3) & 1) * 8) * PITCH2 + (lane >> 4) * 16;
        const uint32_t b_off = (16 + g) * PITCH2 + tig * 4;
        uint32_t n = 0;
        VrInfo v{}, nxt{};
        if (hi2 > 0)
            nxt = load_vr(vb);
        for (int t = 0; t < hi2; ++t) {
            const int blk = t % mt, r0 = r_lo + 16 * blk;
            if (blk == 0) {
                v = nxt;
                if (t + mt < hi2)
                    nxt = load_vr(vb + t / mt + 1);   // in flight while this request's tiles are computed
            }
            for (int kc = 0; kc < nk2; ++kc, ++n)
                compute(full2, empty2, S2, STAGE2, a_off, b_off, n, min(CB2, rb2 - kc * CB2), v.n_tok);
            float r[4];
            if (reduce_tile(r)) {
                const int row = r0 + g;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (tig * 2 + h < v.n_tok) {
                        float *zr = p.zbuf + (size_t)(h ? v.pair1 : v.pair0) * d + row;
                        if (row < r_hi)
                            zr[0] = r[h];
                        if (row + 8 < r_hi)
                            zr[8] = r[2 + h];
                    }
                }
            }
        }
    }
    if (trace && tid == 0)
        trace[6] = globaltimer_ns();
    // ---- combine (Eq. 2) of this CTA's rows, once the call's last group has produced its z
    if (final_group) {
        __threadfence_block();
        consumer_bar();
        const int n_pairs = p.T * p.k;
        const int nr = r_hi - r_lo;
        for (int i = tid; i < nr * p.T; i += kConsumerWarps * 32) {
            const int tk = i / nr, orow = r_lo + i % nr;
            float y = 0.f;
            for (int j = 0; j < p.k; ++j)
                y = fmaf(p.gate[tk * p.k + j], __ldcg(p.zbuf + (size_t)(tk * p.k + j) * d + orow), y);
            for (int sh = 0; sh < p.n_shared; ++sh)
                y += __ldcg(p.zbuf + (size_t)(n_pairs + sh * p.T + tk) * d + orow);
            p.out[(size_t)tk * d + orow] = bf16_rne(y);
        }
    }
    if (trace && tid == 0)
        trace[7] = globaltimer_ns();
    if (*abort_flag && tid == 0)
        atomicExch(p.err, MELINOE_ERR_TIMEOUT);
}

}  // namespace

cudaError_t ffn_stream_configure(int n_sms, size_t max_smem, FfnLaunchCfg *cfg)
{
    const size_t usable = max_smem - 1024;   // room for the kernel's static shared memory
    cudaError_t e = cudaFuncSetAttribute(ffn_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)usable);
    if (e != cudaSuccess)
        return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ffn_stream_kernel, kThreads, usable);
    if (e != cudaSuccess)
        return e;
    if (per_sm < 1)
        return cudaErrorInvalidConfiguration;
    cfg->grid = n_sms;          // one CTA per SM: all of them resident, which the grid barrier needs
    cfg->max_smem = usable;
    return cudaSuccess;
}

// Ring geometry for a call of T tokens on a d x F layer: the same shared memory is cut into
// stages of (16 + operand rows) row pieces twice, once for rows of 2*d bytes (gate/up phase)
// and once for rows of 2*F bytes (down phase).
cudaError_t ffn_stream_geometry(const FfnLaunchCfg &cfg, int d, int F, int T, FfnGeometry *geo)
{
    auto chunk_of = [](int row_bytes) {
        const int c = row_bytes < kMaxChunk ? row_bytes : kMaxChunk;
        return (c + 127) / 128 * 128;
    };
    geo->n_op_rows = T < kTokPerVr ? T : kTokPerVr;
    geo->chunk_bytes = chunk_of(2 * d);
    geo->pitch = geo->chunk_bytes + 16;
    geo->chunk_bytes2 = chunk_of(2 * F);
    geo->pitch2 = geo->chunk_bytes2 + 16;
    const size_t rows = 16 + geo->n_op_rows;
    const size_t stage1 = rows * geo->pitch, stage2 = rows * geo->pitch2;
    const size_t fixed = 2 * kConsumerWarps * 128 * sizeof(float) + 4 * kMaxStages * 8 + 128;
    const size_t big = stage1 > stage2 ? stage1 : stage2;
    if (cfg.max_smem < fixed + 2 * big)
        return cudaErrorInvalidConfiguration;
    const size_t avail = (cfg.max_smem - fixed) / 128 * 128;
    size_t s1 = avail / stage1, s2 = avail / stage2;
    if (s1 > (size_t)kMaxStages)
        s1 = kMaxStages;
    if (s2 > (size_t)kMaxStages)
        s2 = kMaxStages;
    geo->n_stages = (int)s1;
    geo->n_stages2 = (int)s2;
    size_t ring = s1 * stage1 > s2 * stage2 ? s1 * stage1 : s2 * stage2;
    ring = (ring + 127) / 128 * 128;
    geo->ring_bytes = ring;
    geo->smem_bytes = ring + fixed;
    return cudaSuccess;
}

cudaError_t launch_ffn_stream(cudaStream_t stream, const FfnLaunchCfg &cfg, const FfnGeometry &geo, const FfnParams &p)
{
    FfnParams q = p;
    FfnGeometry gq = geo;
    void *args[] = {&q, &gq};
    cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(ffn_stream_kernel), dim3(cfg.grid),
                                                dim3(kThreads), args, geo.smem_bytes, stream);
    count_launch();
    return e;
}

}  // namespace melinoe
