// Streaming SwiGLU expert FFN (Eq. 3) with the gate-weighted combine (Eq. 2) fused in, for
// calls with few tokens per expert (decode).  The work is reading every needed expert once
// from HBM, so the kernel is built around keeping the memory system full: measured on B200,
// bulk copies of whole 4 KB rows stream at the full HBM rate while 256-byte pieces reach
// little more than half of it, so the unit of transfer is a whole row (or a 4 KB piece of a
// longer one).
//
// One cooperative launch per compute group, one CTA per SM: eight consumer warps, three producer
// warps and two warps for the grid barrier.  A "virtual request" is one expert with up to 8 of its tokens.
//
//   phase 1  tile = up to 8 rows of W_g plus the same rows of W_u of one virtual request.
//            D[16 x 8] = [W_g rows; W_u rows] (16 x d) * x^T (d x 8 tokens) on mma.sync
//            (bf16 in, fp32 accumulate); the eight warps split the columns of a stage and
//            their partial sums meet in shared memory once per tile.  In the accumulator
//            layout a thread holds g_f and u_f of the same f and the same two tokens, so
//            h = SiLU(g) * u is thread-local; h goes to global memory as bf16.
//   barrier  grid-wide, and off everybody's critical path.  While the SM streams, any round trip
//            to global memory (a fence after the h stores, a poll of a device counter) takes
//            microseconds, so neither the consumers nor the producers ever make one: the consumer
//            warps arrive on a shared-memory barrier when their part of h is stored and go on; a
//            warp of its own does the device-wide release (fence + atomic) for them, another polls the
//            device counter and raises a shared-memory flag the producers look at.  The requests
//            go through the kernel in two halves, so each half's barrier latency is covered by the
//            other half's streaming.  The W_d rows do not wait for the barrier at all: they are
//            requested the moment a ring slot comes free; only the h rows wait for it.
//   phase 2  every CTA owns a contiguous range of the d_model output rows (d/G of them, so the
//            split is even to within one row) for ALL virtual requests of the launch.  Tile =
//            up to 16 of those W_d rows of one virtual request; warp w computes rows w and w + 8
//            as plain fp32 dot products over d_ff against the h rows (the arithmetic is a few
//            hundred FMAs per lane and tile), complete sums, so z needs no reduction across
//            warps or CTAs; it goes to z[pair][d] in fp32.
//   combine  in the call's last compute group every CTA, having finished its rows, sums
//            gate * z over the ranks in rank order (plus shared experts) for those rows and
//            writes them as bf16: it reads only what itself (or an earlier launch) wrote, so
//            no device-wide synchronisation is involved.  The result does not depend on how the
//            experts were split over groups.
//
// A stage of the shared-memory ring holds one piece (at most 4 KB) of each of the tile's 16
// weight rows plus the matching piece of up to 8 operand rows (hidden rows in phase 1, h rows
// in phase 2), each fetched by its own cp.async.bulk (one producer lane per row; the producer
// warps share out the ring slots) completing on the stage's mbarrier.  Rows sit at a pitch of 16 bytes more than a multiple of 128, which
// makes the ldmatrix reads and the operand-fragment reads bank-conflict free.
//
// Every wait is bounded: when an mbarrier or the grid barrier does not complete in time the
// warp raises the CTA's abort flag, later waits fall through, the kernel ends normally and the
// error word tells the host.
#include <cstdlib>
#include <type_traits>

#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kProducerWarps = 3;                    // a warp needs ~0.6 us to get one stage's copies out
constexpr int kSyncWarp = kConsumerWarps + kProducerWarps;   // the warp that runs the grid barrier
constexpr int kThreads = (kConsumerWarps + kProducerWarps + 2) * 32;
constexpr int kMaxStages = 8;
constexpr int kMaxSub = 16;                          // sub-stages of the down phase, over the whole ring
constexpr int kMaxChunk = 4096;                      // bytes of one row piece
constexpr int kVrShared = 72;                        // virtual-request records kept in shared memory
// Bound of every wait, in SM clock cycles (about 2 s).  Waits are timed with the SM's cycle
// counter: reading the device-wide nanosecond timer costs about 0.6 us each time, which would
// quantise every wait that does not succeed at once.
constexpr long long kWaitLimitCycles = 4000000000ll;

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
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity))
                return true;
        if (*abort_flag)
            return false;
        if (clock64() - t0 > kWaitLimitCycles) {
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

__global__ void __launch_bounds__(kThreads, 1) ffn_stream_kernel(FfnParams p, FfnGeometry geo)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_abort;
    __shared__ int s_passed[2];                 // half's h is complete on every CTA
    __shared__ int s_slot_free[kMaxStages];     // the gate/up phase has let go of the ring slot
    __shared__ __align__(8) uint64_t s_harr[2]; // consumer warps that have stored their part of the half's h
    __shared__ VrRec s_vrs[kVrShared];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int d = p.d, F = p.F, Fpad = p.Fpad;
    const DevPlan *plan = p.plan;
    const int G = (int)gridDim.x;
    const int NOP = geo.n_op_rows;
    (void)NOP;
    const int S1 = geo.n_stages, PITCH1 = geo.pitch, CB1 = geo.chunk_bytes, STAGE1 = geo.stage_bytes;
    // down phase: rows of 2*F bytes in pieces of at most CB2, laid out like the gate/up stages (one
    // piece of every weight row of the tile, the h rows behind them at row ROWS2, padded pitch).  A
    // down stage is often much smaller than a gate/up stage (short W_d rows, fewer than 16 rows per
    // CTA), so a ring slot is cut into NS2 sub-stages for the down phase: more tiles in flight
    // where each tile is small.
    const int CB2 = geo.chunk_bytes2, NS2 = geo.sub2, SUB2 = geo.sub_bytes2, PITCH2 = geo.pitch2, ROWS2 = geo.rows2;

    // optional timeline: 8 device-clock stamps per CTA (see melinoe_moe_set_trace)
    unsigned long long *trace = p.trace ? p.trace + (size_t)blockIdx.x * 8 : nullptr;
    if (trace && tid == 0)
        trace[0] = globaltimer_ns();

    // ring | reduction buffers | barriers (phase 1 full/empty, phase 2 full/empty)
    unsigned char *ring = smem;
    float *red = reinterpret_cast<float *>(smem + geo.ring_bytes);              // [2][8 warps][4][32]
    uint64_t *bars = reinterpret_cast<uint64_t *>(red + 2 * kConsumerWarps * 128);
    const uint32_t ring_s = smem_u32(ring);
    const uint32_t full1 = smem_u32(bars), empty1 = full1 + 8 * kMaxStages;
    const uint32_t full2 = empty1 + 8 * kMaxStages, empty2 = full2 + 8 * kMaxSub;
    volatile int *abort_flag = &s_abort;

    const uint32_t harr = smem_u32(s_harr);
    if (tid == 0) {
        s_abort = 0;
        s_passed[0] = s_passed[1] = 0;
        for (int i = 0; i < kMaxStages; ++i)
            s_slot_free[i] = 0;
        for (int i = 0; i < 2; ++i)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(harr + 8 * i), "r"(kConsumerWarps));
        for (int i = 0; i < kMaxSub; ++i) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full2 + 8 * i), "r"(1));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty2 + 8 * i), "r"(2 * F > CB2 ? kConsumerWarps : 1));
        }
        for (int i = 0; i < kMaxStages; ++i) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full1 + 8 * i), "r"(1));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty1 + 8 * i), "r"(kConsumerWarps));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Everything above touches nothing an earlier kernel wrote.  The launch may have been made with
    // programmatic stream serialisation, in which case this CTA can be running before the kernel
    // ahead of it in the stream (the planner) has finished: wait for it here (returns at once in an
    // ordinary launch), then let the kernel behind this one be scheduled early in the same way.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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

    // the launch's virtual-request records: from shared memory when they fit (always in decode),
    // so that nobody's critical path holds a dependent global load per tile
    const VrRec *vrs = p.vrs + vb;
    if (nv <= kVrShared) {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.vrs + vb);
        uint4 *dst = reinterpret_cast<uint4 *>(s_vrs);
        for (int i = tid; i < nv * (int)(sizeof(VrRec) / 16); i += kThreads)
            dst[i] = src[i];
        vrs = s_vrs;
    }
    __syncthreads();
    if (trace && tid == 0)
        trace[1] = globaltimer_ns();

    // ---- work of this CTA.  The launch's virtual requests are cut into two halves (one when there
    // is a single request) that go through the kernel one behind the other:
    //     gate/up(A)  gate/up(B)  down(A)  down(B)
    // so that the grid-wide wait for h of half A is covered by the streaming of half B's W_g/W_u
    // rows, and the wait for half B by half A's W_d rows.
    // gate/up: rows f of W_g and W_u of the half's requests, numbered request-major, are split
    // evenly over the CTAs at single-row granularity; a tile is up to 8 consecutive f of one
    // request (g rows in tile rows 0..7, u rows in 8..15).
    // down: output rows [r_lo, r_hi) of every request, in tiles of up to 16 rows.
    const int rb1 = 2 * d, rb2 = 2 * F;                       // row bytes
    const int nk1 = (rb1 + CB1 - 1) / CB1, nk2 = (rb2 + CB2 - 1) / CB2;
    const int n_half = nv >= 2 ? 2 : 1;
    // Equal parts measured best (OLMoE shape, 8 requests: 5 + 3, 4 + 4 and 3 + 5 within 0.2 us of one
    // another per launch, 6 + 2 one microsecond slower, 7 + 1 two and a half).
    const int nvA = n_half == 2 ? nv - nv / 2 : nv;           // requests in the first part
    // f-row ranges, relative to the half's first request (scalars, not arrays: an array indexed by
    // the half would live in local memory)
    const long long rowsA = (long long)nvA * F, rowsB = (long long)(nv - nvA) * F;
    const int q_loA = (int)(blockIdx.x * rowsA / G), q_hiA = (int)((blockIdx.x + 1) * rowsA / G);
    const int q_loB = (int)(blockIdx.x * rowsB / G), q_hiB = (int)((blockIdx.x + 1) * rowsB / G);
    const int r_lo = (int)((long long)blockIdx.x * d / G), r_hi = (int)((long long)(blockIdx.x + 1) * d / G);
    const int mt = (r_hi - r_lo + 15) / 16;
    const int hi2 = nv * mt, hi2A = nvA * mt;                 // down tiles: request-major, half A first
    unsigned *sync_word = p.sync + 2 * p.group;               // [half]

    // Down stage j (counted from 0 within the phase) lives in ring slot (n1 + j / NS2) mod S1, sub-stage
    // j mod NS2: the slots are taken in the order in which the gate/up phase lets go of them.  A
    // cursor walks that sequence without divisions.
    struct Down {
        uint32_t slot, sub, use, r;
    };
    auto down_first = [&](uint32_t n1_) -> Down { return Down{n1_ % (uint32_t)S1, 0u, 0u, 0u}; };
    auto down_next = [&](Down &x) {
        if (++x.sub == (uint32_t)NS2) {
            x.sub = 0;
            if (++x.slot == (uint32_t)S1)
                x.slot = 0;
        }
        if (++x.r == (uint32_t)(S1 * NS2)) {
            x.r = 0;
            ++x.use;
        }
    };
    auto down_bar = [&](const Down &x) -> uint32_t { return x.slot * NS2 + x.sub; };
    auto down_off = [&](const Down &x) -> uint32_t { return x.slot * STAGE1 + x.sub * SUB2; };

    if (warp == kSyncWarp) {
        // =================================================================== grid barrier, arriving
        // One lane: when the eight consumer warps have stored their part of a half's h, publish it
        // device-wide (fence, then count this CTA in).  The fence takes microseconds while the SM
        // streams, which is why no warp with other work makes it.
        if (lane != 0)
            return;
        for (int half = 0; half < n_half; ++half) {
            if (!mbar_wait(harr + 8 * half, 0, abort_flag))
                break;
            __threadfence();
            fence_proxy_async();   // h was written through the generic proxy, bulk copies will read it
            atomicAdd(sync_word + half, 1u);
            if (trace && half == n_half - 1)
                trace[4] = globaltimer_ns();
        }
        return;
    }
    if (warp == kSyncWarp + 1) {
        // =================================================================== grid barrier, watching
        // One lane: watch the halves' counters (in order: the first half is complete everywhere
        // before the second is) and tell the producers through a shared-memory flag.
        if (lane != 0)
            return;
        const long long t0 = clock64();
        for (int half = 0; half < n_half; ++half) {
            for (;;) {
                unsigned v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(sync_word + half) : "memory");
                if (v >= (unsigned)G)
                    break;
                if (*abort_flag)
                    return;
                if (clock64() - t0 > kWaitLimitCycles) {
                    *abort_flag = 1;
                    return;
                }
                __nanosleep(100);
            }
            fence_proxy_async();
            __threadfence_block();
            *reinterpret_cast<volatile int *>(&s_passed[half]) = 1;
            if (trace && half == n_half - 1)
                trace[5] = globaltimer_ns();
        }
        return;
    }

    if (warp >= kConsumerWarps && warp < kSyncWarp) {
        // =================================================================== producers
        // The producer warps walk the same stage sequence and share the stages out (a warp is busy
        // for ~0.6 us with one bulk-copy instruction, however few lanes take part, so the stages
        // of a 28 KB-per-stage phase would otherwise leave faster than one warp can issue them).
        // A ring slot always belongs to the same warp (slot s to warp s mod 3), so every wait on a
        // slot's "empty" barrier is made by the one warp that has followed all its earlier phases.
        // Lanes 0..15 fetch the tile's weight rows, lanes 16..23 the operand rows.
        const int pw = warp - kConsumerWarps;
        const bool is_w = lane < 16;
        const int my_row = is_w ? lane : lane - 16;                        // tile row, or token slot
        const int dst_row2 = is_w ? lane : ROWS2 + my_row;             // row of a down sub-stage
        const bool lane_used = lane < 24;
        bool dead = false;
        // One stage of either phase.  src: this lane's source row or null.  parts bit 0: arm the
        // barrier and fetch the weight rows (the caller has made sure the slot is free); bit 1:
        // operand rows.
        auto issue = [&](const char *src, uint32_t bar, uint32_t stage_off, int PITCH, int dst_row, size_t src_off,
                         int wbytes, int obytes, int parts) {
            const bool active = lane_used && src != nullptr;
            if (parts & 1) {
                const unsigned mw = __ballot_sync(0xffffffffu, active && is_w);
                const unsigned mo = __ballot_sync(0xffffffffu, active && !is_w);
                if (lane == 0)
                    mbar_expect(bar, (uint32_t)__popc(mw) * wbytes + (uint32_t)__popc(mo) * obytes);
                __syncwarp();
            }
            if (active && !dead && (is_w ? (parts & 1) : (parts & 2)))
                bulk_g2s(ring_s + stage_off + dst_row * PITCH, src + src_off, (uint32_t)(is_w ? wbytes : obytes), bar);
        };
        // ---- gate/up: lanes 0..7 W_g rows, 8..15 W_u rows, 16..23 hidden rows of the request's tokens
        uint32_t n1 = 0;
        for (int half = 0; half < n_half; ++half) {
            const int v0 = vb + (half ? nvA : 0);
            const int q_end = half ? q_hiB : q_hiA;
            int q = half ? q_loB : q_loA;
            while (q < q_end) {
                const int vr = v0 + q / F, f0 = q % F;
                const int m = min(min(8, F - f0), q_end - q);
                const VrRec *v = vrs + (vr - vb);
                const char *src = nullptr;
                if (lane_used) {
                    if (is_w) {
                        if ((my_row & 7) < m)
                            src = v->blob + (size_t)((my_row < 8 ? 0 : F) + f0 + (my_row & 7)) * rb1;
                    } else if (my_row < v->n_tok) {
                        src = reinterpret_cast<const char *>(p.x) + (size_t)v->tok[my_row] * rb1;
                    }
                }
                for (int kc = 0; kc < nk1; ++kc, ++n1) {
                    if ((int)((n1 % S1) % kProducerWarps) != pw)
                        continue;
                    if (n1 >= (uint32_t)S1 && !dead)
                        dead = !mbar_wait(empty1 + 8 * (n1 % S1), ((n1 / S1) - 1u) & 1u, abort_flag);
                    const int b = min(CB1, rb1 - kc * CB1);
                    issue(src, full1 + 8 * (n1 % S1), (n1 % S1) * STAGE1, PITCH1, lane, (size_t)kc * CB1, b, b, 3);
                }
                q += m;
            }
        }
        // ---- down: lanes 0..15 W_d rows, 16..23 rows of h.  Two cursors walk the same stage
        // sequence: the weight rows run ahead as far as the ring allows, the h rows of a stage
        // follow once the grid has finished the h of the stage's half.  Sub-stage (slot, sub) belongs
        // to warp (slot + sub) mod 3 throughout, so the two tiles that share a slot are requested by
        // two warps side by side (a warp is busy for most of a microsecond with one tile's copies).
        struct Cursor {
            int t, k, blk, v, base_v;
            const char *base;
        };
        auto tile_of = [&](Cursor &c) -> const char * {
            if (c.v != c.base_v) {
                const VrRec *v = vrs + c.v;
                c.base_v = c.v;
                c.base = nullptr;
                if (lane_used) {
                    if (is_w)
                        c.base = v->blob + (size_t)2 * F * rb1 + (size_t)(r_lo + my_row) * rb2;
                    else if (my_row < v->n_tok)
                        c.base = reinterpret_cast<const char *>(p.hbuf) + ((size_t)(vb + c.v) * kTokPerVr + my_row) * Fpad * 2;
                }
            }
            if (!is_w)
                return c.base;
            return (c.base && r_lo + 16 * c.blk + my_row < r_hi) ? c.base + (size_t)c.blk * 16 * rb2 : nullptr;
        };
        auto advance = [&](Cursor &c) {
            if (++c.k == nk2) {
                c.k = 0;
                ++c.t;
                if (++c.blk == mt) {
                    c.blk = 0;
                    ++c.v;
                }
            }
        };
        auto piece2 = [&](int kc) { return min(CB2, rb2 - kc * CB2); };    // one row's piece
        const uint32_t N2 = (uint32_t)hi2 * nk2;
        Cursor wc{0, 0, 0, 0, -1, nullptr}, oc{0, 0, 0, 0, -1, nullptr};
        Down wd = down_first(n1), od = wd;
        uint32_t wn = 0, on = 0;
        bool passedA = false, passedB = false;
        long long t_idle = 0;
        while (on < N2 && !dead) {
            bool progress = false;
            // weight rows of as many stages as there are free sub-stages
            while (wn < N2) {
                const uint32_t bar = down_bar(wd);
                if ((int)((wd.slot + wd.sub) % kProducerWarps) == pw) {
                    // free when its previous down-phase use has been consumed, or, on first use, when the
                    // gate/up phase has let go of the slot for good.  Only the warp that served the slot
                    // in the gate/up phase (it owns sub-stage 0) may read that off the slot's "empty"
                    // barrier; it tells the owners of the slot's other sub-stages through a flag.
                    int ok = 1;
                    if (lane == 0) {
                        if (wd.use > 0) {
                            ok = mbar_try(empty2 + 8 * bar, (wd.use - 1u) & 1u);
                        } else if (n1 > wd.slot) {
                            if (wd.sub == 0) {
                                const uint32_t m_last = n1 - 1u - ((n1 - 1u - wd.slot) % S1);
                                ok = mbar_try(empty1 + 8 * wd.slot, (m_last / S1) & 1u);
                                if (ok) {
                                    __threadfence_block();
                                    *reinterpret_cast<volatile int *>(&s_slot_free[wd.slot]) = 1;
                                }
                            } else {
                                ok = *reinterpret_cast<volatile int *>(&s_slot_free[wd.slot]);
                                if (ok)
                                    __threadfence_block();
                            }
                        }
                    }
                    if (!__shfl_sync(0xffffffffu, ok, 0))
                        break;
                    const char *src = tile_of(wc);
                    issue(src, full2 + 8 * bar, down_off(wd), PITCH2, dst_row2, (size_t)wc.k * CB2, piece2(wc.k),
                          piece2(wc.k), 1);
                }
                advance(wc);
                down_next(wd);
                ++wn;
                progress = true;
            }
            // h rows of the next stages, once their half of h is complete everywhere
            if (on < wn) {
                const int half = oc.t < hi2A ? 0 : 1;
                if (!(half ? passedB : passedA)) {
                    int ok = 0;
                    if (lane == 0)
                        ok = *reinterpret_cast<volatile int *>(&s_passed[half]);
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (ok) {
                        // the barrier warp has made the generic-proxy writes of h visible to the bulk
                        // copies before it raised the flag
                        __threadfence_block();
                        if (half)
                            passedB = true;
                        else
                            passedA = true;
                    }
                }
                while (on < wn && (oc.t < hi2A ? passedA : passedB)) {
                    const uint32_t bar = down_bar(od);
                    if ((int)((od.slot + od.sub) % kProducerWarps) == pw) {
                        const char *src = tile_of(oc);
                        issue(src, full2 + 8 * bar, down_off(od), PITCH2, dst_row2, (size_t)oc.k * CB2, 0, piece2(oc.k), 2);
                    }
                    advance(oc);
                    down_next(od);
                    ++on;
                    progress = true;
                }
            }
            if (progress) {
                t_idle = 0;
            } else {
                const long long now = clock64();
                if (t_idle == 0)
                    t_idle = now;
                int give_up = (now - t_idle > kWaitLimitCycles) || *abort_flag;
                give_up = __shfl_sync(0xffffffffu, give_up, 0);
                if (give_up) {
                    *abort_flag = 1;
                    dead = true;
                }
                // a warp that polls without pause takes issue slots and shared-memory pipeline
                // cycles from the consumer warps
                __nanosleep(100);
            }
        }
        const uint32_t n2 = on;
        if (*abort_flag && lane == 0 && pw == 0) {
            // a wait ran out: give the copies still in flight a bounded time to land before this
            // CTA's shared memory goes away
            const long long t0 = clock64();
            const uint32_t in_ring = (uint32_t)(S1 * NS2);
            Down x = down_first(n1);
            for (uint32_t j = 0; j < n2; ++j, down_next(x)) {
                if (j + in_ring < n2)
                    continue;
                while (!mbar_try(full2 + 8 * down_bar(x), x.use & 1u) && clock64() - t0 < kWaitLimitCycles) {
                }
            }
            atomicExch(p.err, MELINOE_ERR_TIMEOUT);
        }
        return;
    }

    // ======================================================================= consumers
    const int g = lane >> 2, tig = lane & 3;
    int n_tiles = 0;       // tiles finished so far (selects the reduction buffer and the epilogue warp)
    // four accumulator chains: an mma waits some 30 cycles for the one it accumulates onto
    float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f}, c3[4] = {0.f, 0.f, 0.f, 0.f};

    // this warp's share of one stage: some of the 16-column steps of the piece.  Weights in tile
    // rows 0..15, the operand rows (hidden or h) of the request's tokens behind them.
    // 16-column steps [ks, ks_hi) of a stage at shared address base: weights in stage rows 0..15 (a_off
    // is this lane's ldmatrix row), operand rows behind them (b_off is this lane's fragment row)
    auto mma_steps = [&](uint32_t base, uint32_t a_off, uint32_t b_off, int ks, int ks_hi, bool has_tok) {
        for (; ks + 3 < ks_hi; ks += 4) {
            uint32_t a[4][4], b[4][2];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                ldmatrix_x4(base + a_off + (ks + i) * 32, a[i][0], a[i][1], a[i][2], a[i][3]);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                b[i][0] = has_tok ? lds32(base + b_off + (ks + i) * 32) : 0u;
                b[i][1] = has_tok ? lds32(base + b_off + (ks + i) * 32 + 16) : 0u;
            }
            mma_16816(c0, a[0][0], a[0][1], a[0][2], a[0][3], b[0][0], b[0][1]);
            mma_16816(c1, a[1][0], a[1][1], a[1][2], a[1][3], b[1][0], b[1][1]);
            mma_16816(c2, a[2][0], a[2][1], a[2][2], a[2][3], b[2][0], b[2][1]);
            mma_16816(c3, a[3][0], a[3][1], a[3][2], a[3][3], b[3][0], b[3][1]);
        }
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
    };
    // gate/up: this warp's share of one stage, an eighth of the piece's 16-column steps
    auto compute = [&](uint32_t full0, uint32_t empty0, int S, int STAGE, uint32_t a_off, uint32_t b_off, uint32_t n,
                       int bytes, int n_tok) {
        const uint32_t slot = n % S;
        mbar_wait(full0 + 8 * slot, (n / S) & 1u, abort_flag);
        const int ks_total = (bytes + 31) >> 5;
        mma_steps(ring_s + slot * STAGE, a_off, b_off, warp * ks_total / kConsumerWarps,
                  (warp + 1) * ks_total / kConsumerWarps, g < n_tok);
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
            buf[warp * 128 + i * 32 + lane] = (c0[i] + c1[i]) + (c2[i] + c3[i]);
            c0[i] = c1[i] = c2[i] = c3[i] = 0.f;
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
        const VrRec *v = vrs + (vr - vb);
        VrInfo r;
        r.n_tok = v->n_tok;
        const int2 pr = *reinterpret_cast<const int2 *>(v->pair + tig * 2);
        r.pair0 = pr.x;
        r.pair1 = pr.y;
        return r;
    };

    uint32_t n = 0;        // stages consumed so far, over both phases
    // ---- gate/up: h = SiLU(W_g x) * (W_u x), half by half
    {
        const uint32_t a_off = ((lane & 7) + ((lane >> 3) & 1) * 8) * PITCH1 + (lane >> 4) * 16;
        const uint32_t b_off = (16 + g) * PITCH1 + tig * 4;
        for (int half = 0; half < n_half; ++half) {
            const int v0 = vb + (half ? nvA : 0);
            int cur_vr = -1;
            VrInfo v{};
            const int q_end = half ? q_hiB : q_hiA;
            int q = half ? q_loB : q_loA;
            while (q < q_end) {
                const int vr = v0 + q / F, f0 = q % F;
                const int m = min(min(8, F - f0), q_end - q);
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
                if (reduce_tile(r) && g < m) {
                    // rows g and g + 8 of the tile are g_f and u_f for f = f0 + g
                    uint16_t *hrow = p.hbuf + ((size_t)vr * kTokPerVr) * Fpad + f0 + g;
                    if (tig * 2 < v.n_tok)
                        hrow[(size_t)(tig * 2) * Fpad] = bf16_rne(r[0] / (1.0f + __expf(-r[0])) * r[2]);
                    if (tig * 2 + 1 < v.n_tok)
                        hrow[(size_t)(tig * 2 + 1) * Fpad] = bf16_rne(r[1] / (1.0f + __expf(-r[1])) * r[3]);
                }
                q += m;
            }
            if (trace && tid == 0 && half == n_half - 1)
                trace[3] = globaltimer_ns();
            // this warp's part of the half's h is stored: the barrier warp takes it from here
            __syncwarp();
            if (lane == 0)
                mbar_arrive(harr + 8 * half);
        }
    }

    // ---- down: z = W_d h for this CTA's output rows, D[16 rows x 8 tokens] per tile.
    // Short rows (a tile is one stage): a tile belongs to ONE warp, tile j to warp j mod 8, so
    // nothing is reduced across warps and the tiles in the ring are worked on side by side.  (Such
    // a tile costs its warp a few hundred instructions; shared out over eight warps it would cost
    // each of them mostly the latency of seeing the barrier and of meeting the others.)
    // Long rows (a tile is several stages, each a 64 KB piece): one warp would need longer for a
    // stage than the stage takes to arrive, so the eight warps share every stage as in the gate/up
    // phase and meet in shared memory once per tile.
    // Either way every warp waits for every stage in order: a warp that waited for phase k + 1 of a
    // barrier whose phase k it has not seen could be let through by the parity test.
    {
        Down dc = down_first(n);     // the down phase takes the slots in ring order after the gate/up stages
        bool first = true;
        const bool shared2 = nk2 > 1;
        const uint32_t a_off = ((lane & 7) + ((lane >> 3) & 1) * 8) * PITCH2 + (lane >> 4) * 16;
        const uint32_t b_off = (ROWS2 + g) * PITCH2 + tig * 4;
        int tile_no = 0;
        for (int v = 0; v < nv; ++v) {
            const VrInfo vi = load_vr(vb + v);
            for (int blk = 0; blk < mt; ++blk, ++tile_no) {
                const bool mine = shared2 || (tile_no & (kConsumerWarps - 1)) == warp;
                for (int kc = 0; kc < nk2; ++kc) {
                    mbar_wait(full2 + 8 * down_bar(dc), dc.use & 1u, abort_flag);
                    if (trace && first && tid == 0)
                        trace[2] = globaltimer_ns();
                    first = false;
                    if (mine) {
                        const uint32_t base = ring_s + down_off(dc);
                        const int bytes = min(CB2, rb2 - kc * CB2);
                        const bool has_tok = g < vi.n_tok;
                        const int ks_total = bytes >> 5;
                        if (shared2)
                            mma_steps(base, a_off, b_off, warp * ks_total / kConsumerWarps,
                                      (warp + 1) * ks_total / kConsumerWarps, has_tok);
                        else
                            mma_steps(base, a_off, b_off, 0, ks_total, has_tok);
                        if ((bytes & 16) && (!shared2 || warp == kConsumerWarps - 1)) {
                            // the row ends on half a step: columns 8..15 of both operands count as zero
                            const int ks = bytes >> 5;
                            uint32_t a0, a1, a2, a3;
                            ldmatrix_x4(base + a_off + ks * 32, a0, a1, a2, a3);
                            const uint32_t b0 = has_tok ? lds32(base + b_off + ks * 32) : 0u;
                            mma_16816(c1, a0, a1, 0u, 0u, b0, 0u);
                        }
                        __syncwarp();
                        if (lane == 0)
                            mbar_arrive(empty2 + 8 * down_bar(dc));
                    }
                    down_next(dc);
                }
                float r4[4];
                bool store = mine;
                if (shared2) {
                    store = reduce_tile(r4);
                } else if (mine) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        r4[i] = (c0[i] + c1[i]) + (c2[i] + c3[i]);
                        c0[i] = c1[i] = c2[i] = c3[i] = 0.f;
                    }
                }
                if (store) {
                    // rows g and g + 8 of the tile, tokens 2 tig and 2 tig + 1 of the request
                    const int n_rows = min(16, r_hi - r_lo - 16 * blk);
                    float *z0 = p.zbuf + r_lo + 16 * blk + g;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float val = r4[i];
                        const int tok = tig * 2 + (i & 1), row = g + (i >> 1) * 8;
                        if (tok < vi.n_tok && row < n_rows)
                            z0[(size_t)((i & 1) ? vi.pair1 : vi.pair0) * d + (i >> 1) * 8] = val;
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
    const size_t usable = max_smem - 8192;   // room for the kernel's static shared memory
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
    cfg->pdl = pdl_enabled();
    return cudaSuccess;
}

// Ring geometry for a call of T tokens on a d x F layer: stages of (16 + operand rows) row
// pieces, sized for the longer of the two phases' pieces; each phase lays its rows out at its
// own pitch inside a stage.
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
    const size_t stage = rows * (geo->pitch > geo->pitch2 ? geo->pitch : geo->pitch2);
    const size_t fixed = 2 * kConsumerWarps * 128 * sizeof(float) + 2 * kMaxStages * 8 + 2 * kMaxSub * 8 + 128;
    if (cfg.max_smem < fixed + 2 * stage)
        return cudaErrorInvalidConfiguration;
    const size_t avail = (cfg.max_smem - fixed) / 128 * 128;
    size_t n = avail / stage;
    if (n > (size_t)kMaxStages)
        n = kMaxStages;
    geo->n_stages = (int)n;
    geo->stage_bytes = (int)stage;
    // down phase: a CTA has at most ceil(d / grid) output rows, so a tile may have fewer than 16
    // weight rows; the h rows follow them, and the sub-stage is at least 16 rows long because the
    // tensor-core loads always read 16 (what lies in rows the tile does not have only reaches
    // accumulator rows that are never stored).  As many sub-stages per slot as fit.
    const int rows_cta = (d + cfg.grid - 1) / cfg.grid;
    geo->rows2 = rows_cta < 16 ? rows_cta : 16;
    const size_t sub_rows = (size_t)(geo->rows2 + geo->n_op_rows) > 16 ? (size_t)(geo->rows2 + geo->n_op_rows) : 16;
    const size_t sub = (sub_rows * geo->pitch2 + 127) / 128 * 128;
    size_t ns2 = stage / sub;
    if (ns2 < 1)
        ns2 = 1;
    while (ns2 * n > (size_t)kMaxSub)
        --ns2;
    geo->sub2 = (int)ns2;
    geo->sub_bytes2 = (int)sub;
    geo->ring_bytes = (n * stage + 127) / 128 * 128;
    geo->smem_bytes = geo->ring_bytes + fixed;
    return cudaSuccess;
}

cudaError_t launch_ffn_stream(cudaStream_t stream, const FfnLaunchCfg &cfg, const FfnGeometry &geo, const FfnParams &p)
{
    // cooperative (the grid barrier needs every CTA resident) and with programmatic stream
    // serialisation (the CTAs may be scheduled, and set up their barriers, while the kernel ahead in
    // the stream is still draining; the kernel waits for it before it reads the plan)
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(cfg.grid);
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = geo.smem_bytes;
    lc.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = cfg.pdl ? 2 : 1;
    const cudaError_t e = cudaLaunchKernelEx(&lc, ffn_stream_kernel, p, geo);
    count_launch();
    return e;
}

}  // namespace melinoe
