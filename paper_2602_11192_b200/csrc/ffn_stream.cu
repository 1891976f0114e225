// Streaming SwiGLU expert FFN (Eq. 3) with the gate-weighted combine (Eq. 2) fused in, for
// calls with few tokens per expert (decode).  The work is reading every needed expert once
// from HBM, so the kernel is built around keeping the memory system full: measured on B200,
// bulk copies of whole 4 KB rows stream at the full HBM rate while 256-byte pieces reach
// little more than half of it, so the unit of transfer is a whole row (or a 4 KB piece of a
// longer one).
//
// One cooperative launch per compute group, one CTA per SM: four producer warps and eight
// consumer warps.  A "virtual request" is one expert with up to 8 of its tokens.
//
//   phase 1  tile = up to 8 rows of W_g plus the same rows of W_u of one virtual request.
//            D[16 x 8] = [W_g rows; W_u rows] (16 x d) * x^T (d x 8 tokens) on mma.sync
//            (bf16 in, fp32 accumulate); the eight warps split the columns of a stage and
//            their partial sums meet in shared memory once per tile.  In the accumulator
//            layout a thread holds g_f and u_f of the same f and the same two tokens, so
//            h = SiLU(g) * u is thread-local; h goes to global memory as bf16.
//   barrier  grid-wide, crossed by the producer warps only (bounded polling of a device counter):
//            the consumers never wait for it.  The requests go through the kernel in two halves,
//            so each half's barrier latency is covered by the other half's streaming.  Both
//            phases run through one ring and one stage sequence, so the first W_d rows are
//            requested the moment a slot comes free, before the CTA has finished phase 1, and run
//            ahead of the barrier as far as the ring allows; only the h rows wait for it.
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
// in phase 2), each fetched by its own cp.async.bulk (one producer lane per row; the producer
// warps share out the ring slots) completing on the stage's mbarrier.  Rows sit at a pitch of 16 bytes more than a multiple of 128, which
// makes the ldmatrix reads and the operand-fragment reads bank-conflict free.
//
// Every wait is bounded: when an mbarrier or the grid barrier does not complete in time the
// warp raises the CTA's abort flag, later waits fall through, the kernel ends normally and the
// error word tells the host.
#include <cstdlib>
#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kProducerWarps = 4;                    // a warp needs ~0.6 us to get one stage's copies out
constexpr int kThreads = (kConsumerWarps + kProducerWarps) * 32;
constexpr int kMaxStages = 8;
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
    __shared__ VrRec s_vrs[kVrShared];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int d = p.d, F = p.F, Fpad = p.Fpad;
    const DevPlan *plan = p.plan;
    const int G = (int)gridDim.x;
    const int NOP = geo.n_op_rows;
    (void)NOP;
    const int S1 = geo.n_stages, PITCH1 = geo.pitch, CB1 = geo.chunk_bytes, STAGE1 = geo.stage_bytes;
    const int S2 = S1, PITCH2 = geo.pitch2, CB2 = geo.chunk_bytes2, STAGE2 = STAGE1;

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
    const uint32_t full2 = full1, empty2 = empty1;          // one ring, one stage sequence for both phases
    volatile int *abort_flag = &s_abort;

    if (tid == 0) {
        s_abort = 0;
        for (int i = 0; i < kMaxStages; ++i) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full1 + 8 * i), "r"(1));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty1 + 8 * i), "r"(kConsumerWarps));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
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
    const int nvA = n_half == 2 ? nv / 2 : nv;                // requests in half A
    int q_lo[2], q_hi[2];                                     // f-row ranges, relative to the half's first request
    {
        const long long rowsA = (long long)nvA * F, rowsB = (long long)(nv - nvA) * F;
        q_lo[0] = (int)(blockIdx.x * rowsA / G);
        q_hi[0] = (int)((blockIdx.x + 1) * rowsA / G);
        q_lo[1] = (int)(blockIdx.x * rowsB / G);
        q_hi[1] = (int)((blockIdx.x + 1) * rowsB / G);
    }
    const int r_lo = (int)((long long)blockIdx.x * d / G), r_hi = (int)((long long)(blockIdx.x + 1) * d / G);
    const int mt = (r_hi - r_lo + 15) / 16;
    const int hi2 = nv * mt, hi2A = nvA * mt;                 // down tiles: request-major, half A first
    unsigned *sync_word = p.sync + 2 * p.group;               // [half]

    if (warp >= kConsumerWarps) {
        // =================================================================== producers
        // The producer warps walk the same stage sequence and share the stages out (a warp is busy
        // for ~0.6 us with one bulk-copy instruction, however few lanes take part, so the stages
        // of a 28 KB-per-stage phase would otherwise leave faster than one warp can issue them).
        // A ring slot always belongs to the same warp (slot s to warp s mod 4), so every wait on a
        // slot's "empty" barrier is made by the one warp that has followed all its earlier phases.
        // Lanes 0..15 fetch the tile's weight rows, lanes 16..23 the operand rows.
        const int pw = warp - kConsumerWarps;
        const bool is_w = lane < 16;
        const int my_row = is_w ? lane : lane - 16;                        // tile row, or token slot
        const int dst_row = lane;
        const bool lane_used = lane < 24;
        bool dead = false;
        // One stage of either phase.  src: this lane's source row or null.  parts bit 0: arm the
        // barrier and fetch the weight rows (the caller has made sure the slot is free); bit 1:
        // operand rows.
        auto issue = [&](const char *src, uint32_t full0, int S, int STAGE, int PITCH, size_t src_off, int wbytes,
                         int obytes, int parts, uint32_t nn) {
            const uint32_t slot = nn % S;
            const uint32_t bar = full0 + 8 * slot;
            const bool active = lane_used && src != nullptr;
            if (parts & 1) {
                const unsigned mw = __ballot_sync(0xffffffffu, active && is_w);
                const unsigned mo = __ballot_sync(0xffffffffu, active && !is_w);
                if (lane == 0)
                    mbar_expect(bar, (uint32_t)__popc(mw) * wbytes + (uint32_t)__popc(mo) * obytes);
                __syncwarp();
            }
            if (active && !dead && (is_w ? (parts & 1) : (parts & 2)))
                bulk_g2s(ring_s + slot * STAGE + dst_row * PITCH, src + src_off, (uint32_t)(is_w ? wbytes : obytes), bar);
        };
        // ---- gate/up: lanes 0..7 W_g rows, 8..15 W_u rows, 16..23 hidden rows of the request's tokens
        uint32_t n1 = 0;
        for (int half = 0; half < n_half; ++half) {
            const int v0 = vb + (half ? nvA : 0);
            int q = q_lo[half];
            while (q < q_hi[half]) {
                const int vr = v0 + q / F, f0 = q % F;
                const int m = min(min(8, F - f0), q_hi[half] - q);
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
                    issue(src, full1, S1, STAGE1, PITCH1, (size_t)kc * CB1, b, b, 3, n1);
                }
                q += m;
            }
        }
        // ---- down: lanes 0..15 W_d rows, 16..23 rows of h.  Two cursors walk the same stage
        // sequence: the weight rows run ahead as far as the ring allows, the h rows of a stage
        // follow once the grid has finished the h of the stage's half.
        struct Cursor {
            int t, k, vr;
            const char *base;
        };
        auto tile_of = [&](Cursor &c) -> const char * {
            const int vr = vb + c.t / mt, blk = c.t % mt;
            if (vr != c.vr) {
                const VrRec *v = vrs + (vr - vb);
                c.vr = vr;
                c.base = nullptr;
                if (lane_used) {
                    if (is_w)
                        c.base = v->blob + (size_t)2 * F * rb1 + (size_t)(r_lo + my_row) * rb2;
                    else if (my_row < v->n_tok)
                        c.base = reinterpret_cast<const char *>(p.hbuf) + ((size_t)vr * kTokPerVr + my_row) * Fpad * 2;
                }
            }
            if (!is_w)
                return c.base;
            return (c.base && r_lo + 16 * blk + my_row < r_hi) ? c.base + (size_t)blk * 16 * rb2 : nullptr;
        };
        auto advance = [&](Cursor &c) {
            if (++c.k == nk2) {
                c.k = 0;
                ++c.t;
            }
        };
        auto w_bytes2 = [&](int kc) { return min(CB2, rb2 - kc * CB2); };
        auto op_bytes2 = [&](int kc) { return min(CB2, Fpad * 2 - kc * CB2); };
        // the down stages follow the gate/up stages in the same ring: stage numbers run on from n1
        const uint32_t N2 = n1 + (uint32_t)hi2 * nk2;
        Cursor wc{0, 0, -1, nullptr}, oc{0, 0, -1, nullptr};
        uint32_t wn = n1, on = n1;
        bool passed[2] = {false, false};
        long long t_idle = 0;
        while (on < N2 && !dead) {
            bool progress = false;
            // weight rows of as many stages as there are free slots
            while (wn < N2) {
                if ((int)((wn % S2) % kProducerWarps) != pw) {
                    (void)tile_of(wc);
                    advance(wc);
                    ++wn;
                    progress = true;
                    continue;
                }
                if (wn >= (uint32_t)S2) {
                    int ok = 0;
                    if (lane == 0)
                        ok = mbar_try(empty2 + 8 * (wn % S2), ((wn / S2) - 1u) & 1u);
                    if (!__shfl_sync(0xffffffffu, ok, 0))
                        break;
                }
                const char *src = tile_of(wc);
                issue(src, full2, S2, STAGE2, PITCH2, (size_t)wc.k * CB2, w_bytes2(wc.k), op_bytes2(wc.k), 1, wn);
                advance(wc);
                ++wn;
                progress = true;
            }
            // h rows of the next stages, once their half of h is complete everywhere
            if (on < wn) {
                const int half = oc.t < hi2A ? 0 : 1;
                if (!passed[half]) {
                    int ok = 0;
                    if (lane == 0) {
                        ok = *reinterpret_cast<volatile unsigned *>(sync_word + half) >= (unsigned)G;
                        if (ok) {
                            __threadfence();
                            if (trace && pw == 0)
                                trace[5] = globaltimer_ns();
                        }
                    }
                    passed[half] = __shfl_sync(0xffffffffu, ok, 0) != 0;
                }
                while (on < wn && passed[oc.t < hi2A ? 0 : 1]) {
                    const char *src = tile_of(oc);
                    if ((int)((on % S2) % kProducerWarps) != pw) {
                        advance(oc);
                        ++on;
                        progress = true;
                        continue;
                    }
                    issue(src, full2, S2, STAGE2, PITCH2, (size_t)oc.k * CB2, 0, op_bytes2(oc.k), 2, on);
                    advance(oc);
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
            }
        }
        const uint32_t n2 = on;
        if (*abort_flag && lane == 0 && pw == 0) {
            // a wait ran out: give the copies still in flight a bounded time to land before this
            // CTA's shared memory goes away
            const long long t0 = clock64();
            for (uint32_t m = n2 > (uint32_t)S2 ? n2 - S2 : 0u; m < n2; ++m)
                while (!mbar_try(full2 + 8 * (m % S2), (m / S2) & 1u) && clock64() - t0 < kWaitLimitCycles) {
                }
            atomicExch(p.err, MELINOE_ERR_TIMEOUT);
        }
        return;
    }

    // ======================================================================= consumers
    const int g = lane >> 2, tig = lane & 3;
    int n_tiles = 0;       // tiles finished so far (selects the reduction buffer and the epilogue warp)
    float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};

    // this warp's share of one stage: some of the 16-column steps of the piece.  Weights in tile
    // rows 0..15, the operand rows (hidden or h) of the request's tokens behind them.
    auto compute = [&](uint32_t full0, uint32_t empty0, int S, int STAGE, uint32_t a_off, uint32_t b_off, uint32_t n,
                       int bytes, int n_tok) {
        const uint32_t slot = n % S;
        mbar_wait(full0 + 8 * slot, (n / S) & 1u, abort_flag);
        const uint32_t base = ring_s + slot * STAGE;
        const int ks_total = (bytes + 31) >> 5;
        const int ks_hi = (warp + 1) * ks_total / kConsumerWarps;
        int ks = warp * ks_total / kConsumerWarps;
        const bool has_tok = g < n_tok;
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
            int q = q_lo[half];
            while (q < q_hi[half]) {
                const int vr = v0 + q / F, f0 = q % F;
                const int m = min(min(8, F - f0), q_hi[half] - q);
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
            // this CTA's part of the half's h is complete: tell the grid
            __threadfence();
            fence_proxy_async();       // h was written through the generic proxy, bulk copies will read it
            consumer_bar();
            if (tid == 0) {
                atomicAdd(sync_word + half, 1u);
                if (trace && half == n_half - 1)
                    trace[4] = globaltimer_ns();
            }
        }
    }

    // ---- down: z = W_d h for this CTA's output rows
    {
        const uint32_t a_off = ((lane & 7) + ((lane >> 3) & 1) * 8) * PITCH2 + (lane >> 4) * 16;
        const uint32_t b_off = (16 + g) * PITCH2 + tig * 4;
        const uint32_t n_first = n;
        // the requests' records are read two requests ahead of their use
        VrInfo v{}, nxt{}, nxt2{};
        if (hi2 > 0) {
            nxt = load_vr(vb);
            nxt2 = nv > 1 ? load_vr(vb + 1) : nxt;
        }
        for (int t = 0; t < hi2; ++t) {
            const int blk = t % mt, iv = t / mt;
            if (blk == 0) {
                v = nxt;
                nxt = nxt2;
                if (iv + 2 < nv)
                    nxt2 = load_vr(vb + iv + 2);
            }
            for (int kc = 0; kc < nk2; ++kc, ++n) {
                compute(full2, empty2, S2, STAGE2, a_off, b_off, n, min(CB2, rb2 - kc * CB2), v.n_tok);
                if (trace && n == n_first && tid == 0)
                    trace[2] = globaltimer_ns();
            }
            float r[4];
            if (reduce_tile(r)) {
                const int row = r_lo + 16 * blk + g;
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
    const size_t fixed = 2 * kConsumerWarps * 128 * sizeof(float) + 2 * kMaxStages * 8 + 128;
    if (cfg.max_smem < fixed + 2 * stage)
        return cudaErrorInvalidConfiguration;
    const size_t avail = (cfg.max_smem - fixed) / 128 * 128;
    size_t n = avail / stage;
    if (n > (size_t)kMaxStages)
        n = kMaxStages;
    geo->n_stages = (int)n;
    geo->stage_bytes = (int)stage;
    geo->ring_bytes = (n * stage + 127) / 128 * 128;
    geo->smem_bytes = geo->ring_bytes + fixed;
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
