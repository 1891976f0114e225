// Decode expert FFN (Eq. 3) with the gate-weighted combine (Eq. 2) fused in: one launch serves up
// to 8 tokens.  The work is reading every needed expert once (from HBM, or over the host link for
// an expert that is not resident), so the kernel is built around one contiguous stream per SM and
// no synchronisation between SMs until the very end.
//
// Layout of an expert ("blob", written by melinoe_moe_pack_expert): for f = 0 .. d_ff - 1 the
// three rows that belong to hidden unit f back to back,
//     W_g[f][0..d) | W_u[f][0..d) | W_d[0..d)[f]   (the last one is row f of W_d transposed),
// 6 d bytes, and inside each row the 16-byte pieces of every 128-byte group are stored at
// position (piece xor (f mod 8)).  Consequences:
//   - the rows f0 .. f0 + m - 1 are ONE contiguous byte range, fetched by one bulk copy;
//   - everything hidden unit f contributes to the output, gate * SiLU(g_f) * u_f * W_d[:, f], can be
//     formed by the SM that read those three rows: no other SM is involved, so the d_ff rows of all
//     requested experts are simply dealt out evenly (single-row granularity) and every CTA ends up
//     with a partial output vector;
//   - eight consecutive rows, read at the same logical column, fall into eight different groups
//     of shared-memory banks (the xor), so the tensor-core fragment loads (ldmatrix) are free of
//     bank conflicts although the rows sit at a pitch that is a multiple of 128 bytes.
//
// One CTA per SM: 16 consumer warps and one producer warp.
//   producer  one thread; per tile (up to 8 rows f of one expert) one cp.async.bulk into a ring
//             stage, completion on the stage's mbarrier.  A missed expert's rows come straight from
//             the page-locked host store (the device reads host memory over the link).
//   gate/up   D[16 x 8] = [W_g rows ; W_u rows] (16 x d) * x^T (d x 8 tokens) on mma.sync m16n8k16
//             (bf16 in, fp32 accumulate): decode is one multiply-add per weight byte pair, far
//             below what even this legacy tensor path delivers, so it is free compute.  The warps
//             split the columns; their partial tiles meet in shared memory once per tile and every
//             warp forms the complete g_f, u_f (thread-local: a thread holds g and u of the same f and
//             the same two tokens), then h = gate[token][expert] * SiLU(g) * u, rounded once to bf16.
//             The gate is folded in here so that all experts accumulate into one output tile.
//   down      Y[c][t] += sum_f W_d^T[f][c] * h[f][t]: the same 8 rows f are now the K dimension
//             (padded to 16 with zeros), A = W_d^T rows read transposed (ldmatrix.trans), every warp
//             owns d / NW output columns and keeps their fp32 accumulators in registers for the
//             whole kernel.
//   fetched   a tile of a missed expert that stays resident after the call is also stored into its
//   experts   cache slot (bulk copy shared -> global) while it is being computed with.
//   combine   every CTA adds its partial [tokens][d] into the call's accumulator in global memory as
//             64-bit fixed point (units of 2^-40; integer atomics: the sum is exact, so it does not
//             depend on the order of arrival and results are bit-identical from run to run), counts
//             itself out on the handle's counter and exits; the CTA that finds all the others gone
//             converts the sums to bf16, writes the output and clears accumulator and counter.  No CTA
//             ever waits for another.
//   4-bit     the same structure on 4-bit blobs (melinoe_moe_pack_expert_q4): the codes are expanded in
//   blobs     registers on their way into the tensor-core fragments, see consume_q4 below.
//
// Every wait is bounded: when an mbarrier or the wait for the plan does not complete in time the warp
// raises the CTA's abort flag, later waits fall through, copies in flight are given a bounded time
// to land, the kernel ends normally and the error word tells the host.

#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kMaxStages = 8;
constexpr int kMaxMt = 16;                       // m-tiles (16 output columns each) / k-steps per warp
// Bound of every wait, in SM clock cycles (about 2 s).
constexpr long long kWaitLimitCycles = 4000000000ll;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

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

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
// D(16x8) += A(16x16) * B(16x8), bf16 in, fp32 accumulate.
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t addr)
{
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}

// Eight 4-bit codes (one 32-bit word: element j in nibble j) into bf16 weights, as four registers
// P[j] = (element j, element j + 4).  A nibble n placed in the mantissa of 0x4300 is the bf16 number
// 128 + n; minus 136 is the integer n - 8, exactly; times the group's scale, rounded once to nearest
// even, is the weight the format defines.  ss = the scale in both halves.
__device__ __forceinline__ void dequant8(uint32_t w, uint32_t ss, uint32_t (&P)[4])
{
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t t = ((w >> (4 * j)) & 0x000f000fu) | 0x43004300u;
        asm("sub.rn.bf16x2 %0, %0, %1;" : "+r"(t) : "r"(0x43084308u));
        asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(P[j]) : "r"(t), "r"(ss));
    }
}

// Tensor memory as a per-thread operand store: 32 consecutive 32-bit columns of the thread's own lane.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
          "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
          "r"(r[30]), "r"(r[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t bf16_rne(float v)
{
    uint32_t u = __float_as_uint(v);
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void bulk_s2g(void *dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Add without a return value, on the global address space (a generic atomicAdd compiles to the
// returning form on the generic space).
__device__ __forceinline__ void red_add_u64(unsigned long long *addr, unsigned long long v)
{
    asm volatile("red.global.add.u64 [%0], %1;" ::"l"(__cvta_generic_to_global(addr)), "l"(v) : "memory");
}
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// An active request of the launch as the tile loops see it.
struct SReq {
    const char *src;      // where its rows are streamed from: the slot, a shared expert's blob, or the host store
    char *wb;             // null, or the slot the fetched rows are also stored into
    int32_t gate_row;     // its row of the gate table (= its index among the launch's requests)
    int32_t deferred;     // the slot is written by the last CTA once every CTA is done (it is still being computed with)
};

constexpr int NW = 16;                           // consumer warps
constexpr int kThreads = (NW + 1) * 32;          // + the producer warp
constexpr int kBufPitch = 130;                   // floats between the warps' partial tiles (keeps the column sums conflict-free)

// ---------------------------------------------------------------------------------------------------
// The consumer warps' work on 4-bit blobs.  One hidden unit f is a unit of geo.row_bytes bytes: the
// codes of W_g[f], W_u[f], W_d[:, f] (d / 2 bytes each) and their scales (one bf16 per 64 elements).
// A 32-bit word of codes is eight consecutive elements and expands into four registers that pair
// element j with element j + 4 (dequant8).  A tensor-core operand register holds two neighbours
// along the contraction, and a sum does not care in which order its terms are met, so:
//   gate/up   the contraction runs over the columns: a thread takes one word of its W_g row and one of
//             its W_u row (columns c .. c + 7) and feeds two products, the k-slots being columns
//             (c, c + 4, c + 1, c + 5) and (c + 2, c + 6, c + 3, c + 7); the hidden state was staged
//             in the same pairing, so one 16-byte load is the matching token operand of both.  The
//             warps split the columns in steps of 32.
//   down      the contraction runs over f, and the two halves of a register are two COLUMNS of one f.
//             They are made two k-slots of that f, and the token operand carries h[f][t] in the first
//             of them for the output columns n = 0..3 (tokens 0..3) and in the second for n = 4..7
//             (again tokens 0..3): the product's left half is column j of every row of output, its right
//             half column j + 4.  One product so covers 8 hidden units x 32 output columns x 4 tokens;
//             tokens 4..7 take a second product.  The warps split the columns in steps of 32.  (The codes
//             of W_d[:, f] are stored interleaved within every 64, nibble j of word g being column
//             g + 8 j, so that the lanes of one product row own neighbouring output columns.)
constexpr int kMaxWs = 8;                        // 32-column steps per warp (d / 512)

// One tile as the loop sees it.
struct Q4Tile {
    uint32_t stage, st;   // shared-memory address of its ring stage, index of the stage
    int m, f0;            // rows, first hidden unit
    int gate_row;
    bool stored;          // this thread issued the tile's store into the cache slot
};

template <int MT_>
__device__ __forceinline__ void consume_q4(const DecParams &p, const DecGeometry &geo, const SReq *s_req, const float *s_gate,
                                           float *s_sums, float *buf, uint32_t ring_s, uint32_t xs_s, uint32_t full0,
                                           uint32_t empty0, volatile int *abort_flag, long long q_lo, long long q_hi, unsigned long long *trace)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tig = lane & 3;
    const int d = p.d, F = p.F;
    const int TR = geo.tile_rows, S = geo.n_stages, RB = geo.row_bytes, STAGE = geo.stage_bytes, XP = geo.x_pitch, Tc = geo.tokens;
    const int WS = MT_ > 0 ? MT_ / 2 : d / (32 * NW);
    float acc[kMaxWs][2][4];
#pragma unroll
    for (int i = 0; i < kMaxWs; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j)
            acc[i][j][0] = acc[i][j][1] = acc[i][j][2] = acc[i][j][3] = 0.f;
    const bool has_tok = g < Tc, two = Tc > 4;
    const uint32_t xrow = xs_s + g * XP + (warp * WS * 32 + tig * 8) * 2;
    const uint32_t sc_off = 3 * (uint32_t)(d / 2), sc_len = (uint32_t)(d / 32);     // scales: offset in the unit, bytes per vector
    const int t0 = g & 3, sh = g < 4 ? 0 : 16;

    // ---- the tiles of this CTA in order; taking one waits until it has landed and starts its copy into the slot
    int left = (int)(q_hi - q_lo);                  // rows still to take
    int a = (int)(q_lo / F), f0 = (int)(q_lo % F);
    uint32_t st = 0, ph = 0;                        // ring stage of the next tile and the parity of its barrier phase
    bool first = true;
    auto take = [&](Q4Tile &t) -> bool {
        if (left <= 0)
            return false;
        t.m = min(min(TR, F - f0), left);
        t.f0 = f0;
        t.st = st;
        t.stage = ring_s + st * STAGE;
        mbar_wait(full0 + 8 * st, ph, abort_flag);
        if (trace && first && tid == 0)
            trace[2] = globaltimer_ns();
        first = false;
        const SReq rq = s_req[a];
        t.gate_row = rq.gate_row;
        t.stored = rq.wb != nullptr && tid == 0;
        if (t.stored)
            bulk_s2g(rq.wb + (size_t)f0 * RB, t.stage, (uint32_t)t.m * RB);
        if (++st == (uint32_t)S) {
            st = 0;
            ph ^= 1u;
        }
        left -= t.m;
        f0 += t.m;
        if (f0 == F) {
            f0 = 0;
            ++a;
        }
        return true;
    };
    // ---- gate/up of one tile: this warp's columns, into registers.  Rows the tile does not have read row 0;
    // their results are dropped when h is formed.
    auto gate_up = [&](const Q4Tile &t, float (&cg)[4][4]) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            cg[i][0] = cg[i][1] = cg[i][2] = cg[i][3] = 0.f;
        const int rr = g < t.m ? g : 0;
        const uint32_t fx16 = (uint32_t)((t.f0 + rr) & 7) << 4;
        const uint32_t row = t.stage + rr * RB;
        // piece ws of the codes sits at ((ws & ~7) | ((ws ^ f) & 7)) * 16: the warp's first step, then xor per step
        const uint32_t ws0 = (uint32_t)(warp * WS);
        const uint32_t cbase = row + (ws0 & ~7u) * 16 + tig * 4, sbase = row + sc_off + (ws0 >> 1) * 2;
        uint32_t sg = 0, su = 0;
#pragma unroll
        for (int i = 0; i < kMaxWs; ++i) {
            if (i < WS) {
                const uint32_t wsl = (ws0 & 7u) + (uint32_t)i;
                const uint32_t off = ((wsl << 4) ^ fx16) & 0x70u, hi = (wsl >> 3) * 128u;
                const uint32_t wg = lds32(cbase + hi + off);
                const uint32_t wu = lds32(cbase + hi + off + (uint32_t)(d / 2));
                if ((i & 1) == 0 || WS == 1) {
                    sg = lds16(sbase + (i >> 1) * 2) * 0x10001u;
                    su = lds16(sbase + (i >> 1) * 2 + sc_len) * 0x10001u;
                }
                uint4 xb = make_uint4(0u, 0u, 0u, 0u);
                if (has_tok)
                    xb = lds128(xrow + i * 64);
                uint32_t Pg[4], Pu[4];
                dequant8(wg, sg, Pg);
                dequant8(wu, su, Pu);
                mma_16816(cg[(2 * i) & 3], Pg[0], Pu[0], Pg[1], Pu[1], xb.x, xb.y);
                mma_16816(cg[(2 * i + 1) & 3], Pg[2], Pu[2], Pg[3], Pu[3], xb.z, xb.w);
            }
        }
    };
    // The warps' partial tiles meet in shared memory: every warp stores its 128 partial values, warp w sums
    // 8 of the 128 over all warps (four lanes per value, each adding four warps' parts in warp order, then a
    // fixed tree), and every warp reads the complete tile.  Two block-wide named barriers order this; the
    // buffers alternate from tile to tile.  (Measured and dropped: counting mbarriers in their place, with
    // the loop running one tile ahead so that a warp has other work between arriving and waiting -- the
    // hardware barrier is the cheaper way for 16 warps to meet; and h formed once per tile by the summing
    // warps instead of by every warp for itself -- it lengthens the path between the two barriers.)
    auto store_partials = [&](const float (&cg)[4][4], uint32_t sel) {
        float *b = buf + sel * (NW * kBufPitch) + warp * kBufPitch;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            b[i * 32 + lane] = (cg[0][i] + cg[1][i]) + (cg[2][i] + cg[3][i]);
    };
    auto column_sums = [&](uint32_t sel) {
        const float *b = buf + sel * (NW * kBufPitch);
        const int e = warp * 8 + (lane & 7), pg = lane >> 3;
        float v = b[(pg * 4) * kBufPitch + e];
        v += b[(pg * 4 + 1) * kBufPitch + e];
        v += b[(pg * 4 + 2) * kBufPitch + e];
        v += b[(pg * 4 + 3) * kBufPitch + e];
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        if (lane < 8)
            s_sums[sel * 128 + e] = v;
    };
    // ---- h of the tile from the complete sums, then the down product
    auto down = [&](const Q4Tile &t, uint32_t sel) {
        // g_f[t] and u_f[t] of the tile sit at (t & 1) * 32 + 4 f + (t >> 1) and 64 further on (the
        // accumulator layout of the product).  This thread needs h of f = tig, tig + 4 for token g mod 4
        // (and that token + 4).
        const float *sums = s_sums + sel * 128;
        // (h rounded to bf16 once, to nearest even; it goes to the register half of this thread's output column)
        auto hval = [&](int f, int tk) -> uint32_t {
            const int o = (tk & 1) * 32 + f * 4 + (tk >> 1);
            const float vg = sums[o], vu = sums[64 + o];
            const float gt = s_gate[t.gate_row * kTokPerVr + tk];
            float h = __fdividef(vg, 1.0f + __expf(-vg)) * vu * gt;
            if (f >= t.m || gt == 0.0f)
                h = 0.f;
            uint32_t r;
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(sh ? h : 0.f), "f"(sh ? 0.f : h));
            return r;
        };
        const uint32_t b0 = hval(tig, t0), b1 = hval(tig + 4, t0);
        uint32_t b0h = 0u, b1h = 0u;
        if (two) {
            b0h = hval(tig, t0 + 4);
            b1h = hval(tig + 4, t0 + 4);
        }
        const int ra = tig < t.m ? tig : 0, rb = tig + 4 < t.m ? tig + 4 : 0;
        const uint32_t fa16 = (uint32_t)((t.f0 + ra) & 7) << 4, fb16 = (uint32_t)((t.f0 + rb) & 7) << 4;
        const uint32_t rowa = t.stage + ra * RB, rowb = t.stage + rb * RB;
        const int hf = warp & 1;
        // block = 64 output columns = one scale group = two 16-byte pieces of codes; this thread's word is in piece
        // 2 block + g / 4
        const uint32_t blk0 = (uint32_t)(warp * WS) >> 1, pc0 = blk0 * 2 + (uint32_t)(g >> 2);
        const uint32_t cofs = (uint32_t)d + (pc0 & ~7u) * 16 + (g & 3) * 4, sofs = sc_off + 2 * sc_len + blk0 * 2;
#pragma unroll
        for (int b = 0; b < kMaxWs / 2; ++b) {
            if (2 * b < WS) {
                // (pc0 + 2 b) & 7 = (pc0 & 7) + 2 b for b < 4: pc0 & 7 is 0, 1 (four blocks), 0..5 (two), 0..7 (one or half)
                const uint32_t pin = ((pc0 & 7u) + 2u * (uint32_t)b) << 4;
                const uint32_t hi = (pin >> 7) * 128u;
                const uint32_t wa = lds32(rowa + cofs + hi + ((pin ^ fa16) & 0x70u));
                const uint32_t wb = lds32(rowb + cofs + hi + ((pin ^ fb16) & 0x70u));
                const uint32_t sa = lds16(rowa + sofs + b * 2) * 0x10001u;
                const uint32_t sb = lds16(rowb + sofs + b * 2) * 0x10001u;
                uint32_t Pa[4], Pb[4];
                dequant8(wa, sa, Pa);
                dequant8(wb, sb, Pb);
                if (WS == 1) {
                    // two warps share the block: this one owns the product rows made of nibbles 2 hf, 2 hf + 1 (and + 4)
                    const uint32_t a0 = hf ? Pa[2] : Pa[0], a1 = hf ? Pa[3] : Pa[1], a2 = hf ? Pb[2] : Pb[0], a3 = hf ? Pb[3] : Pb[1];
                    mma_16816(acc[0][0], a0, a1, a2, a3, b0, b1);
                    if (two)
                        mma_16816(acc[0][1], a0, a1, a2, a3, b0h, b1h);
                } else {
                    mma_16816(acc[2 * b][0], Pa[0], Pa[1], Pb[0], Pb[1], b0, b1);
                    mma_16816(acc[2 * b + 1][0], Pa[2], Pa[3], Pb[2], Pb[3], b0, b1);
                    if (two) {
                        mma_16816(acc[2 * b][1], Pa[0], Pa[1], Pb[0], Pb[1], b0h, b1h);
                        mma_16816(acc[2 * b + 1][1], Pa[2], Pa[3], Pb[2], Pb[3], b0h, b1h);
                    }
                }
            }
        }
        if (t.stored)
            bulk_wait_read();         // the slot store has read the stage
        __syncwarp();
        if (lane == 0)
            mbar_arrive(empty0 + 8 * t.st);
    };

    Q4Tile cur;
    float cg[4][4];
    for (uint32_t i = 0; take(cur); ++i) {
        gate_up(cur, cg);
        store_partials(cg, i & 1u);
        asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");      // every warp's partial sums of the tile are stored
        column_sums(i & 1u);
        asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");      // the complete sums of the tile are there
        down(cur, i & 1u);
    }
    if (trace && tid == 0)
        trace[3] = globaltimer_ns();
    // ---- this CTA's partial output into the call's accumulator (64-bit fixed point, as in the bf16 path).
    // Accumulator i of the warp is the 32-column step hb = warp * WS + i: block hb / 2, and within the
    // block's 64 columns (whose codes are stored interleaved: nibble j of word g is column g + 8 j),
    // column g + 16 (hb mod 2) + {0, 8} for the product's rows g, g + 8, plus 32 for the product's right
    // half (tig >= 2); its columns there are tokens 2 (tig mod 2), + 1.  Eight lanes of an add are
    // eight neighbouring columns.
    {
        unsigned long long *yacc = reinterpret_cast<unsigned long long *>(p.yacc);
        auto add = [&](int t, int c, float v) {
            if (t < Tc) {
                const long long fx = __float2ll_rn(v * 1099511627776.0f);
                red_add_u64(yacc + (size_t)t * d + c, (unsigned long long)fx);
            }
        };
#pragma unroll
        for (int i = 0; i < kMaxWs; ++i) {
            if (i < WS) {
                const int hb = warp * WS + i;
                const int c = (hb >> 1) * 64 + g + 16 * (hb & 1) + 32 * (tig >> 1);
                const int t = 2 * (tig & 1);
#pragma unroll
                for (int tg = 0; tg < 2; ++tg) {
                    if (tg == 0 || two) {
                        add(t + 4 * tg, c, acc[i][tg][0]);
                        add(t + 4 * tg + 1, c, acc[i][tg][1]);
                        add(t + 4 * tg, c + 8, acc[i][tg][2]);
                        add(t + 4 * tg + 1, c + 8, acc[i][tg][3]);
                    }
                }
            }
        }
    }
}

// MT_: k-steps of the gate/up phase and m-tiles of the down phase per warp (d / 256), 0 = taken from d at run time.
// FMT: 0 = bf16 expert blobs, 1 = 4-bit blobs (melinoe_moe_pack_expert_q4), expanded in registers on
// the way into the tensor-core fragments.
// XT: 1 = the hidden states' tensor-core operand fragments are kept in tensor memory instead of shared
// memory (bf16 blobs, d_model 4096 and more than 4 tokens: 64 KB of shared memory go to the ring instead,
// which doubles the height of the tiles that fit).
template <int MT_, int FMT, int XT = 0>
__global__ void __launch_bounds__(kThreads, 1) ffn_decode_kernel(DecParams p, DecGeometry geo)
{
    static_assert(XT == 0 || (FMT == 0 && MT_ == 16), "tensor-memory operands: bf16 blobs, d_model 4096");
    __shared__ uint32_t s_tmem;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_abort, s_nact, s_last;
    __shared__ int s_hdr[4];                        // status, n_groups, first request, one past the last
    __shared__ DecReq s_raw[kMaxReq];
    __shared__ SReq s_req[kMaxReq];
    __shared__ float s_gate[kMaxReq][kTokPerVr];    // gate of (request, token of the launch); 0 = not routed
    __shared__ unsigned s_match[kMaxReq];
    __shared__ int32_t s_of_expert[kMaxReq];        // request of an expert id (routed 0..E-1, shared E..), -1 = none
    __shared__ int32_t s_idx[kTokPerVr * 32];
    __shared__ float s_gw[kTokPerVr * 32];
    __shared__ float s_sums[256];
    __shared__ __align__(8) uint64_t s_bars[2 * kMaxStages + 1];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int d = p.d, F = p.F;
    const int G = (int)gridDim.x;
    const int TR = geo.tile_rows, S = geo.n_stages, RB = geo.row_bytes, STAGE = geo.stage_bytes, XP = geo.x_pitch;
    const int Tc = geo.tokens, tok0 = p.chunk * kTokPerVr;
    const int MT = MT_ > 0 ? MT_ : d / (16 * NW);

    unsigned long long *trace = p.trace ? p.trace + (size_t)blockIdx.x * 8 : nullptr;
    if (trace && tid == 0)
        trace[0] = globaltimer_ns();

    // ring | staged hidden rows | the warps' partial gate/up tiles
    unsigned char *ring = smem;
    unsigned char *xs = smem + (size_t)S * STAGE;
    float *buf = reinterpret_cast<float *>(xs + (XT ? 0 : (size_t)Tc * XP));        // [NW][kBufPitch]
    const uint32_t ring_s = smem_u32(ring), xs_s = smem_u32(xs);
    const uint32_t full0 = smem_u32(s_bars), empty0 = full0 + 8 * kMaxStages, hzbar = empty0 + 8 * kMaxStages;
    volatile int *abort_flag = &s_abort;

    if (tid == 0) {
        s_abort = 0;
        s_nact = 0;
        for (int i = 0; i < kMaxStages; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, NW);
        }
        mbar_init(hzbar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < kMaxReq; i += kThreads) {
        s_match[i] = 0u;
        s_of_expert[i] = -1;
    }
    // Nothing above reads what an earlier kernel wrote.  With programmatic stream serialisation this
    // CTA may be running while the kernel ahead of it in the stream (the planner) still is.  It does
    // not wait for that grid to drain (which costs microseconds) but for the word the planner writes
    // last, behind a device-wide fence, when the call's plan is complete.  The planner itself has
    // waited for everything ahead of it in the stream, so whatever this kernel reads (hidden states,
    // routing, plan) is in memory once the word is there.  A programmatically launched grid never
    // starts before every CTA of the grid ahead of it is running, and the planner waits for nobody
    // behind it, so the wait ends; it is bounded all the same.
    if (p.wait_prior)
        asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const DevPlan *plan = p.plan;
    if (tid == 0) {
        const long long t0 = clock64();
        for (;;) {
            unsigned v;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(&plan->ready_seq) : "memory");
            if (v == p.call_seq)
                break;
            if (clock64() - t0 > kWaitLimitCycles) {
                s_abort = 1;
                break;
            }
        }
    }
    __syncthreads();

    // ---- everything the launch needs to know, in one round trip to memory
    if (tid == kThreads - 1) {
        const int n_groups = plan->n_groups;
        s_hdr[0] = plan->status;
        s_hdr[1] = n_groups;
        if (p.group < 0) {
            s_hdr[2] = 0;
            s_hdr[3] = plan->n_dreq;
        } else {
            s_hdr[2] = plan->group_vr_begin[p.group];
            s_hdr[3] = plan->group_vr_begin[p.group + 1];
        }
    }
    if (tid < kMaxReq) {
        const uint4 *src = reinterpret_cast<const uint4 *>(plan->dreq + tid);
        uint4 *dst = reinterpret_cast<uint4 *>(s_raw + tid);
        dst[0] = src[0];
        dst[1] = src[1];
    }
    for (int i = tid; i < Tc * p.k; i += kThreads) {
        s_idx[i] = p.idx[(size_t)tok0 * p.k + i];
        s_gw[i] = p.gate[(size_t)tok0 * p.k + i];
    }
    if (XT == 0) {
        const int per_row = d / 8;                  // 16-byte pieces of a hidden row
        for (int i = tid; i < Tc * per_row; i += kThreads) {
            const int t = i / per_row, c = i % per_row;
            uint4 v = *reinterpret_cast<const uint4 *>(p.x + (size_t)(tok0 + t) * d + c * 8);
            if (FMT == 1)       // elements (0,4) (1,5) (2,6) (3,7): the pairing of the expanded weight registers
                v = make_uint4(__byte_perm(v.x, v.z, 0x5410), __byte_perm(v.x, v.z, 0x7632), __byte_perm(v.y, v.w, 0x5410),
                               __byte_perm(v.y, v.w, 0x7632));
            *reinterpret_cast<uint4 *>(xs + (size_t)t * XP + c * 16) = v;
        }
    }
    __syncthreads();
    const int status = s_abort == 1 ? (int)MELINOE_ERR_TIMEOUT : s_hdr[0], n_groups = s_hdr[1], rq0 = s_hdr[2];
    const int nrq = s_hdr[3] - rq0;
    if (status != MELINOE_OK || nrq < 0 || nrq > kMaxReq) {
        if (s_abort == 1 && tid == 0)
            atomicExch(p.err, MELINOE_ERR_TIMEOUT);
        // the call was refused on the device: the output is all zeros, the status tells why
        if (p.group <= 0)
            for (size_t i = (size_t)blockIdx.x * kThreads + tid; i < (size_t)Tc * d; i += (size_t)G * kThreads)
                p.out[(size_t)tok0 * d + i] = 0;
        if (tid == 0) {
            // the counter advances once per CTA and launch, whatever happens
            if (atomicAdd(p.sync, 1u) == (unsigned)(G - 1))
                *p.sync = 0u;
        }
        return;
    }
    if (XT) {
        // 128 columns of tensor memory: 16 warps x 32 columns of operand fragments (see below)
        if (warp == 0) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(128));
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    // gate of every (request, token): the token's gate for that expert if the router chose it
    for (int i = tid; i < nrq * kTokPerVr; i += kThreads) {
        const int r = i / kTokPerVr, t = i % kTokPerVr;
        const int e = s_raw[rq0 + r].expert;
        if (t == 0 && e >= 0 && e < kMaxReq)
            s_of_expert[e] = r;
        float gv = 0.0f;
        if (t < Tc) {
            if (e >= p.E) {
                gv = 1.0f;              // shared expert: every token, gate 1
                atomicOr(&s_match[r], 1u << t);
            } else {
                for (int j = 0; j < p.k; ++j)
                    if (s_idx[t * p.k + j] == e) {
                        gv = s_gw[t * p.k + j];
                        atomicOr(&s_match[r], 1u << t);
                    }
            }
        }
        s_gate[r][t] = gv;
    }
    __syncthreads();
    // The requests that have a token in this launch, in ascending expert id (shared experts last): the
    // rows are dealt out in that order, so the order of every sum depends only on which experts the
    // tokens use, not on which of them happened to be resident.
    if (warp == 0) {
        int base = 0;
        for (int e0 = 0; e0 < kMaxReq; e0 += 32) {
            const int e = e0 + lane;
            const int r = e < kMaxReq ? s_of_expert[e] : -1;
            // a fetched expert that stays resident is streamed (and stored into its slot) by the launch whose
            // job that is even if none of this launch's tokens uses it
            bool act = r >= 0 && s_match[r] != 0u;
            bool pull = false, stays = false, hazard = false;
            if (r >= 0 && p.group < 0 && (s_raw[rq0 + r].flags & kDecMiss)) {
                const int fl = s_raw[rq0 + r].flags;
                pull = true;
                stays = (fl & kDecStays) != 0 && p.write_back != 0;
                hazard = (fl & kDecHazard) != 0;
                if (stays && (hazard ? p.chunk == p.n_chunks - 1 : p.chunk == 0))
                    act = true;
            }
            const unsigned m = __ballot_sync(0xffffffffu, act);
            if (act) {
                const DecReq q = s_raw[rq0 + r];
                SReq sr;
                sr.src = q.blob;
                sr.wb = nullptr;
                sr.gate_row = r;
                sr.deferred = 0;
                if (pull) {
                    // Where a call is made in several launches (more than 8 tokens): the first one stores
                    // the expert into its slot and the later ones read it there, unless the slot still
                    // holds an expert the call computes with: then every launch reads the host store and
                    // the last one stores it once all CTAs are done.
                    if (stays && !hazard && p.chunk > 0) {
                        sr.src = q.blob;
                    } else {
                        sr.src = q.host;
                        if (q.host == nullptr)
                            s_abort = 2;
                        if (stays && !hazard)
                            sr.wb = const_cast<char *>(q.blob);
                        if (stays && hazard && p.chunk == p.n_chunks - 1)
                            sr.deferred = 1;
                    }
                }
                s_req[base + __popc(m & ((1u << lane) - 1u))] = sr;
            }
            base += __popc(m);
        }
        if (lane == 0)
            s_nact = base;
    }
    __syncthreads();
    const int nact = s_nact;
    const bool no_host = s_abort == 2;      // a missed expert cannot be read from here: nothing is computed
    if (trace && tid == 0)
        trace[1] = globaltimer_ns();

    // ---- this CTA's share of the rows: f rows of the active requests, request-major, dealt out evenly
    const long long rows = no_host ? 0 : (long long)nact * F;
    const long long q_lo = blockIdx.x * rows / G, q_hi = (blockIdx.x + 1) * rows / G;

    if (warp == NW) {
        // =================================================================== producer
        if (lane == 0) {
            uint32_t n = 0;
            long long q = q_lo;
            int a = (int)(q / F), f0 = (int)(q % F);
            while (q < q_hi) {
                const int m = (int)min((long long)min(TR, F - f0), q_hi - q);
                const uint32_t st = n % (uint32_t)S;
                if (n >= (uint32_t)S && !mbar_wait(empty0 + 8 * st, ((n / S) - 1u) & 1u, abort_flag))
                    break;
                const uint32_t bytes = (uint32_t)m * RB;
                mbar_expect(full0 + 8 * st, bytes);
                bulk_g2s(ring_s + st * STAGE, s_req[a].src + (size_t)f0 * RB, bytes, full0 + 8 * st);
                ++n;
                q += m;
                f0 += m;
                if (f0 == F) {
                    f0 = 0;
                    ++a;
                }
            }
            if (*abort_flag) {
                // a wait ran out: give the copies still in flight a bounded time to land before this
                // CTA's shared memory goes away
                const long long t0 = clock64();
                for (uint32_t j = n > (uint32_t)S ? n - S : 0; j < n; ++j)
                    while (!mbar_try(full0 + 8 * (j % S), (j / S) & 1u) && clock64() - t0 < kWaitLimitCycles) {
                    }
            }
        }
    } else {
        // =================================================================== consumers
        const int g = lane >> 2, tig = lane & 3;
        if constexpr (FMT == 1) {
            consume_q4<MT_>(p, geo, s_req, &s_gate[0][0], s_sums, buf, ring_s, xs_s, full0, empty0, abort_flag, q_lo, q_hi, trace);
        } else {
        float acc[kMaxMt][4];
#pragma unroll
        for (int i = 0; i < kMaxMt; ++i)
            acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
        const bool has_tok = g < Tc;
        const uint32_t xrow = xs_s + g * XP + tig * 4 + warp * MT * 32;     // this warp's columns of token g
        // XT: the token operand of this thread's 16 gate/up steps (two registers each) never changes, so it is
        // written once into the thread's own lane of tensor memory (warp w may use lanes 32 (w mod 4) ..,
        // the four warps of a lane quarter take 32 columns each) and fetched from there step by step.
        uint32_t xt = 0;
        if constexpr (XT == 1) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            xt = s_tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(warp >> 2) * 32;
            uint32_t r[32];
            const uint16_t *xr = p.x + (size_t)(tok0 + (has_tok ? g : 0)) * d + warp * 256 + 2 * tig;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                r[2 * i] = has_tok ? __ldcg(reinterpret_cast<const uint32_t *>(xr + i * 16)) : 0u;
                r[2 * i + 1] = has_tok ? __ldcg(reinterpret_cast<const uint32_t *>(xr + i * 16 + 8)) : 0u;
            }
            tmem_st32(xt, r);
        }
        // ldmatrix lane roles.  gate/up: matrices (W_g rows, k low), (W_u rows, k low), (W_g rows, k high),
        // (W_u rows, k high); down: four consecutive 8-column pieces of the W_d^T rows
        const int r8 = lane & 7, sel_gu = (lane >> 3) & 1, kh = lane >> 4, mat = lane >> 3;
        const uint32_t src0 = (uint32_t)((2 * tig) * 4 + (g >> 1)), src1 = src0 + 4;
        uint32_t n = 0;
        long long q = q_lo;
        int a = (int)(q / F), f0 = (int)(q % F);
        bool first = true;
        while (q < q_hi) {
            const int m = (int)min((long long)min(TR, F - f0), q_hi - q);
            const uint32_t st = n % (uint32_t)S;
            const uint32_t stage = ring_s + st * STAGE;
            mbar_wait(full0 + 8 * st, (n / S) & 1u, abort_flag);
            if (trace && first && tid == 0)
                trace[2] = globaltimer_ns();
            first = false;
            const SReq rq = s_req[a];
            const bool store_tile = rq.wb != nullptr && tid == 0;
            if (store_tile)
                bulk_s2g(rq.wb + (size_t)f0 * RB, stage, (uint32_t)m * RB);
            const int rr = r8 < m ? r8 : 0;               // rows the tile does not have read row 0 (never used)
            const uint32_t swz = (uint32_t)((f0 + rr) & 7);
            const uint32_t rowbase = stage + rr * RB;
            // ---- gate/up: this warp's columns of the tile's rows.  A dependent mma.sync issues only every
            // ~110 cycles, so the k-steps go to four independent accumulators, and the fragment loads of
            // four steps are issued before their four products.
            // (Where a warp has 16 m-tiles of output accumulators, d_model above 2048, registers only allow
            // two steps at a time.)
            constexpr int GG = (MT_ > 8 || MT_ == 0) ? 2 : 4;
            float cg[GG][4];
#pragma unroll
            for (int i = 0; i < GG; ++i)
                cg[i][0] = cg[i][1] = cg[i][2] = cg[i][3] = 0.f;
            {
                const uint32_t arow = rowbase + sel_gu * 2 * d;
                const uint32_t ch0 = (uint32_t)(2 * warp * MT + kh);
#pragma unroll
                for (int i0 = 0; i0 < kMaxMt; i0 += GG) {
                    if (i0 < MT) {
                        uint32_t af[GG][4], bf[GG][2];
#pragma unroll
                        for (int j = 0; j < GG; ++j) {
                            const int i = i0 + j < MT ? i0 + j : i0;     // beyond the warp's last step: a valid address, product unused
                            ldmatrix_x4(arow + (((ch0 + 2 * i) ^ swz) << 4), af[j][0], af[j][1], af[j][2], af[j][3]);
                            if constexpr (XT == 0) {
                                bf[j][0] = has_tok ? lds32(xrow + i * 32) : 0u;
                                bf[j][1] = has_tok ? lds32(xrow + i * 32 + 16) : 0u;
                            }
                        }
                        if constexpr (XT == 1) {
                            static_assert(XT == 0 || GG == 2, "two steps per group");
                            tmem_ld4(xt + 2 * i0, bf[0][0], bf[0][1], bf[GG - 1][0], bf[GG - 1][1]);
                            tmem_wait_ld();
                        }
#pragma unroll
                        for (int j = 0; j < GG; ++j)
                            if (i0 + j < MT)
                                mma_16816(cg[j], af[j][0], af[j][1], af[j][2], af[j][3], bf[j][0], bf[j][1]);
                    }
                }
            }
            // ---- the warps' partial tiles meet: warp w sums 8 of the tile's 128 values over all warps (four
            // lanes per value, each adding four warps' parts in warp order, then a fixed tree), then every
            // warp reads the complete tile
#pragma unroll
            for (int i = 0; i < 4; ++i)
                buf[warp * kBufPitch + i * 32 + lane] = GG == 4 ? (cg[0][i] + cg[1][i]) + (cg[2][i] + cg[3][i]) : cg[0][i] + cg[GG - 1][i];
            asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");
            {
                const int e = warp * 8 + (lane & 7), pg = lane >> 3;
                float v = buf[(pg * 4) * kBufPitch + e];
                v += buf[(pg * 4 + 1) * kBufPitch + e];
                v += buf[(pg * 4 + 2) * kBufPitch + e];
                v += buf[(pg * 4 + 3) * kBufPitch + e];
                v += __shfl_xor_sync(0xffffffffu, v, 8);
                v += __shfl_xor_sync(0xffffffffu, v, 16);
                if (lane < 8)
                    s_sums[e] = v;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");
            const float s0 = s_sums[lane], s1 = s_sums[32 + lane], s2 = s_sums[64 + lane], s3 = s_sums[96 + lane];
            // rows g and g + 8 of the tile are g_f and u_f of f = f0 + g, columns are tokens 2 tig, 2 tig + 1
            const float gt0 = s_gate[rq.gate_row][2 * tig], gt1 = s_gate[rq.gate_row][2 * tig + 1];
            // (the fast division: the exact one takes its slow path for the zeros of unused token columns)
            float h0 = __fdividef(s0, 1.0f + __expf(-s0)) * s2 * gt0;
            float h1 = __fdividef(s1, 1.0f + __expf(-s1)) * s3 * gt1;
            if (g >= m || gt0 == 0.0f)
                h0 = 0.f;
            if (g >= m || gt1 == 0.0f)
                h1 = 0.f;
            const uint32_t hp = bf16_rne(h0) | (bf16_rne(h1) << 16);
            // B fragment of the down product: h[f = 2 tig', 2 tig' + 1][token g'] from the lanes that hold them
            const uint32_t v0 = __shfl_sync(0xffffffffu, hp, src0), v1 = __shfl_sync(0xffffffffu, hp, src1);
            const uint32_t bd = (g & 1) ? ((v0 >> 16) | (v1 & 0xffff0000u)) : ((v0 & 0xffffu) | (v1 << 16));
            // ---- down: the tile's rows are the K dimension (rows the tile does not have count as zero)
            {
                const uint32_t km = (2 * tig < m ? 0x0000ffffu : 0u) | (2 * tig + 1 < m ? 0xffff0000u : 0u);
                const uint32_t drow = rowbase + 4 * d;
                const uint32_t cc0 = (uint32_t)(warp * MT * 2);
                constexpr int DG = (MT_ > 8 || MT_ == 0) ? 2 : 4;      // loads (of two m-tiles each) per group
#pragma unroll
                for (int m0 = 0; m0 < kMaxMt; m0 += 2 * DG) {
                    if (m0 < MT) {
                        // fragment loads of up to eight m-tiles first, then their products
                        uint32_t rf[DG][4];
#pragma unroll
                        for (int j = 0; j < DG; ++j) {
                            // a load covers two m-tiles; an odd last one is fetched together with the one before
                            // it (or, if it is the warp's only one, with 16 columns that are not used)
                            int mi = m0 + 2 * j;
                            if (mi >= MT)
                                mi = m0;
                            else if (mi + 1 >= MT && mi > 0)
                                mi -= 1;
                            ldmatrix_x4_trans(drow + (((cc0 + 2 * mi + mat) ^ swz) << 4), rf[j][0], rf[j][1], rf[j][2], rf[j][3]);
                        }
#pragma unroll
                        for (int j = 0; j < DG; ++j) {
                            const int mi = m0 + 2 * j;
                            if (mi + 1 < MT) {
                                mma_16816(acc[mi], rf[j][0] & km, rf[j][1] & km, 0u, 0u, bd, 0u);
                                mma_16816(acc[mi + 1], rf[j][2] & km, rf[j][3] & km, 0u, 0u, bd, 0u);
                            } else if (mi < MT) {
                                if (mi > 0)
                                    mma_16816(acc[mi], rf[j][2] & km, rf[j][3] & km, 0u, 0u, bd, 0u);
                                else
                                    mma_16816(acc[mi], rf[j][0] & km, rf[j][1] & km, 0u, 0u, bd, 0u);
                            }
                        }
                    }
                }
            }
            if (store_tile)
                bulk_wait_read();         // the slot store has read the stage
            __syncwarp();
            if (lane == 0)
                mbar_arrive(empty0 + 8 * st);
            ++n;
            q += m;
            f0 += m;
            if (f0 == F) {
                f0 = 0;
                ++a;
            }
        }
        if (trace && tid == 0)
            trace[3] = globaltimer_ns();
        // ---- this CTA's partial output, added into the call's accumulator as 64-bit fixed point (2^-40):
        // integer addition is exact, so the sum does not depend on the order in which the CTAs arrive.
        // (Adds without a return value: atomics that return the old word, which would let the last adder
        // of an element finish it on the spot, measured three times slower under this contention.)
        {
            unsigned long long *yacc = reinterpret_cast<unsigned long long *>(p.yacc);
            auto add = [&](int t, int c, float v) {
                const long long fx = __float2ll_rn(v * 1099511627776.0f);    // exact scaling, then to the nearest 2^-40
                red_add_u64(yacc + (size_t)t * d + c, (unsigned long long)fx);
            };
#pragma unroll
            for (int mi = 0; mi < kMaxMt; ++mi) {
                if (mi < MT) {
                    const int c = (warp * MT + mi) * 16 + g;
                    if (2 * tig < Tc) {
                        add(2 * tig, c, acc[mi][0]);
                        add(2 * tig, c + 8, acc[mi][2]);
                    }
                    if (2 * tig + 1 < Tc) {
                        add(2 * tig + 1, c, acc[mi][1]);
                        add(2 * tig + 1, c + 8, acc[mi][3]);
                    }
                }
            }
        }
        }
        if (tid == 0)
            bulk_wait_all();              // the slot stores of this thread have completed
    }

    // ---- the CTA that finishes last turns the sums into the output; all others are done
    if (XT)
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (XT) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (warp == 0)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(s_tmem), "r"(128));
    }
    if (tid == 0) {
        __threadfence();
        const unsigned ticket = atomicAdd(p.sync, 1u);
        s_last = ticket == (unsigned)(G - 1);
        if (s_last)
            *p.sync = 0u;                 // the counter is back at zero for the next launch
        if (trace)
            trace[4] = globaltimer_ns();
    }
    __syncthreads();
    if (*abort_flag && tid == 0)
        atomicExch(p.err, no_host ? MELINOE_ERR_STATE : MELINOE_ERR_TIMEOUT);
    if (!s_last) {
        if (trace && tid == 0)
            trace[7] = globaltimer_ns();
        return;
    }
    __threadfence();
    if (trace && tid == 0)
        trace[5] = globaltimer_ns();
    {
        const bool acc_in = p.group > 0, acc_out = p.group >= 0 && p.group < n_groups - 1;
        long long *yacc = p.yacc;
        const int N = Tc * d;
        // four elements per thread at a time, all their loads before any store: this CTA is the whole
        // grid's critical path, and a load behind a store that may alias it would wait for it
        constexpr int kBatch = 4;
        for (int e0 = tid; e0 < N; e0 += kBatch * kThreads) {
            long long fx[kBatch];
            float carry[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const int e = e0 + j * kThreads;
                fx[j] = e < N ? __ldcg(yacc + e) : 0ll;
                carry[j] = (acc_in && e < N) ? __ldcg(p.ybuf + (size_t)tok0 * d + e) : 0.0f;
            }
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const int e = e0 + j * kThreads;
                if (e < N) {
                    yacc[e] = 0;                                 // the accumulator is left clean for the next launch
                    float v = __ll2float_rn(fx[j]) * (1.0f / 1099511627776.0f);     // one rounding, then an exact scaling
                    const size_t o = (size_t)tok0 * d + e;       // element e of the launch's [tokens][d] block
                    if (acc_in)
                        v += carry[j];
                    if (acc_out)
                        p.ybuf[o] = v;
                    else
                        p.out[o] = (uint16_t)bf16_rne(v);
                }
            }
        }
    }
    if (trace && tid == 0)
        trace[6] = globaltimer_ns();

    // ---- fetched experts whose slot was still being computed with: stored now that every CTA is done
    if (tid == 0) {
        uint32_t phase = 0;
        bool any = false;
        __syncwarp();
        for (int a = 0; a < nact && *abort_flag != 1; ++a) {
            if (!s_req[a].deferred)
                continue;
            const SReq rq = s_req[a];
            char *slot = const_cast<char *>(s_raw[rq0 + rq.gate_row].blob);
            for (int f = 0; f < F; f += TR) {
                const uint32_t bytes = (uint32_t)min(TR, F - f) * RB;
                if (any)
                    bulk_wait_read();
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect(hzbar, bytes);
                bulk_g2s(ring_s, rq.src + (size_t)f * RB, bytes, hzbar);
                if (!mbar_wait(hzbar, phase & 1u, abort_flag))
                    break;
                ++phase;
                bulk_s2g(slot + (size_t)f * RB, ring_s, bytes);
                any = true;
            }
        }
        if (any)
            bulk_wait_all();
        if (*abort_flag == 1)
            atomicExch(p.err, MELINOE_ERR_TIMEOUT);
    }
    if (trace && tid == 0)
        trace[7] = globaltimer_ns();
}

}  // namespace

bool ffn_decode_supported(int d, int F) { return d % 256 == 0 && d >= 256 && d <= 4096 && F % kUnitRows == 0; }
// 4-bit slots: the warps split the columns in steps of 32 (one 16-byte piece of codes), 16 warps; a warp's
// steps are 1, 2, 4 or 8 (whole scale groups, or half of one shared by two warps).
bool ffn_decode_supported_q4(int d, int F)
{
    return ffn_decode_supported(d, F) && (d == 512 || d == 1024 || d == 2048 || d == 4096);
}

cudaError_t ffn_decode_configure(int n_sms, size_t max_smem, DecLaunchCfg *cfg)
{
    size_t stat = 0;
    const void *fns[7] = {reinterpret_cast<const void *>(ffn_decode_kernel<16, 0, 1>),
                          reinterpret_cast<const void *>(ffn_decode_kernel<0, 0>), reinterpret_cast<const void *>(ffn_decode_kernel<8, 0>),
                          reinterpret_cast<const void *>(ffn_decode_kernel<16, 0>), reinterpret_cast<const void *>(ffn_decode_kernel<0, 1>),
                          reinterpret_cast<const void *>(ffn_decode_kernel<8, 1>), reinterpret_cast<const void *>(ffn_decode_kernel<16, 1>)};
    for (const void *fn : fns) {
        cudaFuncAttributes fa;
        const cudaError_t e = cudaFuncGetAttributes(&fa, fn);
        if (e != cudaSuccess)
            return e;
        if (fa.sharedSizeBytes > stat)
            stat = fa.sharedSizeBytes;
    }
    const size_t usable = (max_smem - stat - 1024) / 128 * 128;
    for (const void *fn : fns) {
        const cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)usable);
        if (e != cudaSuccess)
            return e;
    }
    cfg->grid = n_sms < 255 ? n_sms : 255;   // one CTA per SM (the accumulator words count CTAs in one byte)
    cfg->max_smem = usable;
    cfg->pdl = pdl_enabled();
    return cudaSuccess;
}

cudaError_t ffn_decode_geometry(const DecLaunchCfg &cfg, int d, int F, int tokens, int fmt, DecGeometry *geo)
{
    if (!(fmt == 0 ? ffn_decode_supported(d, F) : fmt == 1 && ffn_decode_supported_q4(d, F)) || tokens < 1 || tokens > kTokPerVr)
        return cudaErrorInvalidValue;
    geo->n_warps = NW;
    // bytes of one hidden unit; pitch of the staged hidden rows (the pad keeps the fragment loads of neighbouring
    // tokens in different banks: 4-byte loads in the bf16 path, 16-byte loads in the 4-bit path)
    geo->row_bytes = fmt == 0 ? 6 * d : (3 * (d / 2) + 3 * (d / 64) * 2 + 15) / 16 * 16;
    geo->x_pitch = fmt == 0 ? 2 * d + 16 : 2 * d + 64;
    geo->tokens = tokens;
    // Wide models with many tokens: the hidden states would take a third of the shared memory and leave
    // room for tiles of two rows only, at which the per-tile work of the warps, not HBM, sets the pace.
    // Their operand fragments go to tensor memory instead.
    geo->x_tmem = fmt == 0 && d == 4096 && tokens > 4 ? 1 : 0;
    // staged hidden rows + the warps' partial tiles; the largest tile (at most 8 rows) of which two
    // stages fit beside them
    const size_t fixed = (geo->x_tmem ? 0 : (size_t)tokens * geo->x_pitch) + (size_t)(fmt == 0 ? 1 : 2) * NW * kBufPitch * sizeof(float);
    int tr = 8;
    for (;; --tr) {
        if (cfg.max_smem >= fixed + (size_t)2 * tr * geo->row_bytes)
            break;
        if (tr == 1)
            return cudaErrorInvalidConfiguration;
    }
    const size_t avail = cfg.max_smem - fixed;
    geo->tile_rows = tr;
    geo->stage_bytes = tr * geo->row_bytes;
    size_t n = avail / geo->stage_bytes;
    if (n > (size_t)kMaxStages)
        n = kMaxStages;
    geo->n_stages = (int)n;
    geo->smem_bytes = n * geo->stage_bytes + fixed;
    return cudaSuccess;
}

cudaError_t launch_ffn_decode(cudaStream_t stream, const DecLaunchCfg &cfg, const DecGeometry &geo, const DecParams &p)
{
    // Programmatic stream serialisation: the CTAs may be scheduled, and set up their barriers, while the
    // kernel ahead in the stream is still running; the kernel waits for the plan word before it reads
    // anything that kernel writes.  No CTA waits for another, so nothing depends on co-residency.
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(cfg.grid);
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = geo.smem_bytes;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    int na = 0;
    if (cfg.pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    lc.attrs = attr;
    lc.numAttrs = na;
    const int mt = p.d / (16 * NW);
    cudaError_t e;
    if (p.fmt == 0)
        e = mt == 8    ? cudaLaunchKernelEx(&lc, ffn_decode_kernel<8, 0>, p, geo)
            : mt == 16 ? (geo.x_tmem ? cudaLaunchKernelEx(&lc, ffn_decode_kernel<16, 0, 1>, p, geo)
                                     : cudaLaunchKernelEx(&lc, ffn_decode_kernel<16, 0>, p, geo))
                       : cudaLaunchKernelEx(&lc, ffn_decode_kernel<0, 0>, p, geo);
    else
        e = mt == 8    ? cudaLaunchKernelEx(&lc, ffn_decode_kernel<8, 1>, p, geo)
            : mt == 16 ? cudaLaunchKernelEx(&lc, ffn_decode_kernel<16, 1>, p, geo)
                       : cudaLaunchKernelEx(&lc, ffn_decode_kernel<0, 1>, p, geo);
    count_launch();
    return e;
}

}  // namespace melinoe
