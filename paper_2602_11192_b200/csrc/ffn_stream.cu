// Streaming SwiGLU expert FFN (Eq. 3) with the gate-weighted combine (Eq. 2) fused in, for
// calls with few tokens per expert (decode).  The work is reading every needed expert once
// from HBM, so the kernel is built around keeping the memory system full.
//
// One cooperative launch per compute group, one CTA per SM, eight independent warps per CTA.
// A "virtual request" is one expert with up to 8 of its tokens.
//
//   phase 1  tile = 8 rows of W_g plus the same 8 rows of W_u of one virtual request.
//            D[16 x 8] = [W_g rows; W_u rows] (16 x d) * x^T (d x 8 tokens) on mma.sync
//            (bf16 in, fp32 accumulate).  In the accumulator layout a thread holds g_f and u_f
//            of the same f and the same two tokens, so h = SiLU(g) * u is thread-local;
//            h goes to global memory as bf16.
//   barrier  grid-wide (bounded spin on a device counter); before waiting, each warp already
//            has the first W_d stages of its phase-2 work in flight.
//   phase 2  tile = 16 rows of W_d of one virtual request: D[16 x 8] = W_d rows (16 x F) * h^T.
//            Every tile is a complete dot product over d_ff, so z needs no cross-CTA reduction
//            and goes to z[pair][d] in fp32.
//   combine  the warp that finishes the last tile of a 16-row block in the call's last
//            compute group sums gate * z over the ranks in rank order (plus shared experts)
//            and writes the bf16 output rows.  The result does not depend on which warp does
//            it, nor on how the experts were split over groups.
//
// Data movement: every warp owns a private ring of S stages in shared memory.  A stage holds
// a KC-column slice of the tile's 16 weight rows plus the matching slice of up to 8 operand rows
// (hidden rows in phase 1, h rows in phase 2), each fetched by its own cp.async.bulk (one lane
// per row) completing on the stage's mbarrier.  Rows sit at a pitch of 2*KC+16 bytes, which
// makes the ldmatrix reads and the operand-fragment reads bank-conflict free.  There is no
// CTA-wide synchronisation after start-up.
//
// Every wait is bounded: when an mbarrier or the grid barrier does not complete in time the
// warp raises the CTA's abort flag, later waits fall through, the kernel ends normally and the
// error word tells the host.
#include <cooperative_groups.h>

#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kStageRows = 24;            // 16 weight rows + 8 operand rows
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

__device__ __forceinline__ void mbar_expect(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// What a warp needs to know about the tile it fetches or computes.
struct Tile {
    const char *src;     // this lane's source row (weights: lanes 0..15, operand rows: lanes 16..23)
    int n_tok;           // tokens of the virtual request
    int vr;              // virtual request (index within the call)
    int blk;             // f-block (phase 1) or 16-row block (phase 2)
};

template <int KC, int S>
__global__ void __launch_bounds__(kThreads, 1) ffn_stream_kernel(FfnParams p)
{
    constexpr int PITCH = 2 * KC + 16;
    constexpr int STAGE = kStageRows * PITCH;
    constexpr int KSTEPS = KC / 16;

    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, tig = lane & 3;
    const int d = p.d, F = p.F, Fpad = p.Fpad;
    const DevPlan *plan = p.plan;
    const int G = (int)gridDim.x;

    if (plan->status != MELINOE_OK) {
        // the call was refused on the device: the output is all zeros, the status tells why
        if (p.group == 0)
            for (size_t i = (size_t)blockIdx.x * kThreads + tid; i < (size_t)p.T * d; i += (size_t)G * kThreads)
                p.out[i] = 0;
        return;
    }
    const int vb = plan->group_vr_begin[p.group];
    const int nv = plan->group_vr_begin[p.group + 1] - vb;
    const bool final_group = p.group == plan->n_groups - 1;
    if (nv <= 0 && !final_group)
        return;

    unsigned char *ring = smem + (size_t)warp * S * STAGE;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)kWarps * S * STAGE) + warp * S;
    const uint32_t ring_s = smem_u32(ring), bar_s = smem_u32(bars);
    volatile int *abort_flag = &s_abort;

    if (tid == 0)
        s_abort = 0;
    if (lane == 0) {
        for (int i = 0; i < S; ++i)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar_s + 8 * i), "r"(1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (F % KC != 0) {
        // the last d_ff slice of a W_d row is shorter than a stage row: what it leaves untouched
        // must be finite, because it meets zeros of the padded h rows in the product
        uint4 *z = reinterpret_cast<uint4 *>(ring);
        for (int i = lane; i < S * STAGE / 16; i += 32)
            z[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async();
    }
    __syncthreads();

    // ---- this warp's tiles: a contiguous range per CTA, dealt round-robin to its warps
    const int upe1 = F / 8, upe2 = d / 16;
    const int nk1 = d / KC, nk2 = (F + KC - 1) / KC;
    const long long NT1 = (long long)nv * upe1, NT2 = (long long)nv * upe2;
    const int lo1 = (int)(blockIdx.x * NT1 / G) + warp, hi1 = (int)((blockIdx.x + 1) * NT1 / G);
    const int lo2 = (int)(blockIdx.x * NT2 / G) + warp, hi2 = (int)((blockIdx.x + 1) * NT2 / G);

    auto blob_of = [&](const VrRec &v) -> const char * {
        const ReqRec rec = plan->req[v.req];
        return rec.slot >= 0 ? p.slots + (size_t)rec.slot * p.slot_stride : p.shared_blobs[rec.expert - p.E];
    };
    // lane's source row for a phase-1 tile: lanes 0..7 W_g rows, 8..15 W_u rows, 16..23 hidden rows
    auto tile1 = [&](int t) -> Tile {
        Tile ti;
        ti.vr = vb + t / upe1;
        ti.blk = t % upe1;
        const VrRec v = p.vrs[ti.vr];
        ti.n_tok = v.n_tok;
        ti.src = nullptr;
        if (lane < 16) {
            const int row = (lane < 8 ? 0 : F) + ti.blk * 8 + (lane & 7);
            ti.src = blob_of(v) + (size_t)row * d * 2;
        } else if (lane - 16 < v.n_tok) {
            const int tok = p.tok_of_sorted[v.tok_off + lane - 16];
            ti.src = reinterpret_cast<const char *>(p.x) + (size_t)tok * d * 2;
        }
        return ti;
    };
    // phase 2: lanes 0..15 W_d rows, 16..23 rows of h
    auto tile2 = [&](int t) -> Tile {
        Tile ti;
        ti.vr = vb + t / upe2;
        ti.blk = t % upe2;
        const VrRec v = p.vrs[ti.vr];
        ti.n_tok = v.n_tok;
        ti.src = nullptr;
        if (lane < 16)
            ti.src = blob_of(v) + ((size_t)2 * F * d + (size_t)(ti.blk * 16 + lane) * F) * 2;
        else if (lane - 16 < v.n_tok)
            ti.src = reinterpret_cast<const char *>(p.hbuf) + ((size_t)ti.vr * kTokPerVr + lane - 16) * Fpad * 2;
        return ti;
    };

    uint32_t n_issued = 0, n_consumed = 0;   // stages, over both phases (ring slot and parity)

    // issue one stage: parts bit 0 = weight rows and the barrier's byte count, bit 1 = operand rows
    auto issue = [&](const Tile &ti, int kc, int wbytes, int parts, uint32_t n) {
        const uint32_t slot = n % S;
        const uint32_t bar = bar_s + 8 * slot;
        if ((parts & 1) && lane == 0)
            mbar_expect(bar, 16u * wbytes + (uint32_t)ti.n_tok * KC * 2);
        __syncwarp();
        if (ti.src) {
            const bool is_w = lane < 16;
            if (is_w ? (parts & 1) : (parts & 2))
                bulk_g2s(ring_s + slot * STAGE + lane * PITCH, ti.src + (size_t)kc * KC * 2,
                         is_w ? (uint32_t)wbytes : (uint32_t)(KC * 2), bar);
        }
    };

    // the mma loop over one stage
    const uint32_t a_off = ((lane & 7) + ((lane >> 3) & 1) * 8) * PITCH + (lane >> 4) * 16;
    const uint32_t b_off = (16 + g) * PITCH + tig * 4;
    auto compute = [&](uint32_t n, int n_tok, float (&c0)[4], float (&c1)[4]) {
        const uint32_t slot = n % S;
        mbar_wait(bar_s + 8 * slot, (n / S) & 1u, abort_flag);
        const uint32_t base = ring_s + slot * STAGE;
        const bool has_tok = g < n_tok;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ks += 2) {
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
        __syncwarp();
    };

    // =========================================================== phase 1: h = SiLU(W_g x) * (W_u x)
    {
        int pt = lo1, pk = 0, ct = lo1, ck = 0;
        Tile ptile{}, ctile{};
        if (pt < hi1)
            ptile = tile1(pt);
        ctile = ptile;
        for (int i = 0; i < S && pt < hi1; ++i) {
            issue(ptile, pk, KC * 2, 3, n_issued++);
            if (++pk == nk1) {
                pk = 0;
                pt += kWarps;
                if (pt < hi1)
                    ptile = tile1(pt);
            }
        }
        float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
        while (ct < hi1) {
            compute(n_consumed++, ctile.n_tok, c0, c1);
            if (pt < hi1) {
                issue(ptile, pk, KC * 2, 3, n_issued++);
                if (++pk == nk1) {
                    pk = 0;
                    pt += kWarps;
                    if (pt < hi1)
                        ptile = tile1(pt);
                }
            }
            if (++ck == nk1) {
                // rows g and g + 8 of the tile are g_f and u_f for f = 8 * blk + g
                const int f = ctile.blk * 8 + g;
                const float gv0 = c0[0] + c1[0], gv1 = c0[1] + c1[1], uv0 = c0[2] + c1[2], uv1 = c0[3] + c1[3];
                uint16_t *hrow = p.hbuf + ((size_t)ctile.vr * kTokPerVr) * Fpad + f;
                if (tig * 2 < ctile.n_tok)
                    hrow[(size_t)(tig * 2) * Fpad] = bf16_rne(gv0 / (1.0f + __expf(-gv0)) * uv0);
                if (tig * 2 + 1 < ctile.n_tok)
                    hrow[(size_t)(tig * 2 + 1) * Fpad] = bf16_rne(gv1 / (1.0f + __expf(-gv1)) * uv1);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    c0[i] = c1[i] = 0.f;
                ck = 0;
                ct += kWarps;
                if (ct < hi1)
                    ctile = tile1(ct);
            }
        }
    }

    // =========================================================== grid barrier, W_d already in flight
    __threadfence();
    fence_proxy_async();       // h was written through the generic proxy, bulk copies will read it
    __syncwarp();
    if (lane == 0)
        atomicAdd(p.sync + p.group, 1u);
    int pt = lo2, pk = 0;
    Tile ptile{};
    if (pt < hi2)
        ptile = tile2(pt);
    auto wbytes2 = [&](int kc) { return 2 * min(KC, F - kc * KC); };
    {
        // first stages of phase 2: weight rows only; their h rows follow once h is complete
        int qt = pt, qk = pk;
        Tile qtile = ptile;
        const uint32_t n0 = n_issued;
        int pre = 0;
        for (; pre < S && pt < hi2; ++pre) {
            issue(ptile, pk, wbytes2(pk), 1, n_issued++);
            if (++pk == nk2) {
                pk = 0;
                pt += kWarps;
                if (pt < hi2)
                    ptile = tile2(pt);
            }
        }
        if (lane == 0) {
            const unsigned target = (unsigned)G * kWarps;
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
        }
        __syncwarp();
        fence_proxy_async();
        for (int i = 0; i < pre; ++i) {
            issue(qtile, qk, 0, 2, n0 + i);
            if (++qk == nk2) {
                qk = 0;
                qt += kWarps;
                if (qt < hi2)
                    qtile = tile2(qt);
            }
        }
    }

    // =========================================================== phase 2: z = W_d h, then the combine
    {
        int ct = lo2, ck = 0;
        Tile ctile{};
        if (ct < hi2)
            ctile = tile2(ct);
        float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
        const int n_pairs = p.T * p.k;
        while (ct < hi2) {
            compute(n_consumed++, ctile.n_tok, c0, c1);
            if (pt < hi2) {
                issue(ptile, pk, wbytes2(pk), 3, n_issued++);
                if (++pk == nk2) {
                    pk = 0;
                    pt += kWarps;
                    if (pt < hi2)
                        ptile = tile2(pt);
                }
            }
            if (++ck == nk2) {
                const VrRec v = p.vrs[ctile.vr];
                const int r = ctile.blk * 16 + g;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int ts = tig * 2 + h;
                    if (ts < ctile.n_tok) {
                        const int pos = v.tok_off + ts;
                        const int pair = pos < n_pairs ? p.perm[pos] : pos;
                        float *zr = p.zbuf + (size_t)pair * d + r;
                        zr[0] = c0[h] + c1[h];
                        zr[8] = c0[2 + h] + c1[2 + h];
                    }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    c0[i] = c1[i] = 0.f;
                if (final_group) {
                    // count the finished tiles of this 16-row block; the last one combines it
                    unsigned old = 0;
                    __threadfence();
                    __syncwarp();
                    if (lane == 0)
                        old = atomicAdd(p.row_done + ctile.blk, 1u);
                    old = __shfl_sync(0xffffffffu, old, 0);
                    if (old == (unsigned)nv - 1u) {
                        __threadfence();
                        const int row = ctile.blk * 16 + (lane & 15);
                        for (int t = lane >> 4; t < p.T; t += 2) {
                            float y = 0.f;
                            for (int j = 0; j < p.k; ++j)
                                y = fmaf(p.gate[t * p.k + j], __ldcg(p.zbuf + (size_t)(t * p.k + j) * d + row), y);
                            for (int s = 0; s < p.n_shared; ++s)
                                y += __ldcg(p.zbuf + (size_t)(n_pairs + s * p.T + t) * d + row);
                            p.out[(size_t)t * d + row] = bf16_rne(y);
                        }
                        if (lane == 0)
                            p.row_done[ctile.blk] = 0;
                    }
                }
                ck = 0;
                ct += kWarps;
                if (ct < hi2)
                    ctile = tile2(ct);
            }
        }
    }
    if (final_group && nv <= 0) {
        // nothing computed in the last group (cannot happen for a well-formed plan): combine all rows
        const int n_pairs = p.T * p.k;
        for (int blk = blockIdx.x * kWarps + warp; blk < upe2; blk += G * kWarps) {
            const int row = blk * 16 + (lane & 15);
            for (int t = lane >> 4; t < p.T; t += 2) {
                float y = 0.f;
                for (int j = 0; j < p.k; ++j)
                    y = fmaf(p.gate[t * p.k + j], __ldcg(p.zbuf + (size_t)(t * p.k + j) * d + row), y);
                for (int s = 0; s < p.n_shared; ++s)
                    y += __ldcg(p.zbuf + (size_t)(n_pairs + s * p.T + t) * d + row);
                p.out[(size_t)t * d + row] = bf16_rne(y);
            }
        }
    }
    __syncwarp();
    if (*abort_flag && lane == 0) {
        // a wait ran out: give the copies this warp still has in flight a bounded time to land
        // before its shared memory goes away, then report
        const unsigned long long t0 = globaltimer_ns();
        const uint32_t first = n_issued > (uint32_t)S ? n_issued - S : 0u;
        for (uint32_t n = first; n < n_issued; ++n)
            while (!mbar_try(bar_s + 8 * (n % S), (n / S) & 1u) && globaltimer_ns() - t0 < kWaitLimitNs) {
            }
        atomicExch(p.err, MELINOE_ERR_TIMEOUT);
    }
}

constexpr int kKC = 128;
constexpr int kS = 4;

}  // namespace

cudaError_t ffn_stream_configure(int n_sms, size_t max_smem, FfnLaunchCfg *cfg)
{
    const size_t need = (size_t)kWarps * kS * kStageRows * (2 * kKC + 16) + (size_t)kWarps * kS * 8 + 64;
    if (need > max_smem)
        return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(ffn_stream_kernel<kKC, kS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)need);
    if (e != cudaSuccess)
        return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ffn_stream_kernel<kKC, kS>, kThreads, need);
    if (e != cudaSuccess)
        return e;
    if (per_sm < 1)
        return cudaErrorInvalidConfiguration;
    cfg->grid = n_sms;          // one CTA per SM: all of them resident, which the grid barrier needs
    cfg->smem_bytes = need;
    return cudaSuccess;
}

cudaError_t launch_ffn_stream(cudaStream_t stream, const FfnLaunchCfg &cfg, const FfnParams &p)
{
    FfnParams q = p;
    void *args[] = {&q};
    cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(ffn_stream_kernel<kKC, kS>),
                                                dim3(cfg.grid), dim3(kThreads), args, cfg.smem_bytes, stream);
    count_launch();
    return e;
}

}  // namespace melinoe
