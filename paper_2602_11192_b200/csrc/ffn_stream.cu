// Streaming SwiGLU expert FFN (Eq. 3) for calls with at most a few tokens per expert
// (decode): the work is reading every needed expert once from HBM, so the kernel is built
// around keeping the memory system full, not around arithmetic.
//
// Work decomposition.  A "virtual request" is one expert with up to 8 of its tokens.  Each
// virtual request is cut along d_ff into units of 8 rows; in the packed expert layout a unit
// is two contiguous byte ranges: 16 rows of [W_g; W_u] interleaved and 8 rows of W_d^T.  All
// units of the launch are split evenly over the CTAs (one per SM), so any number of experts
// loads every SM equally.  A CTA that covers only part of an expert writes a partial output
// row set; the combine kernel adds the partials in a fixed order.
//
// Per CTA: one producer warp issues bulk asynchronous copies (cp.async.bulk, completion on
// mbarriers) of weight rows into a shared-memory ring, far ahead of the math; eight consumer
// warps run the two small products with mma.sync (bf16 inputs, fp32 accumulation):
//   phase 1  [g;u] (16 rows) x hidden (<= 8 tokens): weights are the 8-wide operand, the
//            tokens the 16-wide one; each warp owns d/8 of the columns, partial sums meet in
//            shared memory, h = bf16(SiLU(g) * u);
//   phase 2  z += W_d^T rows (8) x h: each warp owns d/8 of the output columns and keeps its
//            accumulators in registers across all units of the virtual request.
// Weight rows land in shared memory at a pitch of 2*d + 16 bytes, which makes every ldmatrix
// access (plain for phase 1, transposed for phase 2) conflict-free.
//
// Every wait is bounded: if an mbarrier wait runs out, the CTA raises an abort flag, skips
// all later waits, finishes its loops without hanging and reports through the error word.
#include "kernels.cuh"

namespace melinoe {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kFfnThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStages = 16;
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
    if (*abort_flag)
        return false;
    if (mbar_try(bar, parity))
        return true;
    const unsigned long long t0 = globaltimer_ns();
    for (;;) {
        for (int i = 0; i < 256; ++i)
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

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2,
                                                  uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// D(16x8) += A(16x16) * B(16x8), bf16 in, fp32 accumulate.  Rows 8..15 of A are zero here.
__device__ __forceinline__ void mma_k16_top(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    const uint32_t z = 0u;
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(z), "r"(a2), "r"(z), "r"(b0), "r"(b1));
}

// D(16x8) += A(16x8) * B(8x8)
__device__ __forceinline__ void mma_k8(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0)
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(b0));
}

__device__ __forceinline__ uint32_t f32_to_bf16_rne_bits(float v)
{
    uint32_t u = __float_as_uint(v);
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

// KW = d / 8: the columns one consumer warp owns in both phases.
template <int KW>
__global__ void __launch_bounds__(kFfnThreads, 1)
ffn_stream_kernel(FfnParams p, int rpe, int ns)
{
    constexpr int KS2 = KW / 32;   // pairs of 16-wide k-steps in phase 1
    constexpr int MT2 = KW / 32;   // pairs of 16-row output tiles in phase 2

    extern __shared__ __align__(128) unsigned char smem[];
    const int d = p.d, F = p.F;
    const int P = 2 * d + 16;                    // smem pitch of one weight / hidden row
    const int row_bytes = 2 * d;
    const int entry_bytes = rpe * P;
    unsigned char *ring = smem;
    unsigned char *xs = ring + (size_t)ns * entry_bytes;
    float *s_part = reinterpret_cast<float *>(xs + 8 * P);
    uint32_t *s_h32 = reinterpret_cast<uint32_t *>(s_part + kConsumerWarps * 2 * 8 * 8);
    uint64_t *bars = reinterpret_cast<uint64_t *>(s_h32 + 32);
    volatile int *s_abort = reinterpret_cast<volatile int *>(bars + 2 * kMaxStages);

    const DevPlan *plan = p.plan;
    const int vr_begin = plan->group_vr_begin[p.group];
    const int nvr = plan->group_vr_begin[p.group + 1] - vr_begin;
    if (nvr <= 0)
        return;
    const int upe = F / kUnitRows;
    const long long NU = (long long)nvr * upe;
    // CTAs that share this launch: never more than there are units, so no CTA's range is empty
    const long long G = NU < (long long)gridDim.x ? NU : (long long)gridDim.x;
    if ((long long)blockIdx.x >= G)
        return;
    const long long u0 = (long long)blockIdx.x * NU / G;
    const long long u1 = (long long)(blockIdx.x + 1) * NU / G;
    if (u0 >= u1)
        return;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kMaxStages);
    if (tid == 0) {
        *s_abort = 0;
        for (int i = 0; i < ns; ++i) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full0 + 8 * i), "r"(1));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty0 + 8 * i), "r"(kConsumerWarps));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int epu = 24 / rpe;      // ring entries per unit
    const int gue = 16 / rpe;      // of which [W_g;W_u] rows
    const int half = 8 / rpe;      // entries per 8 rows
    const uint32_t ring_s = smem_u32(ring);

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            long long n = 0;
            bool stop = false;
            for (long long u = u0; u < u1 && !stop; ++u) {
                const int vr = vr_begin + (int)(u / upe);
                const int fb = (int)(u % upe) * kUnitRows;
                const ReqRec rec = plan->req[p.vrs[vr].req];
                const char *blob = rec.slot >= 0 ? p.slots + (size_t)rec.slot * p.slot_stride
                                                 : p.shared_blobs[rec.expert - p.E];
                const char *gu = blob + (size_t)(2 * fb) * row_bytes;
                const char *dt = blob + (size_t)(2 * F + fb) * row_bytes;
                for (int e = 0; e < epu; ++e, ++n) {
                    const int slot = (int)(n % ns);
                    if (n >= ns && !mbar_wait(empty0 + 8 * slot, (uint32_t)((n / ns - 1) & 1), s_abort)) {
                        stop = true;
                        break;
                    }
                    const char *src = e < gue ? gu + (size_t)e * rpe * row_bytes
                                              : dt + (size_t)(e - gue) * rpe * row_bytes;
                    const uint32_t bar = full0 + 8 * slot;
                    const uint32_t dst = ring_s + slot * entry_bytes;
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar),
                                 "r"(rpe * row_bytes)
                                 : "memory");
                    for (int r = 0; r < rpe; ++r) {
                        asm volatile(
                            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                            ::"r"(dst + r * P), "l"(src + (size_t)r * row_bytes), "r"(row_bytes), "r"(bar)
                            : "memory");
                    }
                }
            }
            if (stop) {
                // the consumers gave up or a wait ran out: let the copies already issued land
                // (bounded) before this CTA's shared memory goes away
                const long long first = n > ns ? n - ns : 0;
                const unsigned long long t0 = globaltimer_ns();
                for (long long m = first; m < n; ++m) {
                    const uint32_t bar = full0 + 8 * (int)(m % ns);
                    const uint32_t par = (uint32_t)((m / ns) & 1);
                    while (!mbar_try(bar, par) && globaltimer_ns() - t0 < kWaitLimitNs) {
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ consumers
        const int g = lane >> 2, tig = lane & 3;
        const int colbase = warp * KW;           // this warp's hidden columns / output columns
        float zacc[2 * MT2][4];
#pragma unroll
        for (int i = 0; i < 2 * MT2; ++i)
            zacc[i][0] = zacc[i][1] = zacc[i][2] = zacc[i][3] = 0.0f;
        const uint32_t xs_s = smem_u32(xs);
        float *my_part = s_part + warp * (2 * 8 * 8);
        int cur_vr = -1, cur_ntok = 0;

        auto flush = [&](int vr, int n_tok) {
            const long long prow = ((long long)p.group * gridDim.x + blockIdx.x + vr) * kTokPerVr;
            const int t0 = tig * 2;
#pragma unroll
            for (int mt = 0; mt < 2 * MT2; ++mt) {
                const int r = colbase + mt * 16 + g;
                if (t0 < n_tok) {
                    p.part[(prow + t0) * d + r] = zacc[mt][0];
                    p.part[(prow + t0) * d + r + 8] = zacc[mt][2];
                }
                if (t0 + 1 < n_tok) {
                    p.part[(prow + t0 + 1) * d + r] = zacc[mt][1];
                    p.part[(prow + t0 + 1) * d + r + 8] = zacc[mt][3];
                }
                zacc[mt][0] = zacc[mt][1] = zacc[mt][2] = zacc[mt][3] = 0.0f;
            }
        };

        for (long long u = u0; u < u1; ++u) {
            const int vr = vr_begin + (int)(u / upe);
            if (vr != cur_vr) {
                if (cur_vr >= 0)
                    flush(cur_vr, cur_ntok);
                const VrRec v = p.vrs[vr];
                // hidden rows of this virtual request's tokens -> shared memory (zero padded to 8)
                for (int t = 0; t < kTokPerVr; ++t) {
                    const int tok = t < v.n_tok ? p.tok_of_sorted[v.tok_off + t] : -1;
                    const uint4 *src = reinterpret_cast<const uint4 *>(p.x + (size_t)(tok < 0 ? 0 : tok) * d);
                    uint4 *dst = reinterpret_cast<uint4 *>(xs + t * P);
                    for (int i = tid; i < d / 8; i += kConsumerWarps * 32)
                        dst[i] = tok >= 0 ? src[i] : make_uint4(0, 0, 0, 0);
                }
                cur_vr = vr;
                cur_ntok = v.n_tok;
                consumer_bar();
            }
            const long long nb = (u - u0) * epu;

            // ---- phase 1: two blocks of 8 [W_g;W_u] rows
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
                for (int e = 0; e < half; ++e) {
                    const long long n = nb + blk * half + e;
                    mbar_wait(full0 + 8 * (int)(n % ns), (uint32_t)((n / ns) & 1), s_abort);
                }
                // lane's row for ldmatrix: unit-local row blk*8 + (lane & 7); k offset (lane >> 3) * 8
                const int li = blk * 8 + (lane & 7);
                const long long ne = nb + li / rpe;
                const uint32_t rowaddr = ring_s + (int)(ne % ns) * entry_bytes + (li % rpe) * P
                                         + (colbase + (lane >> 3) * 8) * 2;
                const uint32_t xaddr = xs_s + g * P + (colbase + tig * 2) * 2;
                float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int ks = 0; ks < KS2; ++ks) {
                    uint32_t b00, b01, b10, b11;
                    ldmatrix_x4(rowaddr + ks * 64, b00, b01, b10, b11);
                    uint32_t a0, a2, a0n, a2n;
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(a0) : "r"(xaddr + ks * 64));
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(a2) : "r"(xaddr + ks * 64 + 16));
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(a0n) : "r"(xaddr + ks * 64 + 32));
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(a2n) : "r"(xaddr + ks * 64 + 48));
                    mma_k16_top(c, a0, a2, b00, b01);
                    mma_k16_top(c, a0n, a2n, b10, b11);
                }
                __syncwarp();
                if (lane == 0)
                    for (int e = 0; e < half; ++e)
                        mbar_arrive(empty0 + 8 * (int)((nb + blk * half + e) % ns));
                // c[0], c[1]: token g, rows tig*2 and tig*2+1 of this block (g_f and u_f, f = tig)
                *reinterpret_cast<float2 *>(my_part + (blk * 8 + g) * 8 + tig * 2) = make_float2(c[0], c[1]);
            }
            consumer_bar();
            if (tid < 64) {
                const int t = tid >> 3, f = tid & 7, blk = f >> 2, fl = f & 3;
                float gs = 0.0f, us = 0.0f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float2 v = *reinterpret_cast<const float2 *>(s_part + w * 128 + (blk * 8 + t) * 8 + fl * 2);
                    gs += v.x;
                    us += v.y;
                }
                const float h = gs / (1.0f + __expf(-gs)) * us;
                reinterpret_cast<uint16_t *>(s_h32)[t * 8 + f] = (uint16_t)f32_to_bf16_rne_bits(h);
            }
            consumer_bar();

            // ---- phase 2: 8 rows of W_d^T
            for (int e = 0; e < half; ++e) {
                const long long n = nb + gue + e;
                mbar_wait(full0 + 8 * (int)(n % ns), (uint32_t)((n / ns) & 1), s_abort);
            }
            {
                const int li = lane & 7;                       // W_d^T row of the unit
                const long long ne = nb + gue + li / rpe;
                const uint32_t rowaddr = ring_s + (int)(ne % ns) * entry_bytes + (li % rpe) * P
                                         + (colbase + (lane >> 3) * 8) * 2;
                const uint32_t b0 = s_h32[g * 4 + tig];        // h[f = tig*2, tig*2+1][token g]
#pragma unroll
                for (int mt = 0; mt < MT2; ++mt) {
                    uint32_t a00, a01, a10, a11;
                    ldmatrix_x4_trans(rowaddr + mt * 64, a00, a01, a10, a11);
                    mma_k8(zacc[2 * mt], a00, a01, b0);
                    mma_k8(zacc[2 * mt + 1], a10, a11, b0);
                }
                __syncwarp();
                if (lane == 0)
                    for (int e = 0; e < half; ++e)
                        mbar_arrive(empty0 + 8 * (int)((nb + gue + e) % ns));
            }
        }
        if (cur_vr >= 0)
            flush(cur_vr, cur_ntok);
        if (*s_abort && tid == 0)
            atomicExch(p.err, MELINOE_ERR_TIMEOUT);
    }
}

template <int KW>
cudaError_t launch_kw(cudaStream_t stream, const FfnLaunchCfg &cfg, const FfnParams &p)
{
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(ffn_stream_kernel<KW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)cfg.smem_bytes);
        if (e != cudaSuccess)
            return e;
        attr_set = true;
    }
    ffn_stream_kernel<KW><<<cfg.grid, kFfnThreads, cfg.smem_bytes, stream>>>(p, cfg.rows_per_entry, cfg.n_stages);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool ffn_stream_supported(int d)
{
    switch (d) {
    case 256: case 512: case 1024: case 2048: case 3072: case 4096:
        return true;
    default:
        return false;
    }
}

cudaError_t ffn_stream_configure(int d, int n_sms, size_t max_smem, FfnLaunchCfg *cfg)
{
    if (!ffn_stream_supported(d))
        return cudaErrorInvalidValue;
    const size_t P = 2 * (size_t)d + 16;
    const size_t fixed = 8 * P + kConsumerWarps * 2 * 8 * 8 * sizeof(float) + 128 + 2 * kMaxStages * 8 + 16;
    int best_rpe = 1, best_ns = 0;
    for (int rpe = 8; rpe >= 1; rpe >>= 1) {
        if (max_smem <= fixed)
            break;
        int ns = (int)((max_smem - fixed) / (rpe * P));
        if (ns > kMaxStages)
            ns = kMaxStages;
        best_rpe = rpe;
        best_ns = ns;
        if (ns >= 6)
            break;
    }
    // a unit holds at most 8 rows at a time; the ring must cover that plus copies in flight
    if (best_ns * best_rpe < 16)
        return cudaErrorInvalidConfiguration;
    cfg->grid = n_sms;
    cfg->rows_per_entry = best_rpe;
    cfg->n_stages = best_ns;
    cfg->smem_bytes = fixed + (size_t)best_ns * best_rpe * P;
    return cudaSuccess;
}

cudaError_t launch_ffn_stream(cudaStream_t stream, const FfnLaunchCfg &cfg, const FfnParams &p)
{
    switch (p.d) {
    case 256: return launch_kw<32>(stream, cfg, p);
    case 512: return launch_kw<64>(stream, cfg, p);
    case 1024: return launch_kw<128>(stream, cfg, p);
    case 2048: return launch_kw<256>(stream, cfg, p);
    case 3072: return launch_kw<384>(stream, cfg, p);
    case 4096: return launch_kw<512>(stream, cfg, p);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace melinoe
