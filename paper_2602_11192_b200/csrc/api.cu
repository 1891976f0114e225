// Host side of the C ABI: handle management, launch sequencing, and the miss path that turns
// the device-written miss queue into cudaMemcpyAsync calls on a side copy stream.
//
// One forward call on the caller's stream:
//   router -> plan -> FFN(group 0: experts resident at call entry)
//   -> [host reads the miss queue; per miss wave: copies on the copy stream, event] ->
//   wait(event) FFN(group 1) -> ...   (the last group's FFN kernel also does the combine).
// Group 0 is queued before the host knows the plan, so resident experts compute while the
// miss queue travels to the host and while the transfers run.  Every cross-stream dependency
// is a CUDA event (copy stream -> compute stream for arrival, compute stream -> copy stream
// when a wave overwrites a slot that an earlier group of the same call still reads), so the
// ordering is visible to the driver and cannot deadlock however streams share hardware queues.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "kernels.cuh"

using namespace melinoe;

namespace melinoe {

static std::atomic<long long> g_launches{0};
// Test hook (melinoe_debug_fail_host_copy): when positive, counts down once per host-issued expert copy;
// the copy at which it reaches zero is not issued and reports a failure instead.  Host-side only.
static std::atomic<int> g_fail_copy_in{0};
static cudaError_t g_copy_hook()
{
    if (g_fail_copy_in.load() > 0 && g_fail_copy_in.fetch_sub(1) == 1)
        return cudaErrorUnknown;
    return cudaSuccess;
}
static std::atomic<int> g_last_cuda_error{0};

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

bool pdl_enabled()
{
    static const bool on = std::getenv("MELINOE_MOE_NO_PDL") == nullptr;
    return on;
}

}  // namespace melinoe

namespace {

int cuda_fail(cudaError_t e)
{
    g_last_cuda_error.store((int)e);
    (void)cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? MELINOE_ERR_NOMEM : MELINOE_ERR_CUDA;
}

#define CU_TRY(expr)                      \
    do {                                  \
        cudaError_t e__ = (expr);         \
        if (e__ != cudaSuccess)           \
            return cuda_fail(e__);        \
    } while (0)

typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
encode_tiled_fn g_encode_tiled = nullptr;
std::once_flag g_encode_once;

// 2-D bf16 tensor [rows][cols] with rows pitch_bytes apart, box of box_rows x 64 columns; with or
// without the 128-byte swizzle (the expert blobs are stored already permuted, see melinoe_moe_pack_expert).
bool encode_map(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes, uint32_t box_rows,
                bool swizzle)
{
    std::call_once(g_encode_once, [] {
        cudaDriverEntryPointQueryResult qr;
        void *fn = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            g_encode_tiled = reinterpret_cast<encode_tiled_fn>(fn);
        (void)cudaGetLastError();
    });
    if (!g_encode_tiled || rows == 0)
        return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {pitch_bytes};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return g_encode_tiled(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The three views of expert blobs that lie back to back from `base` (n_rows = experts * F rows f):
// W_g rows, W_u rows (boxes of 128 rows), W_d^T rows (boxes of 64 rows), all d columns at a pitch of 6 d bytes.
bool encode_weight_maps(CUtensorMap *m3, const void *base, int d, uint64_t n_rows)
{
    const char *b = static_cast<const char *>(base);
    const uint64_t pitch = (uint64_t)6 * d;
    return encode_map(m3 + 0, b, d, n_rows, pitch, 128, false) && encode_map(m3 + 1, b + (size_t)2 * d, d, n_rows, pitch, 128, false) &&
           encode_map(m3 + 2, b + (size_t)4 * d, d, n_rows, pitch, 64, false);
}

double now_s()
{
    return std::chrono::duration<double>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

struct TimedPair {
    cudaEvent_t a, b;
};

}  // namespace

// Scratch of one forward call.  idx .. tok_of_sorted: routing and gather tables; yacc: the decode
// kernel's output accumulator [<= 8 tokens][d] (64-bit words, all zero between launches); ybuf: fp32
// sums of a call that is computed in several launches.
struct Scratch {
    int32_t *idx = nullptr, *perm = nullptr, *inv_pos = nullptr, *tok_of_sorted = nullptr;
    float *gate = nullptr, *logits = nullptr, *ybuf = nullptr;
    long long *yacc = nullptr;
    int cap_tokens = 0;
};

struct melinoe_moe {
    int d = 0, F = 0, E = 0, k = 0, C = 0, device = 0, n_sms = 0;
    size_t expert_bytes = 0, slot_stride = 0;
    int fmt = 0;                           // what the slots hold: 0 = bf16 blobs, 1 = 4-bit blobs
    DecLaunchCfg cfg{};

    // device memory owned by the handle
    char *slots = nullptr;
    DevCache *cache = nullptr;
    int policy = MELINOE_POLICY_LRU;   // eviction policy, see melinoe_moe_set_policy
    float gamma = 0.0f;
    DevPlan *plan = nullptr;
    int *err_word = nullptr;
    const char **shared_dev = nullptr;
    const char **host_dev = nullptr;       // [E]: the host store's blobs as the device sees them (null: not readable)
    bool pull_ok = false;                  // the decode kernel may read missed experts straight from the host store

    // per-call scratch: the handle's own (sized for cap_tokens), and whichever the most recent call used
    Scratch own{}, last{};
    int cap_shared = -1;
    float *zbuf = nullptr;                 // grouped-GEMM path: expert outputs [sorted rows][d] fp32
    unsigned *sync = nullptr;              // counter of the decode kernel's rare "who is last" step (zero between launches)
    unsigned long long *trace = nullptr;   // borrowed; see melinoe_moe_set_timeline
    char *req_trace = nullptr;             // borrowed; see melinoe_moe_set_trace
    size_t req_trace_cap = 0;              // records it holds
    int req_trace_tokens = 0;
    long long req_trace_count = 0;
    uint16_t *stage_in = nullptr, *stage_out = nullptr;
    // grouped-GEMM path (calls of more than 8 tokens): gathered activations, h, tensor maps
    bool gemm_ok = false, last_used_gemm = false;
    uint16_t *xs = nullptr, *hs = nullptr;
    CUtensorMap *maps_dev = nullptr;
    CUtensorMap maps_host[kMapCount];
    const void *shared_ptrs[kMaxShared] = {nullptr};
    melinoe_moe_stats *stage_stats = nullptr;

    // borrowed
    const uint16_t *w_router = nullptr;
    const float *bias = nullptr;
    const int32_t *token_seq = nullptr;
    int n_seq = 0, n_shared = 0;
    std::vector<const void *> host_experts;
    // 4-bit host store (melinoe_moe_register_host_experts_q4): what travels is the 4-bit blob, a
    // kernel on the copy stream expands it from this staging buffer into the bf16 slot
    bool store_q4 = false;
    size_t q4_bytes = 0;
    char *q4_stage = nullptr;              // two staging buffers of q4_bytes, used alternately
    cudaStream_t dq_stream = nullptr;      // runs the expansion kernels, so the link does not wait for them
    cudaEvent_t ev_q4_copied[2] = {nullptr, nullptr}, ev_q4_expanded[2] = {nullptr, nullptr};
    unsigned q4_turn = 0;                  // staging buffer of the next miss
    bool q4_used[2] = {false, false};

    // page-locked host memory: the miss queue the planning kernel writes
    HostPlan *hplan = nullptr;
    // preload: the fetch list (device, and page-locked host copy), its event on the copy stream
    PreloadList *pre_dev = nullptr, *pre_host = nullptr;
    cudaEvent_t ev_preload = nullptr;
    bool preload_pending = false;       // the next forward call has to wait for ev_preload
    uint32_t preload_seq = 0;

    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_last = nullptr;      // end of the most recent call on the caller's stream
    cudaEvent_t ev_plan = nullptr;      // caller's stream: the planning kernel of the current call is done
    cudaEvent_t ev_arrive = nullptr;    // copy stream: a wave's transfers have landed
    std::vector<cudaEvent_t> ev_group;  // compute stream: FFN group g of the current call is done
    bool has_last = false;
    uint32_t call_seq = 0;
    int last_T = 0;
    std::atomic<int> sticky{0};

    // kernel timing
    bool timing = false;
    std::vector<TimedPair> timed, free_pairs, timed_copy;
    uint64_t timed_copy_bytes = 0;
};

namespace {

// ---------------------------------------------------------------- helpers

void init_cache_host(DevCache &c)
{
    std::memset(&c, 0, sizeof c);
    for (int i = 0; i < kMaxExperts; ++i) {
        c.expert_of_slot[i] = -1;
        c.slot_of_expert[i] = -1;
    }
}

int gmax_for(const melinoe_moe *h, int T)
{
    long long u = (long long)T * h->k;
    if (u > h->E)
        u = h->E;
    if (h->policy == MELINOE_POLICY_COUNT)
        return 1 + (int)u;     // every miss may be a wave of its own
    return 1 + (int)((u + h->C - 1) / h->C);
}

void free_scratch(melinoe_moe *h)
{
    Scratch &o = h->own;
    cudaFree(o.idx);
    cudaFree(o.perm);
    cudaFree(o.inv_pos);
    cudaFree(o.tok_of_sorted);
    cudaFree(o.gate);
    cudaFree(o.logits);
    cudaFree(o.yacc);
    cudaFree(o.ybuf);
    cudaFree(h->zbuf);
    cudaFree(h->stage_in);
    cudaFree(h->stage_out);
    cudaFree(h->xs);
    cudaFree(h->hs);
    h->xs = h->hs = nullptr;
    o = Scratch{};
    h->last = Scratch{};
    h->zbuf = nullptr;
    h->stage_in = h->stage_out = nullptr;
}

int wait_idle(melinoe_moe *h)
{
    if (h->has_last)
        CU_TRY(cudaEventSynchronize(h->ev_last));
    CU_TRY(cudaStreamSynchronize(h->copy_stream));
    if (h->dq_stream)
        CU_TRY(cudaStreamSynchronize(h->dq_stream));
    return MELINOE_OK;
}

// Bounded host wait for the planning kernel of call `seq` to publish its miss queue.
// ev_plan was recorded right behind that kernel.
int wait_for_plan(melinoe_moe *h, uint32_t seq)
{
    volatile uint32_t *w = &h->hplan->hdr.seq;
    for (int i = 0; i < 4096; ++i)
        if (*w == seq)
            return MELINOE_OK;
    const double t0 = now_s();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (*w == seq)
                return MELINOE_OK;
        const double dt = now_s() - t0;
        if (dt > 60.0)
            return MELINOE_ERR_TIMEOUT;
        if (dt > 0.001) {
            // a long queue ahead of this call: stop burning the core, and notice a dead stream
            std::this_thread::yield();
            const cudaError_t q = cudaEventQuery(h->ev_plan);
            if (q == cudaSuccess)
                return *w == seq ? MELINOE_OK : MELINOE_ERR_STATE;  // kernel done, record absent
            if (q != cudaErrorNotReady)
                return cuda_fail(q);
        }
    }
}

int ensure_capacity(melinoe_moe *h, int T)
{
    if (T <= h->own.cap_tokens && h->cap_shared == h->n_shared)
        return MELINOE_OK;
    int rc = wait_idle(h);
    if (rc != MELINOE_OK)
        return rc;
    CU_TRY(cudaDeviceSynchronize());
    const int cap = T > h->own.cap_tokens ? T : h->own.cap_tokens;
    free_scratch(h);
    Scratch &o = h->own;
    const size_t pairs = (size_t)cap * h->k;
    const size_t sorted = pairs + (size_t)h->n_shared * cap;
    const int launch_tokens = cap < kTokPerVr ? cap : kTokPerVr;
    CU_TRY(cudaMalloc(&o.idx, pairs * 4));
    CU_TRY(cudaMalloc(&o.gate, pairs * 4));
    CU_TRY(cudaMalloc(&o.logits, (size_t)cap * h->E * 4));
    CU_TRY(cudaMalloc(&o.perm, sorted * 4));
    CU_TRY(cudaMalloc(&o.inv_pos, pairs * 4));
    CU_TRY(cudaMalloc(&o.tok_of_sorted, sorted * 4));
    CU_TRY(cudaMalloc(&o.yacc, (size_t)launch_tokens * h->d * sizeof(long long)));
    CU_TRY(cudaMemset(o.yacc, 0, (size_t)launch_tokens * h->d * sizeof(long long)));
    CU_TRY(cudaMalloc(&o.ybuf, (size_t)cap * h->d * sizeof(float)));
    CU_TRY(cudaMalloc(&h->stage_in, (size_t)cap * h->d * 2));
    CU_TRY(cudaMalloc(&h->stage_out, (size_t)cap * h->d * 2));
    if (h->gemm_ok && cap > kTokPerVr) {
        CU_TRY(cudaMalloc(&h->zbuf, sorted * h->d * sizeof(float)));
        CU_TRY(cudaMalloc(&h->xs, sorted * h->d * 2));
        CU_TRY(cudaMalloc(&h->hs, sorted * h->F * 2));
        if (!encode_map(&h->maps_host[kMapXs], h->xs, h->d, sorted, (uint64_t)h->d * 2, 128, true) ||
            !encode_map(&h->maps_host[kMapHs], h->hs, h->F, sorted, (uint64_t)h->F * 2, 128, true))
            return MELINOE_ERR_CUDA;
        CU_TRY(cudaMemcpy(h->maps_dev, h->maps_host, sizeof(h->maps_host), cudaMemcpyHostToDevice));
    }
    o.cap_tokens = cap;
    h->cap_shared = h->n_shared;
    return MELINOE_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

// ---------------------------------------------------------------- C ABI

extern "C" {

const char *melinoe_strerror(int status)
{
    switch (status) {
    case MELINOE_OK: return "ok";
    case MELINOE_ERR_INVALID: return "invalid argument";
    case MELINOE_ERR_STATE: return "call out of order or inconsistent state";
    case MELINOE_ERR_CUDA: return "CUDA call failed";
    case MELINOE_ERR_NOMEM: return "out of memory";
    case MELINOE_ERR_TIMEOUT: return "bounded wait ran out";
    case MELINOE_ERR_UNSUPPORTED: return "shape not supported";
    default: return "unknown status";
    }
}

int64_t melinoe_launch_count(void) { return (int64_t)g_launches.load(); }
int melinoe_last_cuda_error(void) { return g_last_cuda_error.load(); }

size_t melinoe_moe_expert_bytes(int d_model, int d_ff)
{
    if (d_model <= 0 || d_ff <= 0)
        return 0;
    return (size_t)3 * (size_t)d_model * (size_t)d_ff * 2;
}

int melinoe_moe_pack_expert(int d, int F, const void *wg_, const void *wu_, const void *wd_, void *blob_)
{
    if (d <= 0 || F <= 0 || !wg_ || !wu_ || !wd_ || !blob_)
        return MELINOE_ERR_INVALID;
    if (d % 64 != 0)
        return MELINOE_ERR_UNSUPPORTED;
    const uint16_t *wg = static_cast<const uint16_t *>(wg_), *wu = static_cast<const uint16_t *>(wu_);
    const uint16_t *wd = static_cast<const uint16_t *>(wd_);
    uint16_t *blob = static_cast<uint16_t *>(blob_);
    // per hidden unit f: W_g[f][:] | W_u[f][:] | W_d[:][f]; 8-element (16-byte) pieces of every 64-element
    // (128-byte) group at position (piece xor (f mod 8))
    for (int f = 0; f < F; ++f) {
        uint16_t *row = blob + (size_t)f * 3 * d;
        const int x = f & 7;
        for (int j = 0; j < d / 8; ++j) {
            const int pj = (j & ~7) | ((j ^ x) & 7);
            std::memcpy(row + (size_t)pj * 8, wg + (size_t)f * d + (size_t)j * 8, 16);
            std::memcpy(row + d + (size_t)pj * 8, wu + (size_t)f * d + (size_t)j * 8, 16);
        }
    }
    // W_d transposed in 8 x 8 blocks (8 output columns c by 8 hidden units f), so that both the reads and
    // the writes move 16 contiguous bytes; F need not be a multiple of 8 here, the tail goes element-wise
    const int F8 = F & ~7;
    for (int j = 0; j < d / 8; ++j) {
        for (int f0 = 0; f0 < F8; f0 += 8) {
            uint16_t t[8][8];
            for (int i = 0; i < 8; ++i)
                std::memcpy(t[i], wd + (size_t)(j * 8 + i) * F + f0, 16);
            for (int r = 0; r < 8; ++r) {
                const int f = f0 + r;
                const int pj = (j & ~7) | ((j ^ (f & 7)) & 7);
                uint16_t *dst = blob + (size_t)f * 3 * d + 2 * (size_t)d + (size_t)pj * 8;
                for (int i = 0; i < 8; ++i)
                    dst[i] = t[i][r];
            }
        }
        for (int f = F8; f < F; ++f) {
            const int pj = (j & ~7) | ((j ^ (f & 7)) & 7);
            uint16_t *dst = blob + (size_t)f * 3 * d + 2 * (size_t)d + (size_t)pj * 8;
            for (int i = 0; i < 8; ++i)
                dst[i] = wd[(size_t)(j * 8 + i) * F + f];
        }
    }
    return MELINOE_OK;
}

// Bytes of one hidden unit's part of a 4-bit blob: three rows of d codes (d / 2 bytes each), three rows of
// d / 64 bf16 scales, rounded up to 16 bytes (bulk copies move multiples of 16 bytes).
static size_t q4_unit_bytes(int d) { return ((size_t)3 * (d / 2) + (size_t)3 * (d / 64) * 2 + 15) / 16 * 16; }

size_t melinoe_moe_expert_bytes_q4(int d_model, int d_ff)
{
    if (d_model <= 0 || d_ff <= 0 || d_model % 256 != 0 || d_ff % kUnitRows != 0)
        return 0;
    return (size_t)d_ff * q4_unit_bytes(d_model);
}

namespace {

float host_bf16_to_f32(uint16_t b)
{
    const uint32_t u = (uint32_t)b << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return f;
}

uint16_t host_f32_to_bf16(float f)
{
    uint32_t u;
    std::memcpy(&u, &f, sizeof u);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

// One vector of d values (read at stride `stride`) into d / 2 code bytes and d / 64 scales: groups of 64
// consecutive values, scale = bf16(max|w| / 7), code = clamp(rint(w / scale), -8, 7) + 8, ties to even.  The
// 16-byte pieces of the codes (32 codes each) go to position (piece xor x) within every group of 8 pieces.
// interleave: element i of a group sits at code position 8 * (i mod 8) + i / 8 of the group instead of i.
void pack_q4_vector(const uint16_t *w, size_t stride, int d, int x, bool interleave, unsigned char *codes, uint16_t *scales)
{
    for (int g = 0; g < d / 64; ++g) {
        float amax = 0.0f;
        for (int j = 0; j < 64; ++j)
            amax = std::fmax(amax, std::fabs(host_bf16_to_f32(w[(size_t)(g * 64 + j) * stride])));
        const uint16_t sb = host_f32_to_bf16(amax / 7.0f);
        const float sc = host_bf16_to_f32(sb);
        scales[g] = sb;
        for (int j = 0; j < 64; j += 2) {       // code positions j, j + 1 of the group share a byte
            int q[2] = {0, 0};
            for (int h2 = 0; h2 < 2; ++h2)
                if (sc > 0.0f) {
                    const int pos = j + h2, i = interleave ? 8 * (pos % 8) + pos / 8 : pos;     // the element at this position
                    const float t = std::nearbyint(host_bf16_to_f32(w[(size_t)(g * 64 + i) * stride]) / sc);   // ties to even
                    q[h2] = (int)std::fmin(7.0f, std::fmax(-8.0f, t));
                }
            const int byte = (g * 64 + j) / 2, piece = byte / 16;
            const int ppiece = (piece & ~7) | ((piece ^ x) & 7);
            codes[ppiece * 16 + byte % 16] = (unsigned char)((q[0] + 8) | ((q[1] + 8) << 4));
        }
    }
}

}  // namespace

int melinoe_moe_pack_expert_q4(int d, int F, const void *wg_, const void *wu_, const void *wd_, void *blob_)
{
    if (d <= 0 || F <= 0 || !wg_ || !wu_ || !wd_ || !blob_)
        return MELINOE_ERR_INVALID;
    if (melinoe_moe_expert_bytes_q4(d, F) == 0)
        return MELINOE_ERR_UNSUPPORTED;
    const uint16_t *wg = static_cast<const uint16_t *>(wg_), *wu = static_cast<const uint16_t *>(wu_);
    const uint16_t *wd = static_cast<const uint16_t *>(wd_);
    unsigned char *blob = static_cast<unsigned char *>(blob_);
    const size_t ub = q4_unit_bytes(d);
    for (int f = 0; f < F; ++f) {
        unsigned char *u = blob + (size_t)f * ub;
        std::memset(u, 0, ub);
        uint16_t *sc = reinterpret_cast<uint16_t *>(u + 3 * (size_t)(d / 2));
        pack_q4_vector(wg + (size_t)f * d, 1, d, f & 7, false, u, sc);
        pack_q4_vector(wu + (size_t)f * d, 1, d, f & 7, false, u + d / 2, sc + d / 64);
        pack_q4_vector(wd + f, (size_t)F, d, f & 7, true, u + 2 * (size_t)(d / 2), sc + 2 * (d / 64));    // column f of W_d
    }
    return MELINOE_OK;
}

static int create_layer(int d, int F, int E, int k, int C, int fmt, melinoe_moe_t **out);

int melinoe_moe_create(int d, int F, int E, int k, int C, melinoe_moe_t **out) { return create_layer(d, F, E, k, C, 0, out); }

int melinoe_moe_create_q4(int d, int F, int E, int k, int C, melinoe_moe_t **out) { return create_layer(d, F, E, k, C, 1, out); }

static int create_layer(int d, int F, int E, int k, int C, int fmt, melinoe_moe_t **out)
{
    if (!out)
        return MELINOE_ERR_INVALID;
    *out = nullptr;
    if (d <= 0 || F <= 0 || E <= 0 || k <= 0 || C <= 0 || k > E || C < k || C > E)
        return MELINOE_ERR_INVALID;
    if (!(fmt == 0 ? ffn_decode_supported(d, F) : ffn_decode_supported_q4(d, F)) || E > kMaxExperts || k > 32)
        return MELINOE_ERR_UNSUPPORTED;
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess)
            e = cudaFree(0);
        if (e != cudaSuccess)
            return cuda_fail(e);  // no usable device: there is no other execution path
    }
    melinoe_moe *h = new (std::nothrow) melinoe_moe();
    if (!h)
        return MELINOE_ERR_NOMEM;
    h->d = d;
    h->F = F;
    h->E = E;
    h->k = k;
    h->C = C;
    h->fmt = fmt;
    h->expert_bytes = fmt == 0 ? melinoe_moe_expert_bytes(d, F) : melinoe_moe_expert_bytes_q4(d, F);
    h->slot_stride = (h->expert_bytes + 1023) / 1024 * 1024;
    h->host_experts.assign(E, nullptr);
    int rc = MELINOE_OK;
    auto fail = [&](int code) {
        melinoe_moe_destroy(h);
        return code;
    };
    cudaDeviceProp prop;
    if (cudaGetDevice(&h->device) != cudaSuccess || cudaGetDeviceProperties(&prop, h->device) != cudaSuccess)
        return fail(cuda_fail(cudaGetLastError()));
    if (prop.major != 10)
        return fail(MELINOE_ERR_UNSUPPORTED);
    h->n_sms = prop.multiProcessorCount;
    if (ffn_decode_configure(h->n_sms, prop.sharedMemPerBlockOptin, &h->cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        return fail(MELINOE_ERR_UNSUPPORTED);
    }
#define CR(expr)                                   \
    do {                                           \
        cudaError_t e__ = (expr);                  \
        if (e__ != cudaSuccess)                    \
            return fail(cuda_fail(e__));           \
    } while (0)
    CR(cudaMalloc(&h->slots, h->slot_stride * (size_t)C));
    CR(cudaMalloc(&h->cache, sizeof(DevCache)));
    CR(cudaMalloc(&h->plan, sizeof(DevPlan)));
    CR(cudaMalloc(&h->err_word, 256));
    CR(cudaMalloc(&h->sync, 256));
    CR(cudaMemset(h->sync, 0, 256));
    CR(cudaMalloc(&h->shared_dev, sizeof(char *) * kMaxShared));
    CR(cudaMalloc(&h->host_dev, sizeof(char *) * kMaxExperts));
    CR(cudaMemset(h->host_dev, 0, sizeof(char *) * kMaxExperts));
    CR(cudaMalloc(&h->stage_stats, sizeof(melinoe_moe_stats)));
    CR(cudaMemset(h->err_word, 0, 256));
    CR(cudaMemset(h->plan, 0, sizeof(DevPlan)));
    CR(cudaMemset(h->shared_dev, 0, sizeof(char *) * kMaxShared));
    DevCache c0;
    init_cache_host(c0);
    CR(cudaMemcpy(h->cache, &c0, sizeof c0, cudaMemcpyHostToDevice));
    CR(cudaHostAlloc(&h->hplan, sizeof(HostPlan), cudaHostAllocMapped | cudaHostAllocPortable));
    std::memset(h->hplan, 0, sizeof(HostPlan));
    CR(cudaMalloc(&h->pre_dev, sizeof(PreloadList)));
    CR(cudaMemset(h->pre_dev, 0, sizeof(PreloadList)));
    CR(cudaHostAlloc(&h->pre_host, sizeof(PreloadList), cudaHostAllocMapped | cudaHostAllocPortable));
    std::memset(h->pre_host, 0, sizeof(PreloadList));
    CR(cudaEventCreateWithFlags(&h->ev_preload, cudaEventDisableTiming));
    CR(cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
    CR(cudaEventCreateWithFlags(&h->ev_last, cudaEventDisableTiming));
    CR(cudaEventCreateWithFlags(&h->ev_plan, cudaEventDisableTiming));
    CR(cudaEventCreateWithFlags(&h->ev_arrive, cudaEventDisableTiming));
    // one event per compute group a call can have, made here so that no forward call ever creates one
    h->ev_group.assign(kMaxGroups + 1, nullptr);
    for (auto &e : h->ev_group)
        CR(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    // grouped GEMM for calls of many tokens: the slots are contiguous, so one tensor map per view
    // (W_g rows, W_u rows, W_d^T rows) covers every slot
    std::memset(h->maps_host, 0, sizeof(h->maps_host));
    if (fmt == 0 && ffn_gemm_supported(d, F) && h->slot_stride == h->expert_bytes && ffn_gemm_configure() == cudaSuccess) {
        CR(cudaMalloc(&h->maps_dev, sizeof(h->maps_host)));
        if (encode_weight_maps(&h->maps_host[kMapSlotsG], h->slots, d, (uint64_t)C * F)) {
            CR(cudaMemcpy(h->maps_dev, h->maps_host, sizeof(h->maps_host), cudaMemcpyHostToDevice));
            h->gemm_ok = true;
        }
    }
    (void)cudaGetLastError();
#undef CR
    (void)rc;
    *out = h;
    return MELINOE_OK;
}

int melinoe_moe_destroy(melinoe_moe_t *h)
{
    if (!h)
        return MELINOE_OK;
    int rc = MELINOE_OK;
    if (h->copy_stream)
        rc = wait_idle(h);
    free_scratch(h);
    cudaFree(h->slots);
    cudaFree(h->cache);
    cudaFree(h->plan);
    cudaFree(h->err_word);
    cudaFree(h->sync);
    cudaFree(h->q4_stage);
    if (h->dq_stream)
        cudaStreamDestroy(h->dq_stream);
    for (int i = 0; i < 2; ++i) {
        if (h->ev_q4_copied[i])
            cudaEventDestroy(h->ev_q4_copied[i]);
        if (h->ev_q4_expanded[i])
            cudaEventDestroy(h->ev_q4_expanded[i]);
    }
    cudaFree(h->shared_dev);
    cudaFree(h->host_dev);
    cudaFree(h->maps_dev);
    cudaFree(h->stage_stats);
    if (h->hplan)
        cudaFreeHost(h->hplan);
    cudaFree(h->pre_dev);
    if (h->pre_host)
        cudaFreeHost(h->pre_host);
    if (h->ev_preload)
        cudaEventDestroy(h->ev_preload);
    if (h->copy_stream)
        cudaStreamDestroy(h->copy_stream);
    if (h->ev_last)
        cudaEventDestroy(h->ev_last);
    if (h->ev_plan)
        cudaEventDestroy(h->ev_plan);
    if (h->ev_arrive)
        cudaEventDestroy(h->ev_arrive);
    for (cudaEvent_t e : h->ev_group)
        cudaEventDestroy(e);
    for (auto &p : h->timed) {
        cudaEventDestroy(p.a);
        cudaEventDestroy(p.b);
    }
    for (auto &p : h->free_pairs) {
        cudaEventDestroy(p.a);
        cudaEventDestroy(p.b);
    }
    for (auto &p : h->timed_copy) {
        cudaEventDestroy(p.a);
        cudaEventDestroy(p.b);
    }
    (void)cudaGetLastError();
    delete h;
    return rc;
}

int melinoe_moe_set_router(melinoe_moe_t *h, const void *w_router_dev)
{
    if (!h || !w_router_dev || !aligned16(w_router_dev))
        return MELINOE_ERR_INVALID;
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, w_router_dev) != cudaSuccess || a.type != cudaMemoryTypeDevice) {
        (void)cudaGetLastError();
        return MELINOE_ERR_INVALID;
    }
    h->w_router = static_cast<const uint16_t *>(w_router_dev);
    return MELINOE_OK;
}

static int register_store(melinoe_moe *h, const void *const *ptrs, size_t bytes_per_expert);

int melinoe_moe_register_host_experts(melinoe_moe_t *h, const void *const *ptrs, size_t bytes_per_expert)
{
    if (!h || !ptrs)
        return MELINOE_ERR_INVALID;
    if (h->fmt != 0)
        return MELINOE_ERR_UNSUPPORTED;   // 4-bit slots are filled from a 4-bit store
    return register_store(h, ptrs, bytes_per_expert);
}

// The store holds blobs of the slots' own format: a miss is a plain copy, by the device where it can
// address the store.
static int register_store(melinoe_moe *h, const void *const *ptrs, size_t bytes_per_expert)
{
    if (bytes_per_expert != h->expert_bytes)
        return MELINOE_ERR_INVALID;
    for (int e = 0; e < h->E; ++e) {
        if (!ptrs[e] || !aligned16(ptrs[e]))
            return MELINOE_ERR_INVALID;
        cudaPointerAttributes a;
        if (cudaPointerGetAttributes(&a, ptrs[e]) != cudaSuccess || a.type != cudaMemoryTypeHost) {
            (void)cudaGetLastError();
            return MELINOE_ERR_INVALID;  // pageable (or device) memory: never staged silently
        }
    }
    int rc = wait_idle(h);
    if (rc != MELINOE_OK)
        return rc;
    // the store as the device sees it: the decode kernel reads missed experts from there itself
    const char *dev_view[kMaxExperts] = {nullptr};
    bool all = true;
    for (int e = 0; e < h->E; ++e) {
        void *dp = nullptr;
        if (cudaHostGetDevicePointer(&dp, const_cast<void *>(ptrs[e]), 0) != cudaSuccess || !dp || !aligned16(dp)) {
            (void)cudaGetLastError();
            all = false;
            break;
        }
        dev_view[e] = static_cast<const char *>(dp);
    }
    if (!all)
        std::memset(dev_view, 0, sizeof dev_view);
    CU_TRY(cudaMemcpy(h->host_dev, dev_view, sizeof dev_view, cudaMemcpyHostToDevice));
    h->pull_ok = all && std::getenv("MELINOE_MOE_HOST_COPIES") == nullptr;
    for (int e = 0; e < h->E; ++e)
        h->host_experts[e] = ptrs[e];
    h->store_q4 = false;
    return MELINOE_OK;
}

int melinoe_moe_register_host_experts_q4(melinoe_moe_t *h, const void *const *ptrs, size_t bytes_per_expert)
{
    if (!h || !ptrs)
        return MELINOE_ERR_INVALID;
    const size_t qb = melinoe_moe_expert_bytes_q4(h->d, h->F);
    if (qb == 0)
        return MELINOE_ERR_UNSUPPORTED;
    if (bytes_per_expert != qb)
        return MELINOE_ERR_INVALID;
    if (h->fmt == 1)
        return register_store(h, ptrs, bytes_per_expert);
    for (int e = 0; e < h->E; ++e) {
        cudaPointerAttributes a;
        if (!ptrs[e] || !aligned16(ptrs[e]) || cudaPointerGetAttributes(&a, ptrs[e]) != cudaSuccess ||
            a.type != cudaMemoryTypeHost) {
            (void)cudaGetLastError();
            return MELINOE_ERR_INVALID;
        }
    }
    int rc = wait_idle(h);
    if (rc != MELINOE_OK)
        return rc;
    if (!h->q4_stage) {
        CU_TRY(cudaMalloc(&h->q4_stage, 2 * qb));
        CU_TRY(cudaStreamCreateWithFlags(&h->dq_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            CU_TRY(cudaEventCreateWithFlags(&h->ev_q4_copied[i], cudaEventDisableTiming));
            CU_TRY(cudaEventCreateWithFlags(&h->ev_q4_expanded[i], cudaEventDisableTiming));
        }
    }
    for (int e = 0; e < h->E; ++e)
        h->host_experts[e] = ptrs[e];
    CU_TRY(cudaMemset(h->host_dev, 0, sizeof(char *) * kMaxExperts));
    h->pull_ok = false;     // 4-bit blobs are expanded into the bf16 slots by a kernel behind the copy
    h->store_q4 = true;
    h->q4_bytes = qb;
    return MELINOE_OK;
}

int melinoe_moe_register_shared_experts(melinoe_moe_t *h, int n_shared, const void *const *ptrs)
{
    if (!h || n_shared < 0 || n_shared > kMaxShared || (n_shared > 0 && !ptrs))
        return MELINOE_ERR_INVALID;
    for (int s = 0; s < n_shared; ++s) {
        cudaPointerAttributes a;
        if (!ptrs[s] || !aligned16(ptrs[s]) || cudaPointerGetAttributes(&a, ptrs[s]) != cudaSuccess ||
            a.type != cudaMemoryTypeDevice) {
            (void)cudaGetLastError();
            return MELINOE_ERR_INVALID;
        }
    }
    int rc = wait_idle(h);
    if (rc != MELINOE_OK)
        return rc;
    const char *tmp[kMaxShared] = {nullptr};
    for (int s = 0; s < n_shared; ++s)
        tmp[s] = static_cast<const char *>(ptrs[s]);
    CU_TRY(cudaMemcpy(h->shared_dev, tmp, sizeof tmp, cudaMemcpyHostToDevice));
    if (h->gemm_ok) {
        for (int s = 0; s < n_shared; ++s)
            if (!encode_weight_maps(&h->maps_host[kMapShared0 + 3 * s], ptrs[s], h->d, (uint64_t)h->F))
                return MELINOE_ERR_CUDA;
        CU_TRY(cudaMemcpy(h->maps_dev, h->maps_host, sizeof(h->maps_host), cudaMemcpyHostToDevice));
    }
    h->n_shared = n_shared;
    return MELINOE_OK;
}

int melinoe_moe_set_router_bias(melinoe_moe_t *h, const float *seq_bias_dev, const int32_t *token_seq_dev,
                                int n_seq)
{
    if (!h || (seq_bias_dev && n_seq <= 0))
        return MELINOE_ERR_INVALID;
    h->bias = seq_bias_dev;
    h->token_seq = seq_bias_dev ? token_seq_dev : nullptr;
    h->n_seq = seq_bias_dev ? n_seq : 0;
    return MELINOE_OK;
}

int melinoe_moe_reserve(melinoe_moe_t *h, int max_tokens)
{
    if (!h || max_tokens <= 0)
        return MELINOE_ERR_INVALID;
    return ensure_capacity(h, max_tokens);
}

}  // extern "C"

namespace {

// Event pair for kernel timing, reused from the handle's pool.
int take_pair(melinoe_moe *h, TimedPair *tp)
{
    if (!h->free_pairs.empty()) {
        *tp = h->free_pairs.back();
        h->free_pairs.pop_back();
        return MELINOE_OK;
    }
    CU_TRY(cudaEventCreate(&tp->a));
    CU_TRY(cudaEventCreate(&tp->b));
    return MELINOE_OK;
}

// One launch of the decode FFN kernel: compute group `group` (or -1: the whole call, missed experts
// read from the host store) for tokens [8 * chunk, 8 * chunk + 8) of the call.
int launch_decode(melinoe_moe *h, cudaStream_t s, const Scratch &sc, const void *hidden_dev, void *out_dev, int T,
                  int group, int chunk, bool first_of_call)
{
    const int tokens = T - chunk * kTokPerVr < kTokPerVr ? T - chunk * kTokPerVr : kTokPerVr;
    DecGeometry geo;
    if (ffn_decode_geometry(h->cfg, h->d, h->F, tokens, h->fmt, &geo) != cudaSuccess)
        return MELINOE_ERR_UNSUPPORTED;
    DecParams dp;
    dp.plan = h->plan;
    dp.x = static_cast<const uint16_t *>(hidden_dev);
    dp.idx = sc.idx;
    dp.gate = sc.gate;
    dp.yacc = sc.yacc;
    dp.ybuf = sc.ybuf;
    dp.out = static_cast<uint16_t *>(out_dev);
    dp.sync = h->sync;
    dp.call_seq = h->call_seq;
    dp.err = h->err_word;
    dp.trace = h->trace;
    dp.d = h->d;
    dp.F = h->F;
    dp.E = h->E;
    dp.k = h->k;
    dp.T = T;
    dp.n_shared = h->n_shared;
    dp.group = group;
    dp.chunk = chunk;
    dp.n_chunks = (T + kTokPerVr - 1) / kTokPerVr;
    dp.write_back = 1;
    dp.wait_prior = first_of_call ? 0 : 1;
    dp.fmt = h->fmt;
    CU_TRY(launch_ffn_decode(s, h->cfg, geo, dp));
    return MELINOE_OK;
}

// The call itself, on the scratch it is given.
int forward_on(melinoe_moe *h, const Scratch &sc, void *cuda_stream, const void *hidden_dev, int T, void *out_dev,
               melinoe_moe_stats *stats_dev)
{
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (h->preload_pending) {
        // a preload is queued on the copy stream: this call's kernels come after it
        CU_TRY(cudaStreamWaitEvent(s, h->ev_preload, 0));
        h->preload_pending = false;
    }
    const uint32_t gmax = (uint32_t)gmax_for(h, T);
    h->call_seq += 1;
    h->last_T = T;
    h->last = sc;

    PlanParams pp;
    pp.idx = sc.idx;
    pp.T = T;
    pp.k = h->k;
    pp.E = h->E;
    pp.C = h->C;
    pp.n_shared = h->n_shared;
    pp.cache = h->cache;
    pp.plan = h->plan;
    pp.slots = h->slots;
    pp.slot_stride = h->slot_stride;
    pp.shared_blobs = h->shared_dev;
    pp.host_blobs = h->host_dev;
    pp.perm = sc.perm;
    pp.inv_pos = sc.inv_pos;
    pp.tok_of_sorted = sc.tok_of_sorted;
    pp.hplan = h->hplan;
    pp.gmax = gmax;
    pp.call_seq = h->call_seq;
    pp.policy = h->policy;
    pp.gamma = h->gamma;
    pp.stats = stats_dev;
    pp.expert_bytes = h->store_q4 ? h->q4_bytes : h->expert_bytes;   // bytes one miss moves over the host link
    pp.gate = sc.gate;
    pp.trace_rec = nullptr;
    pp.trace_max_tokens = h->req_trace_tokens;
    if (h->req_trace) {
        const TraceLayout tl = trace_layout(h->E, h->k, h->req_trace_tokens);
        pp.trace_rec = h->req_trace + (size_t)(h->req_trace_count % (long long)h->req_trace_cap) * tl.bytes;
        h->req_trace_count += 1;
    }
    const bool small = route_plan_small_supported(T, h->k, h->d);
    if (small) {
        CU_TRY(launch_route_plan_small(s, static_cast<const uint16_t *>(hidden_dev), h->w_router, h->bias, h->token_seq,
                                       h->d, sc.idx, sc.gate, sc.logits, pp));
    } else {
        CU_TRY(launch_router(s, static_cast<const uint16_t *>(hidden_dev), h->w_router, h->bias, h->token_seq, T, h->d,
                             h->E, h->k, sc.idx, sc.gate, sc.logits));
        CU_TRY(launch_plan(s, pp));
    }
    // calls of more than 8 tokens go through the grouped GEMM (where the shapes allow it)
    const bool use_gemm = h->gemm_ok && T > kTokPerVr && h->xs != nullptr && sc.idx == h->own.idx;
    const int n_chunks = (T + kTokPerVr - 1) / kTokPerVr;
    h->last_used_gemm = use_gemm;

    // ---- everything on the device: the decode kernel fetches the missed experts itself, the host is
    // not in the path at all and returns at once (the call's cache decisions are in stats_dev)
    // (Only where the call cannot need more distinct experts than there are slots: otherwise a fetched
    // expert may have to take the slot of an expert the same call still computes with, which needs an
    // order between the SMs that only separate launches give; those calls take the path below.)
    if (!use_gemm && h->pull_ok && (long long)T * h->k <= h->C) {
        for (int c = 0; c < n_chunks; ++c) {
            TimedPair tp{nullptr, nullptr};
            if (h->timing) {
                int rc = take_pair(h, &tp);
                if (rc != MELINOE_OK)
                    return rc;
                CU_TRY(cudaEventRecord(tp.a, s));
            }
            int rc = launch_decode(h, s, sc, hidden_dev, out_dev, T, -1, c, c == 0);
            if (rc != MELINOE_OK)
                return rc;
            if (h->timing) {
                CU_TRY(cudaEventRecord(tp.b, s));
                h->timed.push_back(tp);
            }
        }
        CU_TRY(cudaEventRecord(h->ev_last, s));
        h->has_last = true;
        return MELINOE_OK;
    }

    // ---- transfers issued by the host: group 0 is queued at once, the miss waves follow as the host
    // learns of them
    CU_TRY(cudaEventRecord(h->ev_plan, s));
    GemmParams gp;
    gp.plan = h->plan;
    gp.maps = h->maps_dev;
    gp.hs = h->hs;
    gp.zs = h->zbuf;
    gp.err = h->err_word;
    gp.d = h->d;
    gp.F = h->F;
    gp.E = h->E;
    gp.n_shared = h->n_shared;
    if (use_gemm)
        CU_TRY(launch_gather_rows(s, h->plan, static_cast<const uint16_t *>(hidden_dev), sc.tok_of_sorted, h->xs, h->d,
                                  T * h->k + h->n_shared * T, h->n_sms));
    auto launch_group = [&](int g) -> int {
        TimedPair tp{nullptr, nullptr};
        if (h->timing) {
            int rc = take_pair(h, &tp);
            if (rc != MELINOE_OK)
                return rc;
            CU_TRY(cudaEventRecord(tp.a, s));
        }
        if (use_gemm) {
            gp.group = g;
            // CTA pairs share one weight tile over two m-tiles: worth it where an expert has several m-tiles
            // (on average at least two here); MELINOE_MOE_GEMM_SINGLE in the environment keeps the single-CTA form
            static const bool single_only = std::getenv("MELINOE_MOE_GEMM_SINGLE") != nullptr;
            const bool pairs = !single_only && (long long)T * h->k >= 256ll * h->E;
            CU_TRY(launch_ffn_gemm(s, 1, h->n_sms, pairs, gp));
            CU_TRY(launch_ffn_gemm(s, 2, h->n_sms, pairs, gp));
        } else {
            for (int c = 0; c < n_chunks; ++c) {
                int rc = launch_decode(h, s, sc, hidden_dev, out_dev, T, g, c, g == 0 && c == 0);
                if (rc != MELINOE_OK)
                    return rc;
            }
        }
        if (h->timing) {
            CU_TRY(cudaEventRecord(tp.b, s));
            h->timed.push_back(tp);
        }
        return MELINOE_OK;
    };
    // From here on part of the call is queued: a failure must leave the stream and the handle in a
    // state the caller can see (ev_last recorded, the error sticky until the cache is reset).
    auto fail = [&](int code) -> int {
        h->sticky.store(code);
        (void)cudaEventRecord(h->ev_last, s);
        h->has_last = true;
        return code;
    };
    // group 0 (experts resident at call entry, shared experts) goes out before the plan is known
    int rc = launch_group(0);
    if (rc != MELINOE_OK)
        return fail(rc);

    // the miss queue of this call
    rc = wait_for_plan(h, h->call_seq);
    if (rc != MELINOE_OK)
        return fail(rc);
    const volatile HostPlan &vhp = *h->hplan;
    int n_miss = vhp.hdr.n_miss, n_groups = vhp.hdr.n_groups;
    if (vhp.hdr.status != MELINOE_OK || n_miss < 0 || n_miss > h->E || n_groups < 1 || n_groups > (int)gmax)
        n_miss = 0, n_groups = 1;  // the device-side status already tells the caller; nothing to fetch
    // every miss record carries the call's sequence number: take a copy once they have all arrived
    struct {
        HostMiss miss[kMaxExperts];
    } hp;
    for (int i = 0; i < n_miss; ++i) {
        const double t0 = now_s();
        for (;;) {
            HostMiss m;
            m.expert = vhp.miss[i].expert;
            m.slot = vhp.miss[i].slot;
            m.group = vhp.miss[i].group;
            m.dep_group = vhp.miss[i].dep_group;
            m.seq = vhp.miss[i].seq;
            if (m.seq == h->call_seq && vhp.miss[i].expert == m.expert && vhp.miss[i].slot == m.slot) {
                hp.miss[i] = m;
                break;
            }
            if (now_s() - t0 > 10.0)
                return fail(MELINOE_ERR_TIMEOUT);
        }
    }
    // which groups must signal their completion to the copy stream
    bool need_done[kMaxGroups + 1] = {false};
    for (int i = 0; i < n_miss; ++i)
        if (hp.miss[i].dep_group >= 0 && hp.miss[i].dep_group <= kMaxGroups)
            need_done[hp.miss[i].dep_group] = true;
    if (need_done[0])
        CU_TRY(cudaEventRecord(h->ev_group[0], s));
    int i = 0;
    for (int g = 1; g < n_groups; ++g) {
        TimedPair ctp{nullptr, nullptr};
        bool wave_started = false;
        for (; i < n_miss && hp.miss[i].group == g; ++i) {
            const HostMiss m = hp.miss[i];
            if (m.expert < 0 || m.expert >= h->E || m.slot < 0 || m.slot >= h->C || m.dep_group >= g)
                return fail(MELINOE_ERR_STATE);
            // the slot may still feed an earlier compute group of this call: whoever writes the slot
            // (the copy itself, or the expansion kernel of a 4-bit store) waits for that group
            cudaStream_t slot_writer = h->store_q4 ? h->dq_stream : h->copy_stream;
            cudaError_t ce = cudaSuccess;
            if (m.dep_group >= 0)
                ce = cudaStreamWaitEvent(slot_writer, h->ev_group[m.dep_group], 0);
            if (ce == cudaSuccess && h->timing && !wave_started) {
                rc = take_pair(h, &ctp);
                if (rc != MELINOE_OK)
                    return fail(rc);
                ce = cudaEventRecord(ctp.a, h->copy_stream);
                wave_started = true;
            }
            if (h->timing)
                h->timed_copy_bytes += h->store_q4 ? h->q4_bytes : h->expert_bytes;
            if (ce == cudaSuccess && h->store_q4) {
                // the 4-bit blob travels into one of two staging buffers; a kernel on a stream of its own
                // expands it into the slot, so the next blob is on the link meanwhile
                const unsigned b = h->q4_turn++ & 1u;
                char *stage = h->q4_stage + (size_t)b * h->q4_bytes;
                if (h->q4_used[b])
                    ce = cudaStreamWaitEvent(h->copy_stream, h->ev_q4_expanded[b], 0);
                if (ce == cudaSuccess)
                    ce = g_copy_hook();
                if (ce == cudaSuccess)
                    ce = cudaMemcpyAsync(stage, h->host_experts[m.expert], h->q4_bytes, cudaMemcpyHostToDevice, h->copy_stream);
                if (ce == cudaSuccess)
                    ce = cudaEventRecord(h->ev_q4_copied[b], h->copy_stream);
                if (ce == cudaSuccess)
                    ce = cudaStreamWaitEvent(h->dq_stream, h->ev_q4_copied[b], 0);
                if (ce == cudaSuccess)
                    ce = launch_dequant_q4(h->dq_stream, stage, h->slots + (size_t)m.slot * h->slot_stride, h->d, h->F, h->n_sms);
                if (ce == cudaSuccess)
                    ce = cudaEventRecord(h->ev_q4_expanded[b], h->dq_stream);
                h->q4_used[b] = true;
            } else if (ce == cudaSuccess) {
                ce = g_copy_hook();
                if (ce == cudaSuccess)
                    ce = cudaMemcpyAsync(h->slots + (size_t)m.slot * h->slot_stride, h->host_experts[m.expert], h->expert_bytes,
                                         cudaMemcpyHostToDevice, h->copy_stream);
            }
            if (ce != cudaSuccess)
                return fail(cuda_fail(ce));
        }
        if (wave_started) {
            CU_TRY(cudaEventRecord(ctp.b, h->copy_stream));
            h->timed_copy.push_back(ctp);
        }
        cudaError_t ce = cudaEventRecord(h->ev_arrive, h->store_q4 ? h->dq_stream : h->copy_stream);
        if (ce == cudaSuccess)
            ce = cudaStreamWaitEvent(s, h->ev_arrive, 0);
        if (ce != cudaSuccess)
            return fail(cuda_fail(ce));
        rc = launch_group(g);
        if (rc != MELINOE_OK)
            return fail(rc);
        if (need_done[g] && cudaEventRecord(h->ev_group[g], s) != cudaSuccess)
            return fail(cuda_fail(cudaGetLastError()));
    }

    if (use_gemm)
        CU_TRY(launch_combine_rows(s, h->plan, sc.gate, sc.inv_pos, h->zbuf, static_cast<uint16_t *>(out_dev), T, h->d,
                                   h->k, h->n_shared, h->n_sms));
    CU_TRY(cudaEventRecord(h->ev_last, s));
    h->has_last = true;
    return MELINOE_OK;
}

int check_forward_args(melinoe_moe *h, const void *hidden_dev, int T, void *out_dev)
{
    if (!h || T < 0)
        return MELINOE_ERR_INVALID;
    if (T == 0)
        return MELINOE_OK;
    if (!hidden_dev || !out_dev || !aligned16(hidden_dev) || !aligned16(out_dev))
        return MELINOE_ERR_INVALID;
    if (!h->w_router || !h->host_experts[0])
        return MELINOE_ERR_STATE;
    if (h->sticky.load() != MELINOE_OK)
        return h->sticky.load();
    return MELINOE_OK;
}

}  // namespace

extern "C" int melinoe_moe_forward(melinoe_moe_t *h, void *cuda_stream, const void *hidden_dev, int T, void *out_dev,
                                   melinoe_moe_stats *stats_dev)
{
    int rc = check_forward_args(h, hidden_dev, T, out_dev);
    if (rc != MELINOE_OK || T == 0)
        return rc;
    rc = ensure_capacity(h, T);
    if (rc != MELINOE_OK)
        return rc;
    return forward_on(h, h->own, cuda_stream, hidden_dev, T, out_dev, stats_dev);
}

// ---------------------------------------------------------------- forward without allocation
//
// Scratch of melinoe_moe_forward_static: one array in the library's device image, shared by every
// call on the device, instead of per-handle cudaMalloc'd buffers.
constexpr int kStaticMaxTokens = 8;
constexpr int kStaticMaxPairs = 64;                         // n_tokens * top_k
constexpr size_t kStaticSmall = 16 * 1024;                  // idx, gate, logits, perm, inv_pos, tok_of_sorted
constexpr size_t kStaticY = (size_t)kStaticMaxTokens * 4096 * sizeof(float);   // fp32 sums of a call made in several launches
constexpr size_t kStaticAcc = (size_t)kStaticMaxTokens * 4096 * sizeof(long long);   // fixed-point sums of a launch
constexpr size_t kStaticBytes = kStaticSmall + kStaticY + kStaticAcc;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

namespace {
// Device address of g_static_scratch per device ordinal.  In host code the array's name is
// only a handle for the runtime, not an address a kernel could use.
constexpr int kMaxDevices = 64;
unsigned char *g_static_ptr[kMaxDevices] = {nullptr};
std::mutex g_static_mu;
}  // namespace

extern "C" int melinoe_moe_forward_static(melinoe_moe_t *h, void *cuda_stream, const void *hidden_dev, int T,
                                          void *out_dev, melinoe_moe_stats *stats_dev)
{
    int rc = check_forward_args(h, hidden_dev, T, out_dev);
    if (rc != MELINOE_OK || T == 0)
        return rc;
    // everything beyond the static scratch's sizes is refused, never served by allocating
    if (T > kStaticMaxTokens || T * h->k > kStaticMaxPairs || (size_t)h->n_shared * T + (size_t)T * h->k > 1024 ||
        (size_t)T * h->d * sizeof(float) > kStaticY)
        return MELINOE_ERR_UNSUPPORTED;
    if (h->timing)
        return MELINOE_ERR_STATE;   // timed calls create events on demand
    if (h->device < 0 || h->device >= kMaxDevices)
        return MELINOE_ERR_UNSUPPORTED;
    int cur = -1;
    CU_TRY(cudaGetDevice(&cur));
    if (cur != h->device)
        return MELINOE_ERR_STATE;   // the handle's device must be current, as for every call
    unsigned char *base = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_static_mu);
        base = g_static_ptr[h->device];
        if (!base) {
            // first call on this device: look the array's address up
            void *p = nullptr;
            CU_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
            base = g_static_ptr[h->device] = static_cast<unsigned char *>(p);
        }
    }
    // carve the scratch: small tables first, then the fp32 sums, then the fixed-point accumulator.  The
    // tables are written by the call's kernels before they are read; the accumulator must be all zero
    // when a launch starts: it is (static storage starts out zero) and every launch leaves it so.
    unsigned char *q = base;
    auto take = [&](size_t bytes) {
        unsigned char *r = q;
        q += (bytes + 255) / 256 * 256;
        return r;
    };
    const size_t pairs = kStaticMaxPairs, sorted = 1024;
    Scratch sc;
    sc.idx = reinterpret_cast<int32_t *>(take(pairs * 4));
    sc.gate = reinterpret_cast<float *>(take(pairs * 4));
    sc.logits = reinterpret_cast<float *>(take((size_t)kStaticMaxTokens * kMaxExperts * 4));
    sc.perm = reinterpret_cast<int32_t *>(take(sorted * 4));
    sc.inv_pos = reinterpret_cast<int32_t *>(take(pairs * 4));
    sc.tok_of_sorted = reinterpret_cast<int32_t *>(take(sorted * 4));
    if ((size_t)(q - base) > kStaticSmall)
        return MELINOE_ERR_STATE;
    sc.ybuf = reinterpret_cast<float *>(base + kStaticSmall);
    sc.yacc = reinterpret_cast<long long *>(base + kStaticSmall + kStaticY);
    sc.cap_tokens = kStaticMaxTokens;
    return forward_on(h, sc, cuda_stream, hidden_dev, T, out_dev, stats_dev);
}

extern "C" size_t melinoe_moe_static_scratch_bytes(void) { return kStaticBytes; }

extern "C" {

int melinoe_moe_forward_host(melinoe_moe_t *h, void *cuda_stream, const void *hidden_host, int T, void *out_host,
                             melinoe_moe_stats *stats_host)
{
    if (!h || T < 0)
        return MELINOE_ERR_INVALID;
    if (T == 0)
        return MELINOE_OK;
    if (!hidden_host || !out_host)
        return MELINOE_ERR_INVALID;
    int rc = ensure_capacity(h, T);
    if (rc != MELINOE_OK)
        return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t bytes = (size_t)T * h->d * 2;
    {
        // decode-sized input from page-locked (device-mapped) memory: fetched by a small kernel, which
        // costs the stream less than a copy-engine operation; otherwise a plain copy
        cudaPointerAttributes a;
        if (T <= kTokPerVr && cudaPointerGetAttributes(&a, hidden_host) == cudaSuccess && a.type == cudaMemoryTypeHost &&
            a.devicePointer && aligned16(a.devicePointer)) {
            CU_TRY(launch_stage_in(s, a.devicePointer, h->stage_in, bytes));
        } else {
            (void)cudaGetLastError();
            CU_TRY(cudaMemcpyAsync(h->stage_in, hidden_host, bytes, cudaMemcpyHostToDevice, s));
        }
    }
    // A decode-sized result goes straight to page-locked host memory from the kernels that produce it
    // (a few hundred posted writes) instead of through two more copy-engine operations, each of
    // which costs the stream several microseconds.  Pageable buffers and large calls are staged.
    void *out_direct = nullptr, *stats_direct = nullptr;
    if (T <= kTokPerVr) {
        cudaPointerAttributes a;
        if (cudaPointerGetAttributes(&a, out_host) == cudaSuccess && a.type == cudaMemoryTypeHost && a.devicePointer &&
            aligned16(a.devicePointer))
            out_direct = a.devicePointer;
        if (stats_host && cudaPointerGetAttributes(&a, stats_host) == cudaSuccess && a.type == cudaMemoryTypeHost &&
            a.devicePointer && (reinterpret_cast<uintptr_t>(a.devicePointer) & 7u) == 0)
            stats_direct = a.devicePointer;
        (void)cudaGetLastError();
    }
    rc = melinoe_moe_forward(h, cuda_stream, h->stage_in, T, out_direct ? out_direct : h->stage_out,
                             stats_host ? (stats_direct ? static_cast<melinoe_moe_stats *>(stats_direct) : h->stage_stats)
                                        : nullptr);
    if (rc != MELINOE_OK)
        return rc;
    if (!out_direct)
        CU_TRY(cudaMemcpyAsync(out_host, h->stage_out, bytes, cudaMemcpyDeviceToHost, s));
    if (stats_host && !stats_direct)
        CU_TRY(cudaMemcpyAsync(stats_host, h->stage_stats, sizeof(melinoe_moe_stats), cudaMemcpyDeviceToHost, s));
    CU_TRY(cudaEventRecord(h->ev_last, s));
    return MELINOE_OK;
}

int melinoe_trace_miss_proxies(void *cuda_stream, const int32_t *trace_dev, int n_layers, int n_tokens, int top_k,
                               int n_experts, const melinoe_proxy_config *configs_dev, int n_configs,
                               double *soft_mean_dev, int64_t *hard_total_dev)
{
    if (!trace_dev || !configs_dev || !soft_mean_dev || !hard_total_dev || n_layers <= 0 || n_tokens < 0 || top_k <= 0 ||
        n_experts <= 0 || n_configs < 0 || top_k > n_experts)
        return MELINOE_ERR_INVALID;
    if (n_experts > kMaxExperts)
        return MELINOE_ERR_UNSUPPORTED;
    if (n_configs == 0)
        return MELINOE_OK;
    CU_TRY(launch_miss_proxies(static_cast<cudaStream_t>(cuda_stream), trace_dev, n_layers, n_tokens, top_k, n_experts, configs_dev,
                               n_configs, soft_mean_dev, reinterpret_cast<long long *>(hard_total_dev)));
    return MELINOE_OK;
}

int melinoe_moe_reset_cache(melinoe_moe_t *h)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    int rc = wait_idle(h);
    if (rc != MELINOE_OK)
        return rc;
    DevCache c0;
    init_cache_host(c0);
    CU_TRY(cudaMemcpy(h->cache, &c0, sizeof c0, cudaMemcpyHostToDevice));
    CU_TRY(cudaMemset(h->err_word, 0, 4));
    h->sticky.store(MELINOE_OK);
    return MELINOE_OK;
}

int melinoe_moe_set_policy(melinoe_moe_t *h, int policy, float gamma)
{
    if (!h || (policy != MELINOE_POLICY_LRU && policy != MELINOE_POLICY_COUNT) || !(gamma >= 0.0f && gamma <= 1.0f))
        return MELINOE_ERR_INVALID;
    int rc = wait_idle(h);
    if (rc != MELINOE_OK)
        return rc;
    h->policy = policy;
    h->gamma = gamma;
    return MELINOE_OK;
}

int melinoe_moe_cache_counts(melinoe_moe_t *h, float *counts_host)
{
    if (!h || !counts_host)
        return MELINOE_ERR_INVALID;
    int rc = wait_idle(h);
    if (rc != MELINOE_OK)
        return rc;
    DevCache c;
    CU_TRY(cudaMemcpy(&c, h->cache, sizeof c, cudaMemcpyDeviceToHost));
    for (int e = 0; e < h->E; ++e)
        counts_host[e] = c.count[e];
    return MELINOE_OK;
}

int melinoe_moe_preload(melinoe_moe_t *h, const int32_t *ids, int n)
{
    if (!h || n < 0 || (n > 0 && !ids) || n > h->C)
        return MELINOE_ERR_INVALID;
    for (int i = 0; i < n; ++i)
        if (ids[i] < 0 || ids[i] >= h->E)
            return MELINOE_ERR_INVALID;
    if (!h->host_experts[0])
        return MELINOE_ERR_STATE;
    if (h->sticky.load() != MELINOE_OK)
        return h->sticky.load();
    if (n == 0)
        return MELINOE_OK;
    // behind everything already queued on the handle (whose kernels may still read the slots)
    if (h->has_last)
        CU_TRY(cudaStreamWaitEvent(h->copy_stream, h->ev_last, 0));
    PreloadParams pp;
    pp.cache = h->cache;
    pp.list = h->pre_dev;
    pp.host_list = nullptr;
    for (int i = 0; i < kMaxExperts; ++i)
        pp.ids[i] = i < n ? ids[i] : -1;
    pp.n = n;
    pp.C = h->C;
    pp.policy = h->policy;
    pp.seq = ++h->preload_seq;
    if (h->pull_ok) {
        // the cache requests and the copies both run on the device: nothing to wait for here
        CU_TRY(launch_preload_plan(h->copy_stream, pp));
        FetchParams fp;
        fp.list = h->pre_dev;
        fp.host_blobs = h->host_dev;
        fp.slots = h->slots;
        fp.slot_stride = h->slot_stride;
        fp.rows = h->F;
        fp.row_bytes = (int)(h->expert_bytes / (size_t)h->F);     // one hidden unit of the slots' format
        fp.rows_per_piece = 49152 / fp.row_bytes > 0 ? 49152 / fp.row_bytes : 1;
        fp.piece_bytes = fp.rows_per_piece * fp.row_bytes;
        fp.err = h->err_word;
        CU_TRY(launch_fetch_experts(h->copy_stream, h->n_sms, fp));
        CU_TRY(cudaEventRecord(h->ev_preload, h->copy_stream));
    } else {
        // the host issues the copies: it has to see the list the planning kernel wrote
        void *hl = nullptr;
        CU_TRY(cudaHostGetDevicePointer(&hl, h->pre_host, 0));
        pp.host_list = static_cast<PreloadList *>(hl);
        CU_TRY(launch_preload_plan(h->copy_stream, pp));
        CU_TRY(cudaStreamSynchronize(h->copy_stream));
        const volatile PreloadList &vl = *h->pre_host;
        if (vl.seq != pp.seq || vl.n < 0 || vl.n > n)
            return MELINOE_ERR_STATE;
        const int nf = vl.n;
        for (int i = 0; i < nf; ++i) {
            const int e = vl.expert[i], slot = vl.slot[i];
            if (e < 0 || e >= h->E || slot < 0 || slot >= h->C)
                return MELINOE_ERR_STATE;
            if (h->store_q4) {
                const unsigned b = h->q4_turn++ & 1u;
                char *stage = h->q4_stage + (size_t)b * h->q4_bytes;
                if (h->q4_used[b])
                    CU_TRY(cudaStreamWaitEvent(h->copy_stream, h->ev_q4_expanded[b], 0));
                CU_TRY(cudaMemcpyAsync(stage, h->host_experts[e], h->q4_bytes, cudaMemcpyHostToDevice, h->copy_stream));
                CU_TRY(cudaEventRecord(h->ev_q4_copied[b], h->copy_stream));
                CU_TRY(cudaStreamWaitEvent(h->dq_stream, h->ev_q4_copied[b], 0));
                CU_TRY(launch_dequant_q4(h->dq_stream, stage, h->slots + (size_t)slot * h->slot_stride, h->d, h->F, h->n_sms));
                CU_TRY(cudaEventRecord(h->ev_q4_expanded[b], h->dq_stream));
                h->q4_used[b] = true;
            } else {
                CU_TRY(cudaMemcpyAsync(h->slots + (size_t)slot * h->slot_stride, h->host_experts[e], h->expert_bytes,
                                       cudaMemcpyHostToDevice, h->copy_stream));
            }
        }
        if (h->store_q4) {
            // the event has to cover the copy stream (planning kernel) and the expansion stream
            CU_TRY(cudaEventRecord(h->ev_arrive, h->dq_stream));
            CU_TRY(cudaStreamWaitEvent(h->copy_stream, h->ev_arrive, 0));
        }
        CU_TRY(cudaEventRecord(h->ev_preload, h->copy_stream));
    }
    h->preload_pending = true;
    return MELINOE_OK;
}

int melinoe_moe_preload_pooled(melinoe_moe_t *h, const int32_t *lists_host, int n_seq, int per_seq)
{
    if (!h || !lists_host || n_seq <= 0 || per_seq <= 0)
        return MELINOE_ERR_INVALID;
    // votes: in how many sequences' lists an expert appears (once per list)
    int votes[kMaxExperts] = {0};
    for (int q = 0; q < n_seq; ++q) {
        bool seen[kMaxExperts] = {false};
        for (int j = 0; j < per_seq; ++j) {
            const int e = lists_host[(size_t)q * per_seq + j];
            if (e < 0 || e >= h->E)
                return MELINOE_ERR_INVALID;
            if (!seen[e]) {
                seen[e] = true;
                votes[e] += 1;
            }
        }
    }
    // the cache_slots experts with the most votes, the lower id first among equals, loaded in that order
    int32_t chosen[kMaxExperts];
    int n = 0;
    for (int v = n_seq; v >= 1 && n < h->C; --v)
        for (int e = 0; e < h->E && n < h->C; ++e)
            if (votes[e] == v)
                chosen[n++] = e;
    return melinoe_moe_preload(h, chosen, n);
}

int melinoe_moe_last_routing(melinoe_moe_t *h, int32_t *idx_host, float *gate_host)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    if (h->last_T <= 0)
        return MELINOE_ERR_STATE;
    const size_t n = (size_t)h->last_T * h->k;
    if (idx_host)
        CU_TRY(cudaMemcpy(idx_host, h->last.idx, n * 4, cudaMemcpyDeviceToHost));
    if (gate_host)
        CU_TRY(cudaMemcpy(gate_host, h->last.gate, n * 4, cudaMemcpyDeviceToHost));
    return MELINOE_OK;
}

int melinoe_moe_last_logits(melinoe_moe_t *h, float *logits_host)
{
    if (!h || !logits_host)
        return MELINOE_ERR_INVALID;
    if (h->last_T <= 0)
        return MELINOE_ERR_STATE;
    CU_TRY(cudaMemcpy(logits_host, h->last.logits, (size_t)h->last_T * h->E * 4, cudaMemcpyDeviceToHost));
    return MELINOE_OK;
}

int melinoe_moe_last_requests(melinoe_moe_t *h, melinoe_moe_request *req_host, int *n_out)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    if (h->last_T <= 0)
        return MELINOE_ERR_STATE;
    DevPlan *pl = new (std::nothrow) DevPlan;
    if (!pl)
        return MELINOE_ERR_NOMEM;
    cudaError_t e = cudaMemcpy(pl, h->plan, sizeof(DevPlan), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) {
        delete pl;
        return cuda_fail(e);
    }
    if (n_out)
        *n_out = pl->n_req;
    if (req_host)
        for (int i = 0; i < pl->n_req; ++i) {
            req_host[i].expert = pl->req[i].expert;
            req_host[i].slot = pl->req[i].slot;
            req_host[i].hit = pl->req[i].hit;
            req_host[i].evicted = pl->req[i].evicted;
        }
    delete pl;
    return MELINOE_OK;
}

int melinoe_moe_last_gather(melinoe_moe_t *h, int32_t *counts_host, int32_t *offsets_host, int32_t *perm_host)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    if (h->last_T <= 0)
        return MELINOE_ERR_STATE;
    if (counts_host)
        CU_TRY(cudaMemcpy(counts_host, reinterpret_cast<char *>(h->plan) + offsetof(DevPlan, counts), (size_t)h->E * 4,
                          cudaMemcpyDeviceToHost));
    if (offsets_host)
        CU_TRY(cudaMemcpy(offsets_host, reinterpret_cast<char *>(h->plan) + offsetof(DevPlan, offsets),
                          (size_t)(h->E + 1) * 4, cudaMemcpyDeviceToHost));
    if (perm_host)
        CU_TRY(cudaMemcpy(perm_host, h->last.perm, (size_t)h->last_T * h->k * 4, cudaMemcpyDeviceToHost));
    return MELINOE_OK;
}

int melinoe_moe_cache_state(melinoe_moe_t *h, int32_t *expert_of_slot_host, uint64_t *totals_host)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    DevCache c;
    CU_TRY(cudaMemcpy(&c, h->cache, sizeof c, cudaMemcpyDeviceToHost));
    if (expert_of_slot_host)
        for (int s = 0; s < h->C; ++s)
            expert_of_slot_host[s] = c.expert_of_slot[s];
    if (totals_host) {
        totals_host[0] = c.tot_hits;
        totals_host[1] = c.tot_misses;
        totals_host[2] = c.tot_evictions;
    }
    int err = 0;
    CU_TRY(cudaMemcpy(&err, h->err_word, 4, cudaMemcpyDeviceToHost));
    if (err != 0)
        return err;
    return h->sticky.load();
}

int melinoe_moe_transfer_time_ms(melinoe_moe_t *h, double *ms_out, uint64_t *bytes_out)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    double total = 0.0;
    for (auto &p : h->timed_copy) {
        CU_TRY(cudaEventSynchronize(p.b));
        float ms = 0.f;
        CU_TRY(cudaEventElapsedTime(&ms, p.a, p.b));
        total += ms;
    }
    if (ms_out)
        *ms_out = total;
    if (bytes_out)
        *bytes_out = h->timed_copy_bytes;
    for (auto &p : h->timed_copy)
        h->free_pairs.push_back(p);
    h->timed_copy.clear();
    h->timed_copy_bytes = 0;
    return MELINOE_OK;
}

int melinoe_moe_set_timeline(melinoe_moe_t *h, void *trace_dev, size_t bytes)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    if (!trace_dev) {
        h->trace = nullptr;
        return MELINOE_OK;
    }
    if (bytes < (size_t)h->cfg.grid * 8 * sizeof(unsigned long long) || (reinterpret_cast<uintptr_t>(trace_dev) & 7u))
        return MELINOE_ERR_INVALID;
    h->trace = static_cast<unsigned long long *>(trace_dev);
    return MELINOE_OK;
}

int melinoe_moe_timeline_ctas(melinoe_moe_t *h) { return h ? h->cfg.grid : 0; }

size_t melinoe_moe_trace_record_bytes(melinoe_moe_t *h, int max_tokens)
{
    if (!h || max_tokens <= 0)
        return 0;
    return trace_layout(h->E, h->k, max_tokens).bytes;
}

int melinoe_moe_set_trace(melinoe_moe_t *h, void *trace_buf, size_t bytes, int max_tokens)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    if (!trace_buf) {
        h->req_trace = nullptr;
        h->req_trace_cap = 0;
        return MELINOE_OK;
    }
    if (max_tokens <= 0 || !aligned16(trace_buf))
        return MELINOE_ERR_INVALID;
    const size_t rb = trace_layout(h->E, h->k, max_tokens).bytes;
    if (bytes < rb)
        return MELINOE_ERR_INVALID;
    // the device must be able to write it: device memory, or page-locked host memory it can address
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, trace_buf) != cudaSuccess || (a.type != cudaMemoryTypeDevice && a.type != cudaMemoryTypeHost) ||
        !a.devicePointer) {
        (void)cudaGetLastError();
        return MELINOE_ERR_INVALID;
    }
    h->req_trace = static_cast<char *>(a.devicePointer);
    h->req_trace_cap = bytes / rb;
    h->req_trace_tokens = max_tokens;
    h->req_trace_count = 0;
    return MELINOE_OK;
}

int64_t melinoe_moe_trace_count(melinoe_moe_t *h) { return h ? (int64_t)h->req_trace_count : 0; }

int melinoe_allocate_slots(const int64_t *hard, int n_layers, int n_sizes, int first_size, int64_t budget, int32_t *slots_out)
{
    if (!hard || !slots_out || n_layers <= 0 || n_sizes <= 0 || first_size <= 0)
        return MELINOE_ERR_INVALID;
    long long left = (long long)budget - (long long)n_layers * first_size;
    if (left < 0)
        return MELINOE_ERR_INVALID;
    std::vector<int> at((size_t)n_layers, 0);
    while (left > 0) {
        int best = -1;
        long long gain = -1;
        for (int l = 0; l < n_layers; ++l)
            if (at[l] + 1 < n_sizes) {
                const long long g = (long long)(hard[(size_t)l * n_sizes + at[l]] - hard[(size_t)l * n_sizes + at[l] + 1]);
                if (g > gain) {
                    best = l;
                    gain = g;
                }
            }
        if (best < 0)
            break;
        at[best] += 1;
        left -= 1;
    }
    for (int l = 0; l < n_layers; ++l)
        slots_out[l] = first_size + at[l];
    return MELINOE_OK;
}

int melinoe_moe_last_call_used_gemm(melinoe_moe_t *h) { return h && h->last_used_gemm ? 1 : 0; }

int melinoe_debug_fail_host_copy(int nth)
{
    g_fail_copy_in.store(nth > 0 ? nth : 0);
    return MELINOE_OK;
}

int melinoe_moe_enable_timing(melinoe_moe_t *h, int enable)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    h->timing = enable != 0;
    return MELINOE_OK;
}

int melinoe_moe_ffn_launch_times_ms(melinoe_moe_t *h, float *ms_out, int capacity, int *n_out)
{
    if (!h || capacity < 0 || (capacity > 0 && !ms_out))
        return MELINOE_ERR_INVALID;
    int n = 0;
    for (auto &p : h->timed) {
        if (n >= capacity)
            break;
        CU_TRY(cudaEventSynchronize(p.b));
        CU_TRY(cudaEventElapsedTime(&ms_out[n], p.a, p.b));
        ++n;
    }
    if (n_out)
        *n_out = (int)h->timed.size();
    return MELINOE_OK;
}

int melinoe_moe_ffn_time_ms(melinoe_moe_t *h, double *ms_out, int64_t *launches_out)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    double total = 0.0;
    for (auto &p : h->timed) {
        CU_TRY(cudaEventSynchronize(p.b));
        float ms = 0.f;
        CU_TRY(cudaEventElapsedTime(&ms, p.a, p.b));
        total += ms;
    }
    if (ms_out)
        *ms_out = total;
    if (launches_out)
        *launches_out = (int64_t)h->timed.size();
    for (auto &p : h->timed)
        h->free_pairs.push_back(p);
    h->timed.clear();
    return MELINOE_OK;
}

}  // extern "C"
