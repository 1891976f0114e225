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

// 2-D bf16 tensor [rows][cols], row-major, 128-byte swizzle, box of box_rows x 64 columns.
bool encode_map(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint32_t box_rows)
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
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return g_encode_tiled(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

double now_s()
{
    return std::chrono::duration<double>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

struct TimedPair {
    cudaEvent_t a, b;
};

}  // namespace

struct melinoe_moe {
    int d = 0, F = 0, E = 0, k = 0, C = 0, device = 0, n_sms = 0;
    size_t expert_bytes = 0, slot_stride = 0;
    FfnLaunchCfg cfg{};

    // device memory owned by the handle
    char *slots = nullptr;
    DevCache *cache = nullptr;
    int policy = MELINOE_POLICY_LRU;   // eviction policy, see melinoe_moe_set_policy
    float gamma = 0.0f;
    DevPlan *plan = nullptr;
    int *err_word = nullptr;
    const char **shared_dev = nullptr;

    // scratch sized for cap_tokens
    int cap_tokens = 0, cap_shared = -1, vr_capacity = 0;
    int32_t *idx = nullptr, *perm = nullptr, *inv_pos = nullptr, *tok_of_sorted = nullptr;
    float *gate = nullptr, *logits = nullptr, *zbuf = nullptr;
    uint16_t *hbuf = nullptr;
    unsigned *sync = nullptr;
    unsigned long long *trace = nullptr;   // borrowed; see melinoe_moe_set_trace
    VrRec *vrs = nullptr;
    uint16_t *stage_in = nullptr, *stage_out = nullptr;
    // grouped-GEMM path (calls of more than 8 tokens): gathered activations, h, tensor maps
    bool gemm_ok = false, pair_ok = false, last_used_gemm = false, last_used_pair = false;
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
    cudaFree(h->idx);
    cudaFree(h->perm);
    cudaFree(h->inv_pos);
    cudaFree(h->tok_of_sorted);
    cudaFree(h->gate);
    cudaFree(h->logits);
    cudaFree(h->zbuf);
    cudaFree(h->hbuf);
    cudaFree(h->vrs);
    cudaFree(h->stage_in);
    cudaFree(h->stage_out);
    cudaFree(h->xs);
    cudaFree(h->hs);
    h->xs = h->hs = nullptr;
    h->idx = h->perm = h->inv_pos = h->tok_of_sorted = nullptr;
    h->gate = h->logits = h->zbuf = nullptr;
    h->hbuf = nullptr;
    h->vrs = nullptr;
    h->stage_in = h->stage_out = nullptr;
    h->cap_tokens = 0;
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
    if (T <= h->cap_tokens && h->cap_shared == h->n_shared)
        return MELINOE_OK;
    int rc = wait_idle(h);
    if (rc != MELINOE_OK)
        return rc;
    CU_TRY(cudaDeviceSynchronize());
    const int cap = T > h->cap_tokens ? T : h->cap_tokens;
    free_scratch(h);
    const size_t pairs = (size_t)cap * h->k;
    const size_t sorted = pairs + (size_t)h->n_shared * cap;
    const int vr_cap = (int)(pairs / kTokPerVr) + h->E + h->n_shared * (cap / kTokPerVr + 1) + 8;
    const size_t fpad = ((size_t)h->F + 255) / 256 * 256;
    const size_t hbytes = (size_t)vr_cap * kTokPerVr * fpad * 2;
    CU_TRY(cudaMalloc(&h->idx, pairs * 4));
    CU_TRY(cudaMalloc(&h->gate, pairs * 4));
    CU_TRY(cudaMalloc(&h->logits, (size_t)cap * h->E * 4));
    CU_TRY(cudaMalloc(&h->perm, sorted * 4));
    CU_TRY(cudaMalloc(&h->inv_pos, pairs * 4));
    CU_TRY(cudaMalloc(&h->tok_of_sorted, sorted * 4));
    CU_TRY(cudaMalloc(&h->vrs, (size_t)vr_cap * sizeof(VrRec)));
    CU_TRY(cudaMalloc(&h->zbuf, sorted * h->d * sizeof(float)));
    CU_TRY(cudaMalloc(&h->hbuf, hbytes));
    CU_TRY(cudaMemset(h->hbuf, 0, hbytes));   // the padding of every h row stays zero for good
    CU_TRY(cudaMalloc(&h->stage_in, (size_t)cap * h->d * 2));
    CU_TRY(cudaMalloc(&h->stage_out, (size_t)cap * h->d * 2));
    if (h->gemm_ok && cap > kTokPerVr) {
        CU_TRY(cudaMalloc(&h->xs, sorted * h->d * 2));
        CU_TRY(cudaMalloc(&h->hs, sorted * h->F * 2));
        if (!encode_map(&h->maps_host[kMapXs], h->xs, h->d, sorted, 128) ||
            !encode_map(&h->maps_host[kMapHs], h->hs, h->F, sorted, 128))
            return MELINOE_ERR_CUDA;
        CU_TRY(cudaMemcpy(h->maps_dev, h->maps_host, sizeof(h->maps_host), cudaMemcpyHostToDevice));
    }
    h->vr_capacity = vr_cap;
    h->cap_tokens = cap;
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
    const size_t m = (size_t)d * F * 2;
    char *blob = static_cast<char *>(blob_);
    std::memcpy(blob, wg_, m);
    std::memcpy(blob + m, wu_, m);
    std::memcpy(blob + 2 * m, wd_, m);
    return MELINOE_OK;
}

size_t melinoe_moe_expert_bytes_q4(int d_model, int d_ff)
{
    if (d_model <= 0 || d_ff <= 0 || d_model % 64 != 0 || d_ff % 64 != 0)
        return 0;
    const size_t n = (size_t)d_model * (size_t)d_ff;
    return 3 * (n / 2 + n / 32);
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

// One matrix [rows][cols] into its section: codes [rows][cols / 2], then scales [rows][cols / 64].
void pack_q4_matrix(const uint16_t *w, size_t rows, size_t cols, unsigned char *section)
{
    unsigned char *codes = section;
    uint16_t *scales = reinterpret_cast<uint16_t *>(section + rows * cols / 2);
    for (size_t r = 0; r < rows; ++r) {
        for (size_t g = 0; g < cols / 64; ++g) {
            const uint16_t *src = w + r * cols + g * 64;
            float amax = 0.0f;
            for (int j = 0; j < 64; ++j)
                amax = std::fmax(amax, std::fabs(host_bf16_to_f32(src[j])));
            const uint16_t sb = host_f32_to_bf16(amax / 7.0f);
            const float sc = host_bf16_to_f32(sb);
            scales[r * (cols / 64) + g] = sb;
            unsigned char *dst = codes + (r * cols + g * 64) / 2;
            for (int j = 0; j < 64; j += 2) {
                int q[2] = {0, 0};
                for (int h2 = 0; h2 < 2; ++h2)
                    if (sc > 0.0f) {
                        const float t = std::nearbyint(host_bf16_to_f32(src[j + h2]) / sc);   // ties to even
                        q[h2] = (int)std::fmin(7.0f, std::fmax(-8.0f, t));
                    }
                dst[j / 2] = (unsigned char)((q[0] + 8) | ((q[1] + 8) << 4));
            }
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
    const size_t n = (size_t)d * F, sec = n / 2 + n / 32;
    unsigned char *blob = static_cast<unsigned char *>(blob_);
    pack_q4_matrix(static_cast<const uint16_t *>(wg_), (size_t)F, (size_t)d, blob);
    pack_q4_matrix(static_cast<const uint16_t *>(wu_), (size_t)F, (size_t)d, blob + sec);
    pack_q4_matrix(static_cast<const uint16_t *>(wd_), (size_t)d, (size_t)F, blob + 2 * sec);
    return MELINOE_OK;
}

int melinoe_moe_create(int d, int F, int E, int k, int C, melinoe_moe_t **out)
{
    if (!out)
        return MELINOE_ERR_INVALID;
    *out = nullptr;
    if (d <= 0 || F <= 0 || E <= 0 || k <= 0 || C <= 0 || k > E || C < k || C > E)
        return MELINOE_ERR_INVALID;
    if (d % 256 != 0 || d > 8192 || F % kUnitRows != 0 || E > kMaxExperts || k > 32)
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
    h->expert_bytes = melinoe_moe_expert_bytes(d, F);
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
    if (!prop.cooperativeLaunch ||
        ffn_stream_configure(h->n_sms, prop.sharedMemPerBlockOptin, &h->cfg) != cudaSuccess) {
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
    CR(cudaMalloc(&h->sync, sizeof(unsigned) * (2 * (kMaxGroups + 1) + 1)));
    CR(cudaMemset(h->sync, 0, sizeof(unsigned) * (2 * (kMaxGroups + 1) + 1)));
    CR(cudaMalloc(&h->shared_dev, sizeof(char *) * kMaxShared));
    CR(cudaMalloc(&h->stage_stats, sizeof(melinoe_moe_stats)));
    CR(cudaMemset(h->err_word, 0, 256));
    CR(cudaMemset(h->plan, 0, sizeof(DevPlan)));
    CR(cudaMemset(h->shared_dev, 0, sizeof(char *) * kMaxShared));
    DevCache c0;
    init_cache_host(c0);
    CR(cudaMemcpy(h->cache, &c0, sizeof c0, cudaMemcpyHostToDevice));
    CR(cudaHostAlloc(&h->hplan, sizeof(HostPlan), cudaHostAllocMapped | cudaHostAllocPortable));
    std::memset(h->hplan, 0, sizeof(HostPlan));
    CR(cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
    CR(cudaEventCreateWithFlags(&h->ev_last, cudaEventDisableTiming));
    CR(cudaEventCreateWithFlags(&h->ev_plan, cudaEventDisableTiming));
    CR(cudaEventCreateWithFlags(&h->ev_arrive, cudaEventDisableTiming));
    // grouped GEMM for calls of many tokens: the slots are contiguous, so one tensor map per view
    // (rows of d elements: W_g, W_u; rows of F elements: W_d) covers every slot
    std::memset(h->maps_host, 0, sizeof(h->maps_host));
    if (ffn_gemm_supported(d, F) && h->slot_stride == h->expert_bytes && ffn_gemm_configure() == cudaSuccess) {
        CR(cudaMalloc(&h->maps_dev, sizeof(h->maps_host)));
        if (encode_map(&h->maps_host[kMapSlotsD], h->slots, d, (uint64_t)C * 3 * F, 128) &&
            encode_map(&h->maps_host[kMapSlotsF], h->slots, F, (uint64_t)C * 3 * d, 256) &&
            encode_map(&h->maps_host[kMapSlotsF128], h->slots, F, (uint64_t)C * 3 * d, 128)) {
            CR(cudaMemcpy(h->maps_dev, h->maps_host, sizeof(h->maps_host), cudaMemcpyHostToDevice));
            h->gemm_ok = true;
            h->pair_ok = ffn_gemm_pair_configure() == cudaSuccess && (h->n_sms & ~1) >= 2;
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
    cudaFree(h->maps_dev);
    cudaFree(h->stage_stats);
    if (h->hplan)
        cudaFreeHost(h->hplan);
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

int melinoe_moe_register_host_experts(melinoe_moe_t *h, const void *const *ptrs, size_t bytes_per_expert)
{
    if (!h || !ptrs || bytes_per_expert != h->expert_bytes)
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
            if (!encode_map(&h->maps_host[kMapShared0 + 2 * s], ptrs[s], h->d, (uint64_t)3 * h->F, 128) ||
                !encode_map(&h->maps_host[kMapShared0 + 2 * s + 1], ptrs[s], h->F, (uint64_t)3 * h->d, 256) ||
                !encode_map(&h->maps_host[kMapSharedF128 + s], ptrs[s], h->F, (uint64_t)3 * h->d, 128))
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

int melinoe_moe_forward(melinoe_moe_t *h, void *cuda_stream, const void *hidden_dev, int T, void *out_dev,
                        melinoe_moe_stats *stats_dev)
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
    int rc = ensure_capacity(h, T);
    if (rc != MELINOE_OK)
        return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const uint32_t gmax = (uint32_t)gmax_for(h, T);
    h->call_seq += 1;
    h->last_T = T;

    PlanParams pp;
    pp.idx = h->idx;
    pp.T = T;
    pp.k = h->k;
    pp.E = h->E;
    pp.C = h->C;
    pp.n_shared = h->n_shared;
    pp.cache = h->cache;
    pp.plan = h->plan;
    pp.vrs = h->vrs;
    pp.slots = h->slots;
    pp.slot_stride = h->slot_stride;
    pp.shared_blobs = h->shared_dev;
    pp.perm = h->perm;
    pp.inv_pos = h->inv_pos;
    pp.tok_of_sorted = h->tok_of_sorted;
    pp.hplan = h->hplan;
    pp.sync = h->sync;
    pp.gmax = gmax;
    pp.call_seq = h->call_seq;
    pp.policy = h->policy;
    pp.gamma = h->gamma;
    pp.stats = stats_dev;
    pp.expert_bytes = h->store_q4 ? h->q4_bytes : h->expert_bytes;   // bytes one miss moves over the host link
    pp.vr_capacity = h->vr_capacity;
    if (route_plan_small_supported(T, h->k, h->d)) {
        CU_TRY(launch_route_plan_small(s, static_cast<const uint16_t *>(hidden_dev), h->w_router, h->bias, h->token_seq,
                                       h->d, h->idx, h->gate, h->logits, pp));
    } else {
        CU_TRY(launch_router(s, static_cast<const uint16_t *>(hidden_dev), h->w_router, h->bias, h->token_seq, T, h->d,
                             h->E, h->k, h->idx, h->gate, h->logits));
        CU_TRY(launch_plan(s, pp));
    }
    CU_TRY(cudaEventRecord(h->ev_plan, s));

    FfnParams fp;
    fp.plan = h->plan;
    fp.vrs = h->vrs;
    fp.x = static_cast<const uint16_t *>(hidden_dev);
    fp.gate = h->gate;
    fp.hbuf = h->hbuf;
    fp.zbuf = h->zbuf;
    fp.out = static_cast<uint16_t *>(out_dev);
    fp.sync = h->sync;
    fp.err = h->err_word;
    fp.trace = h->trace;
    fp.d = h->d;
    fp.F = h->F;
    fp.Fpad = (h->F + 255) / 256 * 256;
    fp.E = h->E;
    fp.k = h->k;
    fp.T = T;
    fp.n_shared = h->n_shared;
    FfnGeometry geo;
    if (ffn_stream_geometry(h->cfg, h->d, h->F, T, &geo) != cudaSuccess)
        return MELINOE_ERR_UNSUPPORTED;
    // calls of more than 8 tokens go through the grouped GEMM (where the shapes allow it)
    const bool use_gemm = h->gemm_ok && T > kTokPerVr && h->xs != nullptr;
    // Alternative for calls with many tokens per expert: 256-token tiles on CTA pairs (each B tile staged
    // once per 256 rows).  Measured no faster than single CTAs (Phi-3.5-shaped prompt 1097 against
    // 1126 TFLOP/s, DeepSeek-shaped 1026 against 1015), so it runs only when MELINOE_MOE_PAIR is set.
    const bool use_pair = use_gemm && h->pair_ok && (long long)T * h->k >= (long long)192 * h->E &&
                          std::getenv("MELINOE_MOE_PAIR") != nullptr;
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
    h->last_used_gemm = use_gemm;
    h->last_used_pair = use_pair;
    if (use_gemm)
        CU_TRY(launch_gather_rows(s, h->plan, static_cast<const uint16_t *>(hidden_dev), h->tok_of_sorted, h->xs, h->d,
                                  T * h->k + h->n_shared * T, h->n_sms));
    auto launch_group = [&](int g) -> int {
        TimedPair tp{nullptr, nullptr};
        if (h->timing) {
            if (!h->free_pairs.empty()) {
                tp = h->free_pairs.back();
                h->free_pairs.pop_back();
            } else {
                CU_TRY(cudaEventCreate(&tp.a));
                CU_TRY(cudaEventCreate(&tp.b));
            }
            CU_TRY(cudaEventRecord(tp.a, s));
        }
        if (use_gemm) {
            gp.group = g;
            if (use_pair) {
                CU_TRY(launch_ffn_gemm_pair(s, 1, h->n_sms, gp));
                CU_TRY(launch_ffn_gemm_pair(s, 2, h->n_sms, gp));
            } else {
                CU_TRY(launch_ffn_gemm(s, 1, h->n_sms, gp));
                CU_TRY(launch_ffn_gemm(s, 2, h->n_sms, gp));
            }
        } else {
            fp.group = g;
            CU_TRY(launch_ffn_stream(s, h->cfg, geo, fp));
        }
        if (h->timing) {
            CU_TRY(cudaEventRecord(tp.b, s));
            h->timed.push_back(tp);
        }
        return MELINOE_OK;
    };
    // group 0 (experts resident at call entry, shared experts) goes out before the plan is known
    rc = launch_group(0);
    if (rc != MELINOE_OK)
        return rc;

    // the miss queue of this call
    rc = wait_for_plan(h, h->call_seq);
    if (rc != MELINOE_OK) {
        h->sticky.store(rc);
        return rc;
    }
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
            if (now_s() - t0 > 10.0) {
                h->sticky.store(MELINOE_ERR_TIMEOUT);
                return MELINOE_ERR_TIMEOUT;
            }
        }
    }
    // which groups must signal their completion to the copy stream
    bool need_done[kMaxGroups + 1] = {false};
    for (int i = 0; i < n_miss; ++i)
        if (hp.miss[i].dep_group >= 0 && hp.miss[i].dep_group <= kMaxGroups)
            need_done[hp.miss[i].dep_group] = true;
    auto group_event = [&](int g) -> cudaEvent_t {
        while ((int)h->ev_group.size() <= g) {
            cudaEvent_t e = nullptr;
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess)
                return nullptr;
            h->ev_group.push_back(e);
        }
        return h->ev_group[g];
    };
    if (need_done[0]) {
        cudaEvent_t e = group_event(0);
        if (!e)
            return cuda_fail(cudaGetLastError());
        CU_TRY(cudaEventRecord(e, s));
    }
    int i = 0;
    for (int g = 1; g < n_groups; ++g) {
        TimedPair ctp{nullptr, nullptr};
        bool wave_started = false;
        for (; i < n_miss && hp.miss[i].group == g; ++i) {
            const HostMiss m = hp.miss[i];
            if (m.expert < 0 || m.expert >= h->E || m.slot < 0 || m.slot >= h->C || m.dep_group >= g) {
                h->sticky.store(MELINOE_ERR_STATE);
                return MELINOE_ERR_STATE;
            }
            // the slot may still feed an earlier compute group of this call: whoever writes the slot
            // (the copy itself, or the expansion kernel of a 4-bit store) waits for that group
            cudaStream_t slot_writer = h->store_q4 ? h->dq_stream : h->copy_stream;
            if (m.dep_group >= 0)
                CU_TRY(cudaStreamWaitEvent(slot_writer, h->ev_group[m.dep_group], 0));
            if (h->timing && !wave_started) {
                if (!h->free_pairs.empty()) {
                    ctp = h->free_pairs.back();
                    h->free_pairs.pop_back();
                } else {
                    CU_TRY(cudaEventCreate(&ctp.a));
                    CU_TRY(cudaEventCreate(&ctp.b));
                }
                CU_TRY(cudaEventRecord(ctp.a, h->copy_stream));
                wave_started = true;
            }
            if (h->timing)
                h->timed_copy_bytes += h->store_q4 ? h->q4_bytes : h->expert_bytes;
            if (h->store_q4) {
                // the 4-bit blob travels into one of two staging buffers; a kernel on a stream of its own
                // expands it into the slot, so the next blob is on the link meanwhile
                const unsigned b = h->q4_turn++ & 1u;
                char *stage = h->q4_stage + (size_t)b * h->q4_bytes;
                if (h->q4_used[b])
                    CU_TRY(cudaStreamWaitEvent(h->copy_stream, h->ev_q4_expanded[b], 0));
                CU_TRY(cudaMemcpyAsync(stage, h->host_experts[m.expert], h->q4_bytes, cudaMemcpyHostToDevice,
                                       h->copy_stream));
                CU_TRY(cudaEventRecord(h->ev_q4_copied[b], h->copy_stream));
                CU_TRY(cudaStreamWaitEvent(h->dq_stream, h->ev_q4_copied[b], 0));
                CU_TRY(launch_dequant_q4(h->dq_stream, stage, h->slots + (size_t)m.slot * h->slot_stride, h->d, h->F,
                                         h->n_sms));
                CU_TRY(cudaEventRecord(h->ev_q4_expanded[b], h->dq_stream));
                h->q4_used[b] = true;
            } else {
                CU_TRY(cudaMemcpyAsync(h->slots + (size_t)m.slot * h->slot_stride, h->host_experts[m.expert],
                                       h->expert_bytes, cudaMemcpyHostToDevice, h->copy_stream));
            }
        }
        if (wave_started) {
            CU_TRY(cudaEventRecord(ctp.b, h->copy_stream));
            h->timed_copy.push_back(ctp);
        }
        CU_TRY(cudaEventRecord(h->ev_arrive, h->store_q4 ? h->dq_stream : h->copy_stream));
        CU_TRY(cudaStreamWaitEvent(s, h->ev_arrive, 0));
        rc = launch_group(g);
        if (rc != MELINOE_OK)
            return rc;
        if (need_done[g]) {
            cudaEvent_t e = group_event(g);
            if (!e)
                return cuda_fail(cudaGetLastError());
            CU_TRY(cudaEventRecord(e, s));
        }
    }

    if (use_gemm)
        CU_TRY(launch_combine_rows(s, h->plan, h->gate, h->inv_pos, h->zbuf, static_cast<uint16_t *>(out_dev), T, h->d,
                                   h->k, h->n_shared, h->n_sms));
    CU_TRY(cudaEventRecord(h->ev_last, s));
    h->has_last = true;
    return MELINOE_OK;
}

}  // extern "C"

// ---------------------------------------------------------------- forward without allocation
//
// Scratch of melinoe_moe_forward_static: one array in the library's device image, shared by every
// call on the device, instead of per-handle cudaMalloc'd buffers.
constexpr int kStaticMaxTokens = 8;
constexpr int kStaticMaxPairs = 16;                         // n_tokens * top_k
constexpr int kStaticMaxSharedRows = 64;                    // n_shared * n_tokens
constexpr int kStaticMaxVr = kStaticMaxPairs + kMaxShared;  // one virtual request per routed pair or shared expert
constexpr int kStaticMaxD = 8192, kStaticMaxF = 16384;
constexpr size_t kStaticSmall = 16 * 1024;                  // idx, gate, logits, perm, inv_pos, tok_of_sorted, vrs
constexpr size_t kStaticZ = (size_t)(kStaticMaxPairs + kStaticMaxSharedRows) * kStaticMaxD * sizeof(float);
constexpr size_t kStaticH = (size_t)kStaticMaxVr * kTokPerVr * kStaticMaxF * 2;
constexpr size_t kStaticBytes = kStaticSmall + kStaticZ + kStaticH;   // about 8.6 MiB
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
    if (!h || T < 0)
        return MELINOE_ERR_INVALID;
    if (T == 0)
        return MELINOE_OK;
    // everything beyond the static scratch's sizes is refused, never served by allocating
    if (T > kStaticMaxTokens || T * h->k > kStaticMaxPairs || T * h->k > h->C || h->n_shared * T > kStaticMaxSharedRows ||
        h->d > kStaticMaxD || h->F > kStaticMaxF)
        return MELINOE_ERR_UNSUPPORTED;
    if (h->timing)
        return MELINOE_ERR_STATE;   // timed calls create events on demand
    if (h->device < 0 || h->device >= kMaxDevices)
        return MELINOE_ERR_UNSUPPORTED;
    unsigned char *base = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_static_mu);
        base = g_static_ptr[h->device];
        if (!base) {
            // first call on this device (the handle's device must be current, as for every call)
            int cur = -1;
            CU_TRY(cudaGetDevice(&cur));
            if (cur != h->device)
                return MELINOE_ERR_STATE;
            void *p = nullptr;
            CU_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
            base = g_static_ptr[h->device] = static_cast<unsigned char *>(p);
        }
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // carve the scratch: small tables first, then z, then h
    unsigned char *q = base;
    auto take = [&](size_t bytes) {
        unsigned char *r = q;
        q += (bytes + 255) / 256 * 256;
        return r;
    };
    const size_t pairs = kStaticMaxPairs, sorted = kStaticMaxPairs + kStaticMaxSharedRows;
    int32_t *idx = reinterpret_cast<int32_t *>(take(pairs * 4));
    float *gate = reinterpret_cast<float *>(take(pairs * 4));
    float *logits = reinterpret_cast<float *>(take((size_t)kStaticMaxTokens * kMaxExperts * 4));
    int32_t *perm = reinterpret_cast<int32_t *>(take(sorted * 4));
    int32_t *inv_pos = reinterpret_cast<int32_t *>(take(pairs * 4));
    int32_t *tok_of_sorted = reinterpret_cast<int32_t *>(take(sorted * 4));
    VrRec *vrs = reinterpret_cast<VrRec *>(take((size_t)kStaticMaxVr * sizeof(VrRec)));
    if ((size_t)(q - base) > kStaticSmall)
        return MELINOE_ERR_STATE;
    float *zbuf = reinterpret_cast<float *>(base + kStaticSmall);
    uint16_t *hbuf = reinterpret_cast<uint16_t *>(base + kStaticSmall + kStaticZ);
    // the padding behind every h row has to read as zero, and the array keeps whatever the last
    // call (of any handle, with any d_ff) left there
    const size_t fpad = ((size_t)h->F + 255) / 256 * 256;
    CU_TRY(cudaMemsetAsync(hbuf, 0, (size_t)kStaticMaxVr * kTokPerVr * fpad * 2, s));

    // run the ordinary call on the static scratch: swap the handle's scratch pointers for its duration
    struct Saved {
        int32_t *idx, *perm, *inv_pos, *tok_of_sorted;
        float *gate, *logits, *zbuf;
        uint16_t *hbuf;
        VrRec *vrs;
        int cap_tokens, cap_shared, vr_capacity;
    } keep{h->idx, h->perm, h->inv_pos, h->tok_of_sorted, h->gate, h->logits, h->zbuf, h->hbuf, h->vrs,
           h->cap_tokens, h->cap_shared, h->vr_capacity};
    h->idx = idx;
    h->perm = perm;
    h->inv_pos = inv_pos;
    h->tok_of_sorted = tok_of_sorted;
    h->gate = gate;
    h->logits = logits;
    h->zbuf = zbuf;
    h->hbuf = hbuf;
    h->vrs = vrs;
    h->cap_tokens = kStaticMaxTokens;
    h->cap_shared = h->n_shared;
    h->vr_capacity = kStaticMaxVr;
    const int rc = melinoe_moe_forward(h, cuda_stream, hidden_dev, T, out_dev, stats_dev);
    h->idx = keep.idx;
    h->perm = keep.perm;
    h->inv_pos = keep.inv_pos;
    h->tok_of_sorted = keep.tok_of_sorted;
    h->gate = keep.gate;
    h->logits = keep.logits;
    h->zbuf = keep.zbuf;
    h->hbuf = keep.hbuf;
    h->vrs = keep.vrs;
    h->cap_tokens = keep.cap_tokens;
    h->cap_shared = keep.cap_shared;
    h->vr_capacity = keep.vr_capacity;
    h->last_T = 0;   // the inspection calls read the handle's own scratch, which this call did not touch
    return rc;
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
    if (!h->host_experts[0])
        return MELINOE_ERR_STATE;
    int rc = wait_idle(h);
    if (rc != MELINOE_OK)
        return rc;
    DevCache c;
    CU_TRY(cudaMemcpy(&c, h->cache, sizeof c, cudaMemcpyDeviceToHost));
    for (int i = 0; i < n; ++i) {
        const int e = ids[i];
        if (e < 0 || e >= h->E)
            return MELINOE_ERR_INVALID;
        c.call_no += 1;
        const uint64_t st = ++c.counter;
        if (h->policy == MELINOE_POLICY_COUNT)
            c.count[e] += 1.0f;
        if (c.slot_of_expert[e] >= 0) {
            c.stamp[c.slot_of_expert[e]] = st;
            c.tot_hits += 1;
            continue;
        }
        int victim = -1;
        for (int s = 0; s < h->C && victim < 0; ++s)
            if (c.expert_of_slot[s] < 0)
                victim = s;
        if (victim < 0) {
            for (int s = 0; s < h->C; ++s) {
                if (victim < 0) {
                    victim = s;
                } else if (h->policy == MELINOE_POLICY_COUNT) {
                    const float cs = c.count[c.expert_of_slot[s]], cv = c.count[c.expert_of_slot[victim]];
                    if (cs < cv || (cs == cv && c.stamp[s] < c.stamp[victim]))
                        victim = s;
                } else if (c.stamp[s] < c.stamp[victim]) {
                    victim = s;
                }
            }
            c.slot_of_expert[c.expert_of_slot[victim]] = -1;
            c.tot_evictions += 1;
        }
        if (h->store_q4) {
            // the handle is idle (wait_idle above): stage, expand, wait
            CU_TRY(cudaMemcpy(h->q4_stage, h->host_experts[e], h->q4_bytes, cudaMemcpyHostToDevice));
            CU_TRY(launch_dequant_q4(h->dq_stream, h->q4_stage, h->slots + (size_t)victim * h->slot_stride, h->d, h->F,
                                     h->n_sms));
            CU_TRY(cudaStreamSynchronize(h->dq_stream));
        } else {
            CU_TRY(cudaMemcpy(h->slots + (size_t)victim * h->slot_stride, h->host_experts[e], h->expert_bytes,
                              cudaMemcpyHostToDevice));
        }
        c.expert_of_slot[victim] = e;
        c.slot_of_expert[e] = victim;
        c.stamp[victim] = st;
        c.tot_misses += 1;
    }
    CU_TRY(cudaMemcpy(h->cache, &c, sizeof c, cudaMemcpyHostToDevice));
    return MELINOE_OK;
}

int melinoe_moe_last_routing(melinoe_moe_t *h, int32_t *idx_host, float *gate_host)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    if (h->last_T <= 0)
        return MELINOE_ERR_STATE;
    const size_t n = (size_t)h->last_T * h->k;
    if (idx_host)
        CU_TRY(cudaMemcpy(idx_host, h->idx, n * 4, cudaMemcpyDeviceToHost));
    if (gate_host)
        CU_TRY(cudaMemcpy(gate_host, h->gate, n * 4, cudaMemcpyDeviceToHost));
    return MELINOE_OK;
}

int melinoe_moe_last_logits(melinoe_moe_t *h, float *logits_host)
{
    if (!h || !logits_host)
        return MELINOE_ERR_INVALID;
    if (h->last_T <= 0)
        return MELINOE_ERR_STATE;
    CU_TRY(cudaMemcpy(logits_host, h->logits, (size_t)h->last_T * h->E * 4, cudaMemcpyDeviceToHost));
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
        CU_TRY(cudaMemcpy(perm_host, h->perm, (size_t)h->last_T * h->k * 4, cudaMemcpyDeviceToHost));
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

int melinoe_moe_set_trace(melinoe_moe_t *h, void *trace_dev, size_t bytes)
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

int melinoe_moe_trace_ctas(melinoe_moe_t *h) { return h ? h->cfg.grid : 0; }

int melinoe_moe_last_call_used_gemm(melinoe_moe_t *h) { return h && h->last_used_gemm ? (h->last_used_pair ? 2 : 1) : 0; }

int melinoe_moe_enable_timing(melinoe_moe_t *h, int enable)
{
    if (!h)
        return MELINOE_ERR_INVALID;
    h->timing = enable != 0;
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
