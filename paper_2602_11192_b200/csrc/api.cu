// Host side of the C ABI: handle management, launch sequencing, and the transfer service that
// turns the device-written miss queue into cudaMemcpyAsync calls on a side copy stream.
//
// Ordering of one forward call on the caller's stream:
//   router -> plan -> FFN(group 0: resident experts) -> [wait wave 1] FFN(group 1) -> ...
//   -> combine.
// The waits are stream memory operations (cuStreamWaitValue32) on a device word that the copy
// stream advances (cuStreamWriteValue32) after each wave's transfers, so the host never blocks
// in forward(), and a call without misses is released by the planning kernel itself without
// touching the host at all.  The number of FFN launches is fixed per call shape
// (1 + ceil(min(E, T*k) / C)); launches whose group turns out empty exit immediately.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <chrono>
#include <condition_variable>
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

}  // namespace melinoe

namespace {

typedef CUresult (*stream_value_fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
stream_value_fn g_wait_value = nullptr, g_write_value = nullptr;
std::once_flag g_entry_once;

void load_entry_points()
{
    std::call_once(g_entry_once, [] {
        cudaDriverEntryPointQueryResult qr;
        void *fw = nullptr, *fr = nullptr;
        if (cudaGetDriverEntryPoint("cuStreamWaitValue32", &fw, cudaEnableDefault, &qr) == cudaSuccess)
            g_wait_value = reinterpret_cast<stream_value_fn>(fw);
        if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &fr, cudaEnableDefault, &qr) == cudaSuccess)
            g_write_value = reinterpret_cast<stream_value_fn>(fr);
        (void)cudaGetLastError();
    });
}

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
    DevPlan *plan = nullptr;
    uint32_t *arrive_word = nullptr;
    int *err_word = nullptr;
    const char **shared_dev = nullptr;

    // scratch sized for cap_tokens
    int cap_tokens = 0, cap_shared = -1, vr_capacity = 0;
    int32_t *idx = nullptr, *perm = nullptr, *inv_pos = nullptr, *tok_of_sorted = nullptr;
    float *gate = nullptr, *logits = nullptr, *part = nullptr;
    VrRec *vrs = nullptr;
    uint16_t *stage_in = nullptr, *stage_out = nullptr;
    melinoe_moe_stats *stage_stats = nullptr;

    // borrowed
    const uint16_t *w_router = nullptr;
    const float *bias = nullptr;
    const int32_t *token_seq = nullptr;
    int n_seq = 0, n_shared = 0;
    std::vector<const void *> host_experts;

    // page-locked host memory
    HostPlan *hplan = nullptr;
    uint32_t *done_word = nullptr;

    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_last = nullptr;
    bool has_last = false;
    uint32_t call_seq = 0, arrive_base = 0, done_base = 0;
    int last_T = 0;

    // shared with the service thread
    std::atomic<uint32_t> enqueued{0};
    uint32_t serviced_seq = 0;
    std::atomic<uint32_t> retired{0};
    std::atomic<int> sticky{0};
    bool inline_service = false;

    // kernel timing
    bool timing = false;
    std::vector<TimedPair> timed, free_pairs;
};

namespace {

// ---------------------------------------------------------------- transfer service

// Issue the transfers of the call whose plan record sits in h->hplan.  Called with the record
// already validated (snapshot taken by the caller).
void issue_transfers(melinoe_moe *h, const HostPlan &hp)
{
    if (hp.n_miss <= 0 || hp.status != MELINOE_OK)
        return;  // the planning kernel released the waves itself
    int cur_group = -1;
    auto signal = [&](uint32_t value) {
        CUresult r = g_write_value((CUstream)h->copy_stream, (CUdeviceptr)(uintptr_t)h->arrive_word, value, 0);
        if (r != CUDA_SUCCESS) {
            // last resort so the compute stream is never left waiting: write from the host
            h->sticky.store(MELINOE_ERR_CUDA);
            cudaStreamSynchronize(h->copy_stream);
            cudaMemcpy(h->arrive_word, &value, 4, cudaMemcpyHostToDevice);
        }
    };
    for (int i = 0; i < hp.n_miss; ++i) {
        const HostMiss m = hp.miss[i];
        if (m.group != cur_group) {
            if (cur_group >= 0)
                signal(hp.arrive_base + (uint32_t)cur_group);
            cur_group = m.group;
        }
        if (m.dep_group >= 0) {
            // the slot still feeds an earlier compute group of this call: wait for that group
            const uint32_t target = hp.done_base + (uint32_t)m.dep_group + 1u;
            const double t0 = now_s();
            while ((int32_t)(*(volatile uint32_t *)h->done_word - target) < 0) {
                if (now_s() - t0 > 20.0) {
                    h->sticky.store(MELINOE_ERR_TIMEOUT);
                    break;
                }
            }
        }
        bool ok = m.expert >= 0 && m.expert < h->E && m.slot >= 0 && m.slot < h->C;
        if (ok) {
            cudaError_t e = cudaMemcpyAsync(h->slots + (size_t)m.slot * h->slot_stride, h->host_experts[m.expert],
                                            h->expert_bytes, cudaMemcpyHostToDevice, h->copy_stream);
            if (e != cudaSuccess) {
                g_last_cuda_error.store((int)e);
                h->sticky.store(MELINOE_ERR_CUDA);
            }
        } else {
            h->sticky.store(MELINOE_ERR_STATE);
        }
    }
    signal(hp.arrive_base + hp.gmax - 1u);
}

// Look at a handle's plan record; if a new, consistent one is there, serve it.
// Returns the number of calls retired.
uint32_t poll_handle(melinoe_moe *h)
{
    volatile HostPlan *vp = h->hplan;
    const uint32_t s = vp->seq;
    if (s == h->serviced_seq)
        return 0;
    std::atomic_thread_fence(std::memory_order_acquire);
    HostPlan snap;
    snap.n_miss = vp->n_miss;
    snap.n_groups = vp->n_groups;
    snap.status = vp->status;
    snap.arrive_base = vp->arrive_base;
    snap.done_base = vp->done_base;
    snap.gmax = vp->gmax;
    const int nm = snap.n_miss < 0 ? 0 : (snap.n_miss > kMaxExperts ? kMaxExperts : snap.n_miss);
    for (int i = 0; i < nm; ++i) {
        snap.miss[i].expert = vp->miss[i].expert;
        snap.miss[i].slot = vp->miss[i].slot;
        snap.miss[i].group = vp->miss[i].group;
        snap.miss[i].dep_group = vp->miss[i].dep_group;
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    if (vp->seq_open != s)
        return 0;  // a later call without misses is overwriting the record: look again
    snap.n_miss = nm;
    issue_transfers(h, snap);
    const uint32_t n = s - h->serviced_seq;
    h->serviced_seq = s;
    h->retired.fetch_add(n);
    return n;
}

class Service {
public:
    static Service &get()
    {
        static Service *s = new Service();  // never destroyed: the thread may outlive static teardown
        return *s;
    }
    void add(melinoe_moe *h)
    {
        std::lock_guard<std::mutex> lk(mu_);
        handles_.push_back(h);
        if (!started_) {
            started_ = true;
            std::thread(&Service::run, this).detach();
        }
    }
    void remove(melinoe_moe *h)
    {
        std::lock_guard<std::mutex> lk(mu_);
        for (size_t i = 0; i < handles_.size(); ++i)
            if (handles_[i] == h) {
                handles_.erase(handles_.begin() + i);
                break;
            }
    }
    void notify(melinoe_moe *h)
    {
        h->enqueued.fetch_add(1);
        pending_.fetch_add(1);
        std::lock_guard<std::mutex> lk(cv_mu_);
        cv_.notify_one();
    }

private:
    void run()
    {
        int cur_dev = -1;
        for (;;) {
            {
                std::unique_lock<std::mutex> lk(cv_mu_);
                cv_.wait(lk, [&] { return pending_.load() > 0; });
            }
            while (pending_.load() > 0) {
                std::lock_guard<std::mutex> lk(mu_);
                bool any = false;
                for (melinoe_moe *h : handles_) {
                    if (h->enqueued.load() == h->retired.load())
                        continue;
                    any = true;
                    if (h->device != cur_dev) {
                        cudaSetDevice(h->device);
                        cur_dev = h->device;
                    }
                    const uint32_t n = poll_handle(h);
                    if (n)
                        pending_.fetch_sub((int)n);
                }
                if (!any) {
                    // every live handle is drained (e.g. a handle was destroyed with calls pending)
                    pending_.store(0);
                }
            }
        }
    }
    std::mutex mu_, cv_mu_;
    std::condition_variable cv_;
    std::vector<melinoe_moe *> handles_;
    std::atomic<int> pending_{0};
    bool started_ = false;
};

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
    cudaFree(h->part);
    cudaFree(h->vrs);
    cudaFree(h->stage_in);
    cudaFree(h->stage_out);
    h->idx = h->perm = h->inv_pos = h->tok_of_sorted = nullptr;
    h->gate = h->logits = h->part = nullptr;
    h->vrs = nullptr;
    h->stage_in = h->stage_out = nullptr;
    h->cap_tokens = 0;
}

int wait_idle(melinoe_moe *h)
{
    if (h->has_last)
        CU_TRY(cudaEventSynchronize(h->ev_last));
    CU_TRY(cudaStreamSynchronize(h->copy_stream));
    if (!h->inline_service) {
        const double t0 = now_s();
        while (h->retired.load() != h->enqueued.load()) {
            if (now_s() - t0 > 30.0)
                return MELINOE_ERR_TIMEOUT;
            std::this_thread::yield();
        }
    }
    return MELINOE_OK;
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
    const size_t part_rows = ((size_t)gmax_for(h, cap) * h->cfg.grid + vr_cap) * kTokPerVr;
    CU_TRY(cudaMalloc(&h->idx, pairs * 4));
    CU_TRY(cudaMalloc(&h->gate, pairs * 4));
    CU_TRY(cudaMalloc(&h->logits, (size_t)cap * h->E * 4));
    CU_TRY(cudaMalloc(&h->perm, sorted * 4));
    CU_TRY(cudaMalloc(&h->inv_pos, pairs * 4));
    CU_TRY(cudaMalloc(&h->tok_of_sorted, sorted * 4));
    CU_TRY(cudaMalloc(&h->vrs, (size_t)vr_cap * sizeof(VrRec)));
    CU_TRY(cudaMalloc(&h->part, part_rows * h->d * sizeof(float)));
    CU_TRY(cudaMalloc(&h->stage_in, (size_t)cap * h->d * 2));
    CU_TRY(cudaMalloc(&h->stage_out, (size_t)cap * h->d * 2));
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
    const uint16_t *wg = static_cast<const uint16_t *>(wg_);
    const uint16_t *wu = static_cast<const uint16_t *>(wu_);
    const uint16_t *wd = static_cast<const uint16_t *>(wd_);
    uint16_t *blob = static_cast<uint16_t *>(blob_);
    for (int f = 0; f < F; ++f) {
        std::memcpy(blob + (size_t)(2 * f) * d, wg + (size_t)f * d, (size_t)d * 2);
        std::memcpy(blob + (size_t)(2 * f + 1) * d, wu + (size_t)f * d, (size_t)d * 2);
    }
    uint16_t *dt = blob + (size_t)2 * F * d;  // [F][d], dt[f][r] = wd[r][f]
    constexpr int B = 32;
    for (int r0 = 0; r0 < d; r0 += B)
        for (int f0 = 0; f0 < F; f0 += B) {
            const int r1 = r0 + B < d ? r0 + B : d, f1 = f0 + B < F ? f0 + B : F;
            for (int r = r0; r < r1; ++r)
                for (int f = f0; f < f1; ++f)
                    dt[(size_t)f * d + r] = wd[(size_t)r * F + f];
        }
    return MELINOE_OK;
}

int melinoe_moe_create(int d, int F, int E, int k, int C, melinoe_moe_t **out)
{
    if (!out)
        return MELINOE_ERR_INVALID;
    *out = nullptr;
    if (d <= 0 || F <= 0 || E <= 0 || k <= 0 || C <= 0 || k > E || C < k || C > E)
        return MELINOE_ERR_INVALID;
    if (d % 256 != 0 || F % kUnitRows != 0 || E > kMaxExperts || !ffn_stream_supported(d))
        return MELINOE_ERR_UNSUPPORTED;
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess)
            e = cudaFree(0);
        if (e != cudaSuccess)
            return cuda_fail(e);  // no usable device: there is no other execution path
    }
    load_entry_points();
    if (!g_wait_value || !g_write_value)
        return MELINOE_ERR_UNSUPPORTED;
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
    const char *mode = std::getenv("MELINOE_SERVICE");
    h->inline_service = mode && std::strcmp(mode, "inline") == 0;
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
    if (ffn_stream_configure(d, h->n_sms, prop.sharedMemPerBlockOptin, &h->cfg) != cudaSuccess)
        return fail(MELINOE_ERR_UNSUPPORTED);
#define CR(expr)                                   \
    do {                                           \
        cudaError_t e__ = (expr);                  \
        if (e__ != cudaSuccess)                    \
            return fail(cuda_fail(e__));           \
    } while (0)
    CR(cudaMalloc(&h->slots, h->slot_stride * (size_t)C));
    CR(cudaMalloc(&h->cache, sizeof(DevCache)));
    CR(cudaMalloc(&h->plan, sizeof(DevPlan)));
    CR(cudaMalloc(&h->arrive_word, 256));
    CR(cudaMalloc(&h->err_word, 256));
    CR(cudaMalloc(&h->shared_dev, sizeof(char *) * kMaxShared));
    CR(cudaMalloc(&h->stage_stats, sizeof(melinoe_moe_stats)));
    CR(cudaMemset(h->arrive_word, 0, 256));
    CR(cudaMemset(h->err_word, 0, 256));
    CR(cudaMemset(h->plan, 0, sizeof(DevPlan)));
    CR(cudaMemset(h->shared_dev, 0, sizeof(char *) * kMaxShared));
    DevCache c0;
    init_cache_host(c0);
    CR(cudaMemcpy(h->cache, &c0, sizeof c0, cudaMemcpyHostToDevice));
    CR(cudaHostAlloc(&h->hplan, sizeof(HostPlan), cudaHostAllocMapped | cudaHostAllocPortable));
    CR(cudaHostAlloc(&h->done_word, 256, cudaHostAllocMapped | cudaHostAllocPortable));
    std::memset(h->hplan, 0, sizeof(HostPlan));
    std::memset(h->done_word, 0, 256);
    CR(cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
    CR(cudaEventCreateWithFlags(&h->ev_last, cudaEventDisableTiming));
#undef CR
    if (!h->inline_service)
        Service::get().add(h);
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
    if (!h->inline_service)
        Service::get().remove(h);
    free_scratch(h);
    cudaFree(h->slots);
    cudaFree(h->cache);
    cudaFree(h->plan);
    cudaFree(h->arrive_word);
    cudaFree(h->err_word);
    cudaFree(h->shared_dev);
    cudaFree(h->stage_stats);
    if (h->hplan)
        cudaFreeHost(h->hplan);
    if (h->done_word)
        cudaFreeHost(h->done_word);
    if (h->copy_stream)
        cudaStreamDestroy(h->copy_stream);
    if (h->ev_last)
        cudaEventDestroy(h->ev_last);
    for (auto &p : h->timed) {
        cudaEventDestroy(p.a);
        cudaEventDestroy(p.b);
    }
    for (auto &p : h->free_pairs) {
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
    if (!h->inline_service)
        Service::get().notify(h);  // before any device work is queued: the service must be polling

    CU_TRY(launch_router(s, static_cast<const uint16_t *>(hidden_dev), h->w_router, h->bias, h->token_seq, T, h->d,
                         h->E, h->k, h->idx, h->gate, h->logits));
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
    pp.perm = h->perm;
    pp.inv_pos = h->inv_pos;
    pp.tok_of_sorted = h->tok_of_sorted;
    pp.hplan = h->hplan;
    pp.arrive_word = h->arrive_word;
    pp.arrive_base = h->arrive_base;
    pp.done_base = h->done_base;
    pp.gmax = gmax;
    pp.call_seq = h->call_seq;
    pp.stats = stats_dev;
    pp.expert_bytes = h->expert_bytes;
    pp.vr_capacity = h->vr_capacity;
    CU_TRY(launch_plan(s, pp));

    FfnParams fp;
    fp.slots = h->slots;
    fp.slot_stride = h->slot_stride;
    fp.shared_blobs = h->shared_dev;
    fp.plan = h->plan;
    fp.vrs = h->vrs;
    fp.tok_of_sorted = h->tok_of_sorted;
    fp.x = static_cast<const uint16_t *>(hidden_dev);
    fp.part = h->part;
    fp.err = h->err_word;
    fp.d = h->d;
    fp.F = h->F;
    fp.E = h->E;
    int status = MELINOE_OK;
    for (uint32_t g = 0; g < gmax; ++g) {
        if (g >= 1) {
            CUresult r = g_wait_value((CUstream)s, (CUdeviceptr)(uintptr_t)h->arrive_word, h->arrive_base + g,
                                      CU_STREAM_WAIT_VALUE_GEQ);
            if (r != CUDA_SUCCESS) {
                status = MELINOE_ERR_CUDA;
                break;
            }
        }
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
        fp.group = (int)g;
        CU_TRY(launch_ffn_stream(s, h->cfg, fp));
        if (h->timing) {
            CU_TRY(cudaEventRecord(tp.b, s));
            h->timed.push_back(tp);
        }
        if (gmax > 2 && g + 1 < gmax) {
            CUresult r = g_write_value((CUstream)s, (CUdeviceptr)(uintptr_t)h->done_word, h->done_base + g + 1u, 0);
            if (r != CUDA_SUCCESS) {
                status = MELINOE_ERR_CUDA;
                break;
            }
        }
    }
    if (status == MELINOE_OK) {
        CombineParams cp;
        cp.plan = h->plan;
        cp.idx = h->idx;
        cp.gate = h->gate;
        cp.inv_pos = h->inv_pos;
        cp.part = h->part;
        cp.out = static_cast<uint16_t *>(out_dev);
        cp.T = T;
        cp.d = h->d;
        cp.k = h->k;
        cp.E = h->E;
        cp.n_shared = h->n_shared;
        cp.grid = h->cfg.grid;
        cp.units_per_vr = h->F / kUnitRows;
        CU_TRY(launch_combine(s, cp));
    }
    CU_TRY(cudaEventRecord(h->ev_last, s));
    h->has_last = true;
    h->arrive_base += gmax;
    h->done_base += gmax;

    if (h->inline_service) {
        // debugging mode: the calling thread serves this call's misses itself (blocks until the
        // planning kernel has run)
        const double t0 = now_s();
        while (*(volatile uint32_t *)&h->hplan->seq != h->call_seq) {
            if (now_s() - t0 > 30.0)
                return MELINOE_ERR_TIMEOUT;
        }
        poll_handle(h);
    }
    if (status != MELINOE_OK)
        h->sticky.store(status);
    return status;
}

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
    CU_TRY(cudaMemcpyAsync(h->stage_in, hidden_host, bytes, cudaMemcpyHostToDevice, s));
    rc = melinoe_moe_forward(h, cuda_stream, h->stage_in, T, h->stage_out, stats_host ? h->stage_stats : nullptr);
    if (rc != MELINOE_OK)
        return rc;
    CU_TRY(cudaMemcpyAsync(out_host, h->stage_out, bytes, cudaMemcpyDeviceToHost, s));
    if (stats_host)
        CU_TRY(cudaMemcpyAsync(stats_host, h->stage_stats, sizeof(melinoe_moe_stats), cudaMemcpyDeviceToHost, s));
    CU_TRY(cudaEventRecord(h->ev_last, s));
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
            for (int s = 0; s < h->C; ++s)
                if (victim < 0 || c.stamp[s] < c.stamp[victim])
                    victim = s;
            c.slot_of_expert[c.expert_of_slot[victim]] = -1;
            c.tot_evictions += 1;
        }
        CU_TRY(cudaMemcpy(h->slots + (size_t)victim * h->slot_stride, h->host_experts[e], h->expert_bytes,
                          cudaMemcpyHostToDevice));
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
