/*
 * melinoe_moe.h - C ABI of the cached Mixture-of-Experts layer for NVIDIA B200 (sm_100a).
 *
 * One handle is one MoE layer (Section 2 of the paper, Eq. 1-3) executed under a bounded,
 * GPU-resident expert cache (Section 2 "Expert Offloading Systems", Section 3.2): all experts
 * live in page-locked host memory, `cache_slots` of them are resident in device memory, and a
 * forward call fetches the experts it misses over the host link, evicting by LRU.
 *
 * Conventions
 *  - Every function returns a melinoe_status (0 = OK).  Nothing throws, aborts or exits.
 *  - "dev" pointers are device memory on the device that was current at create time; "host"
 *    pointers are host memory.  The library never takes ownership of caller memory.
 *  - bf16 tensors are raw 16-bit patterns, row-major.
 *  - A handle is driven by one host thread at a time, and all forward calls of one handle must
 *    be ordered with respect to each other on the device (same stream, or caller-made
 *    dependencies): a call's cache decisions depend on the previous call's.
 *  - melinoe_moe_forward is asynchronous with respect to the host: for calls of at most 8 tokens
 *    (and no more token-expert pairs than cache slots) it queues two kernels and returns (the
 *    missed experts are fetched by the compute kernel itself); otherwise it returns once the call's cache decisions are known to
 *    the host and all of its transfers and kernels are queued.  It never waits for transfers or
 *    compute.
 *  - Environment switches, read once per process (for measurements and tests; none changes results):
 *    MELINOE_MOE_NO_PDL          launch the decode kernels without programmatic stream serialisation;
 *    MELINOE_MOE_HOST_COPIES     every expert transfer is a cudaMemcpyAsync issued by the host;
 *    MELINOE_MOE_GEMM_SINGLE     the prefill GEMM never pairs CTAs (tcgen05 cta_group::1 only).
 */
#ifndef MELINOE_MOE_H_
#define MELINOE_MOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct melinoe_moe melinoe_moe_t;

typedef enum melinoe_status {
    MELINOE_OK = 0,
    MELINOE_ERR_INVALID = 1,     /* bad argument (null, misaligned, out of range, not pinned) */
    MELINOE_ERR_STATE = 2,       /* call order: e.g. forward before router / experts are set  */
    MELINOE_ERR_CUDA = 3,        /* a CUDA call failed; melinoe_last_cuda_error() has its code */
    MELINOE_ERR_NOMEM = 4,       /* device or host allocation failed                           */
    MELINOE_ERR_TIMEOUT = 5,     /* a bounded device-side or host-side wait ran out            */
    MELINOE_ERR_UNSUPPORTED = 6  /* shape outside what the kernels cover                       */
} melinoe_status;

/*
 * Per-call statistics, written on the device in stream order by the call's planning kernel.
 * The caller passes device-accessible memory (device memory or page-locked host memory) and
 * reads it after synchronising the stream.  `misses` is the paper's hard miss count of the
 * call (Appendix C.1: one miss = one host-to-device expert transfer).
 */
typedef struct melinoe_moe_stats {
    int32_t status;       /* melinoe_status of the device-side part of the call            */
    int32_t n_tokens;     /* T                                                             */
    int32_t n_distinct;   /* number of distinct experts the call's tokens selected         */
    int32_t hits;         /* requests served from the cache                                */
    int32_t misses;       /* requests fetched from host memory                             */
    int32_t evictions;    /* misses that displaced a resident expert                       */
    int32_t groups;       /* compute groups the call was split in (1 + miss waves)         */
    int32_t reserved;
    uint64_t bytes_h2d;   /* misses * bytes_per_expert                                     */
    uint64_t call_no;     /* 1-based count of forward calls on this handle since reset     */
} melinoe_moe_stats;

/* One cache request of a call, in the order the cache saw it (hits in ascending expert id,
 * then misses in ascending expert id).  evicted = expert displaced, or -1. */
typedef struct melinoe_moe_request {
    int32_t expert, slot, hit, evicted;
} melinoe_moe_request;

/*
 * Request trace (optional, melinoe_moe_set_trace): one record per forward call, written on the device
 * in stream order by the call's routing / planning kernels, so that routing and cache decisions can
 * be recorded without synchronising after every call.  A record is melinoe_moe_trace_record_bytes()
 * long and holds, in this order:
 *     melinoe_moe_trace_header
 *     melinoe_moe_request  req[n_experts]         the first n_requests are the call's cache requests in order
 *     int32_t              idx[max_tokens][top_k] routing indices of the call's first max_tokens tokens
 *     float                gate[max_tokens][top_k] their gates
 * (the whole rounded up to 16 bytes).
 */
typedef struct melinoe_moe_trace_header {
    uint64_t call_no;     /* as in melinoe_moe_stats                                        */
    int32_t n_tokens;     /* T of the call (indices beyond max_tokens are not recorded)     */
    int32_t n_requests;   /* distinct routed experts of the call                            */
    int32_t hits, misses;
    int32_t status;       /* melinoe_status of the device-side part of the call             */
    int32_t reserved;
} melinoe_moe_trace_header;

/*
 * Create one layer.  Shapes follow Eq. 1-3: router W_r [n_experts][d_model]; each expert has
 * W_g, W_u [d_ff][d_model] and W_d [d_model][d_ff].  Allocates, on the current device,
 * cache_slots expert slots of melinoe_moe_expert_bytes() each plus small tables, and creates
 * a copy stream.  Limits: d_model % 256 == 0, d_model <= 4096, d_ff % 8 == 0,
 * 1 <= top_k <= n_experts <= 64, top_k <= 32, top_k <= cache_slots <= n_experts  (INVALID / UNSUPPORTED
 * otherwise).
 */
int melinoe_moe_create(int d_model, int d_ff, int n_experts, int top_k, int cache_slots,
                       melinoe_moe_t **out);

/*
 * Same layer with 4-bit cache slots (Section 3.2 and Appendix D.5: 4-bit experts let the same memory hold
 * about 3.76 times as many of them): a slot is melinoe_moe_expert_bytes_q4() long, the store is registered
 * with melinoe_moe_register_host_experts_q4 and a miss is a plain copy of the 4-bit blob; the compute
 * kernel expands the codes in registers on their way into the tensor-core fragments, so HBM and the
 * host link only ever carry 4-bit data.  The layer computes with exactly the weights the format defines
 * (see melinoe_moe_pack_expert_q4).  Shared experts, if any, are registered as 4-bit blobs too.  Calls of
 * every size run the decode kernel, 8 tokens per launch (there is no 4-bit grouped GEMM).  Needs
 * d_model = 512, 1024, 2048 or 4096 on top of the limits above.
 */
int melinoe_moe_create_q4(int d_model, int d_ff, int n_experts, int top_k, int cache_slots,
                          melinoe_moe_t **out);

/* Waits for the handle's outstanding transfers and device work, then frees everything the
 * library allocated.  Caller memory (router, experts, bias) is untouched. */
int melinoe_moe_destroy(melinoe_moe_t *h);

/* Bytes of one packed expert: 3 * d_model * d_ff * 2. */
size_t melinoe_moe_expert_bytes(int d_model, int d_ff);

/*
 * Pack one expert from the paper's matrices (Eq. 3: W_g, W_u [d_ff][d_model], W_d [d_model][d_ff];
 * bf16, row-major, host memory) into one contiguous blob (host memory, `melinoe_moe_expert_bytes`
 * long).  The blob holds, for every hidden unit f = 0 .. d_ff - 1, the three vectors that belong to
 * it back to back, 3 * d_model elements:
 *     W_g[f][0 .. d_model) | W_u[f][0 .. d_model) | W_d[0 .. d_model)[f]
 * so that everything f contributes to the layer's output (Eq. 3) is one contiguous byte range, and
 * any run of consecutive f is too.  Within each of the three vectors, every group of 64 elements
 * (128 bytes) has its eight 16-byte pieces stored at position (piece xor (f mod 8)): shared-memory
 * bank conflicts of the kernels' tensor-core fragment loads are avoided by this permutation, and it
 * is the arrangement the tensor cores' 128-byte-swizzled operand layout expects.  Pure host code;
 * does not touch the device.  blob_out must not overlap the inputs.  d_model % 64 == 0.
 */
int melinoe_moe_pack_expert(int d_model, int d_ff, const void *w_gate_host, const void *w_up_host,
                            const void *w_down_host, void *blob_out_host);

/*
 * 4-bit expert format (Section 3.2 keeps the expert weights in 4-bit form; the calibrated HQQ format
 * of the paper is a third-party method, what is implemented is plain symmetric group
 * quantisation).  Every vector of d_model weights that belongs to one hidden unit f -- W_g[f],
 * W_u[f] and column f of W_d -- is cut into groups of 64 consecutive elements; a group's scale is
 * bf16(max|w| / 7); code = clamp(rint(w / scale), -8, 7) + 8, ties to even; the weight the layer
 * computes with is bf16(scale * (code - 8)).  Blob of one expert, `melinoe_moe_expert_bytes_q4`
 * long (3.76 times smaller than the bf16 blob): for every hidden unit f a unit of
 * ceil16(3 * d_model / 2 + 3 * (d_model / 64) * 2) bytes holding
 *     codes W_g[f] | codes W_u[f] | codes W_d[:, f]    d_model / 2 bytes each, even element in the low nibble
 *     scales W_g[f] | scales W_u[f] | scales W_d[:, f]  d_model / 64 bf16 each
 * then zero padding to a multiple of 16 bytes (none when d_model % 512 == 0).  Within each code
 * vector, the 16-byte pieces of every group of eight sit at position (piece xor (f mod 8)); in the
 * codes of W_d[:, f], position p of a group of 64 holds element 8 (p mod 8) + p / 8 of that group (the
 * order in which the compute kernel's output fragments own the columns).  As in
 * the bf16 blob, everything f contributes is one contiguous byte range.  Needs d_model % 256 == 0 and
 * d_ff % 8 == 0 (else the size is 0 and packing returns MELINOE_ERR_UNSUPPORTED).  Pure host code.
 */
size_t melinoe_moe_expert_bytes_q4(int d_model, int d_ff);
int melinoe_moe_pack_expert_q4(int d_model, int d_ff, const void *w_gate_host, const void *w_up_host,
                               const void *w_down_host, void *blob_out_host);

/* Router matrix W_r (Eq. 1): dev pointer, [n_experts][d_model] bf16, 16-byte aligned, borrowed
 * until the handle is destroyed or the router is replaced.  Its contents must not change while a
 * forward call is queued or running (a decode call may read it before the work ahead of it in the
 * stream has finished). */
int melinoe_moe_set_router(melinoe_moe_t *h, const void *w_router_dev);

/*
 * The host-resident expert store (Section 3.2: offloaded experts stay in pinned CPU memory).
 * expert_host_ptrs[e] points to expert e packed by melinoe_moe_pack_expert, in page-locked
 * host memory, 16-byte aligned; bytes_per_expert must equal melinoe_moe_expert_bytes().
 * Pointers are checked with the CUDA runtime: pageable memory is rejected with INVALID (the
 * library never stages silently).  Borrowed, read-only, must outlive the handle.  Where the device
 * can address the store (memory from cudaHostAlloc, or registered with cudaHostRegister), calls of
 * at most 8 tokens read the experts they miss straight from it inside the compute kernel, with no
 * host involvement; MELINOE_MOE_HOST_COPIES in the environment keeps every transfer a
 * cudaMemcpyAsync issued by the host.
 */
int melinoe_moe_register_host_experts(melinoe_moe_t *h, const void *const *expert_host_ptrs,
                                      size_t bytes_per_expert);   /* UNSUPPORTED on a handle with 4-bit slots */

/*
 * Same registration for a store of 4-bit blobs (melinoe_moe_pack_expert_q4).  On a handle with 4-bit slots
 * (melinoe_moe_create_q4) this is the one way to register the store, and everything said above holds.
 * On a handle with bf16 slots a miss then moves the
 * 4-bit blob over the host link (3.76 times fewer bytes, which is what a miss costs, Eq. 4) and a
 * kernel expands it into the bf16 slot behind the copy, so the cache slots and the compute kernels
 * are the same as with a bf16 store and the layer computes with exactly the weights the format
 * defines.  The statistics count the bytes that travelled.  Transfers of such a store are issued by
 * the host (the forward call waits for the call's cache decisions, see melinoe_moe_forward).
 * Page-locked, 16-byte aligned, borrowed, as above.  Registering one kind of store replaces the
 * other; the cache should be reset when the store changes.
 */
int melinoe_moe_register_host_experts_q4(melinoe_moe_t *h, const void *const *expert_host_ptrs,
                                         size_t bytes_per_expert);

/* Always-resident shared experts (not in the paper; DeepSeekMoE-style stacks): blobs packed in
 * the format of the handle's slots, in DEVICE memory, applied to every token with gate 1, never cached, never counted in
 * hits or misses.  n_shared <= 8.  Borrowed. */
int melinoe_moe_register_shared_experts(melinoe_moe_t *h, int n_shared,
                                        const void *const *expert_dev_ptrs);

/*
 * Optional additive router bias (emulates a fine-tuned, sequence-concentrated router):
 * logits = W_r x + seq_bias[token_seq[t]].  seq_bias_dev [n_seq][n_experts] fp32;
 * token_seq_dev [T] int32 with values in [0, n_seq), or NULL = every token uses row 0.
 * seq_bias_dev == NULL restores Eq. 1 exactly.  Borrowed; takes effect for later calls.
 */
int melinoe_moe_set_router_bias(melinoe_moe_t *h, const float *seq_bias_dev,
                                const int32_t *token_seq_dev, int n_seq);

/* Make room for calls of up to max_tokens tokens (scratch grows on demand otherwise, which
 * synchronises the device). */
int melinoe_moe_reserve(melinoe_moe_t *h, int max_tokens);

/*
 * One forward call of the layer for n_tokens tokens (Eq. 1-3 under the cache):
 * router softmax + top-k (ties to the lowest expert id), slot lookup with LRU eviction,
 * asynchronous fetch of the missed experts from host memory on the handle's copy stream
 * overlapped with the compute of the resident ones, token-to-expert gather, SwiGLU expert
 * FFN with fp32 accumulation, and the gate-weighted sum, rounded once to bf16.
 * Gates are renormalised over the selected experts (they sum to 1 per token).
 *
 * cuda_stream: a cudaStream_t (NULL = legacy default stream).  hidden_dev [n_tokens][d_model]
 * bf16 and out_dev [n_tokens][d_model] bf16 are device memory, 16-byte aligned, borrowed
 * until the stream work of this call has finished.  stats_dev: see melinoe_moe_stats; may be
 * NULL.  n_tokens == 0 is a no-op.
 *
 * Host behaviour.  Calls of at most 8 tokens (or of any size on shapes the grouped GEMM does not
 * cover) on a bf16 store the device can address: the routing / planning kernel and the expert-FFN
 * kernel are queued and the call returns; the FFN kernel reads the experts the call misses from the
 * host store itself, stores those that stay resident into their slots, and writes the result.  The
 * host learns the call's cache decisions only through stats_dev.
 * All other calls (more than 8 tokens through the grouped GEMM; a 4-bit store; host copies forced):
 * the router, planning and resident-expert kernels are queued first; the call then waits (bounded;
 * TIMEOUT after 60 s) until the planning kernel has published the call's miss queue in page-locked
 * memory, issues one cudaMemcpyAsync per missed expert on the handle's copy stream, ties the streams
 * together with events, queues the remaining kernels and returns.  It then waits for earlier work on
 * cuda_stream, but never for its own transfers, FFN kernels or combine.  If queuing fails part-way,
 * the error is returned, stays on the handle (every later call returns it until
 * melinoe_moe_reset_cache) and the handle can still be synchronised and destroyed.
 */
int melinoe_moe_forward(melinoe_moe_t *h, void *cuda_stream, const void *hidden_dev,
                        int n_tokens, void *out_dev, melinoe_moe_stats *stats_dev);

/*
 * Same call with HOST buffers: copies hidden_host to the device, runs the layer, copies the
 * result to out_host and (if not NULL) the statistics to stats_host, all in stream order.
 * Page-locked buffers make the copies asynchronous; pageable buffers work but block.  For calls of
 * at most 8 tokens with page-locked (device-mapped), 16-byte aligned hidden_host / out_host and
 * 8-byte aligned stats_host, a small kernel fetches the input and the layer's kernels write the
 * result and the statistics straight into those buffers (no copy-engine operation at all); they
 * are complete when the stream reaches the end of the call, as with the copies.
 */
int melinoe_moe_forward_host(melinoe_moe_t *h, void *cuda_stream, const void *hidden_host,
                             int n_tokens, void *out_host, melinoe_moe_stats *stats_host);

/*
 * melinoe_moe_forward for callers that must not allocate (no counterpart in the paper).
 *
 * melinoe_moe_forward grows its per-handle scratch with cudaMalloc when a call is larger than
 * anything seen before, and creates CUDA events on demand.  Some callers cannot have that happen
 * inside the call: a serving loop that has handed all remaining device memory to a KV cache or to
 * another allocator and would get an out-of-memory error (or a device-wide synchronisation) from a
 * stray cudaMalloc, and code that runs where the CUDA allocator must not be entered at all.  This
 * entry point runs the same layer, same kernels and same cache state, but takes every byte of
 * scratch (routing tables, gather lists, the FFN kernel's per-SM partial outputs) from one array
 * of melinoe_moe_static_scratch_bytes() (400 KiB) that is part of the library's device
 * image: each GPU that loads the library holds it until the process exits.  It calls no
 * cudaMalloc, cudaFree, event-creating or otherwise allocating routine, under either eviction
 * policy (the events a call may need are made when the handle is created).
 *
 * Limits, all checked before anything is queued, MELINOE_ERR_UNSUPPORTED beyond them:
 *   n_tokens <= 8 and n_tokens * top_k <= 64 (every width the library supports fits).
 * MELINOE_ERR_STATE if kernel timing is enabled on the handle (timed calls create events), or if
 * the handle's device is not the current one.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) with
 * that device current; make this first call before any stream capture begins.
 * Every call on a device, of every handle, uses the same array: it keeps the previous call's
 * contents (the tables are written by the call's own kernels before they are read; the one part that
 * has to start from zero, the output accumulator, is cleared by the kernel that used it), and two
 * such calls that can overlap on the GPU (different streams without an
 * ordering between them) race on it.  Calls on one stream, or ordered by events, are safe, and may
 * be mixed freely with melinoe_moe_forward on the same handle.
 * The inspection calls (melinoe_moe_last_*) read the scratch of the most recent call, so after a
 * call through this entry point they are valid only until the next static call on the device.
 * Arguments and results otherwise as melinoe_moe_forward.
 */
int melinoe_moe_forward_static(melinoe_moe_t *h, void *cuda_stream, const void *hidden_dev,
                               int n_tokens, void *out_dev, melinoe_moe_stats *stats_dev);
size_t melinoe_moe_static_scratch_bytes(void);

/*
 * Eviction policy of the handle's cache (Section 4: the paper's experiments run an LFU cache;
 * Definition C.1: the gamma-discounted count whose Top-C is the cache state, gamma = 1 being LFU
 * and gamma -> 0+ LRU).
 *   MELINOE_POLICY_LRU    (default) a miss takes the lowest empty slot, else the least recently
 *                         requested expert's slot;
 *   MELINOE_POLICY_COUNT  every forward call is one time step: each expert's count becomes
 *                         gamma * count + (requested by this call ? 1 : 0), in fp32 with the product
 *                         rounded before the sum; a miss takes the lowest empty slot, else the slot
 *                         of the expert with the smallest count, the less recently requested one on
 *                         ties.  0 <= gamma <= 1.  A preloaded expert's count is raised by one
 *                         without a decay step.
 * Takes effect from the next call; the cache contents and the counts are kept (the counts are
 * maintained only while the count policy is set; melinoe_moe_reset_cache zeroes them).  Under the
 * count policy a call's misses may form up to one compute group each (a freshly fetched expert
 * has the smallest count), so they are served with less overlap than under LRU.  Waits for the
 * handle's queued calls.  Returns MELINOE_ERR_INVALID for an unknown policy or a gamma out of range.
 */
#define MELINOE_POLICY_LRU 0
#define MELINOE_POLICY_COUNT 1
int melinoe_moe_set_policy(melinoe_moe_t *h, int policy, float gamma);

/* The experts' discounted counts (see melinoe_moe_set_policy): counts_host [n_experts] fp32.
 * Waits for the handle's queued calls. */
int melinoe_moe_cache_counts(melinoe_moe_t *h, float *counts_host);

/*
 * Cache-miss proxies of a recorded routing trace, forward only: what a cache of a given size
 * would have cost on routing that has already happened, for choosing per-layer cache sizes under
 * one memory budget.  No handle and no expert weights are involved.
 *   soft  Section 3.1: the mean over the layer's tokens of sum_i r_i (1 - c_i), c the soft cache
 *         state of the cache simulation loss (zero start, un-normalised fill until its L1 norm
 *         reaches C, the update that reaches C rescaled to exactly C, then the normalised update
 *         with Z' = gamma Z + K / C): the layer's term of L_cs;
 *   hard  Definition C.1: requested experts outside Top-C of the gamma-discounted counts (zero
 *         start, only non-zero counts are resident, lower index first among equal counts), summed
 *         over the tokens: the transfers of a gamma-cache (Appendix C.1).
 * trace_dev [n_layers][n_tokens][top_k] int32 expert ids (device); configs_dev [n_configs]
 * (device), each naming a layer, a cache size in [1, n_experts] and a gamma in [0, 1];
 * soft_mean_dev [n_configs] fp64 and hard_total_dev [n_configs] int64 (device) receive the
 * results.  Asynchronous on cuda_stream.  fp64 throughout; n_experts <= 64, top_k <= n_experts.
 * A configuration whose layer, cache size or gamma is out of range is not evaluated: its results
 * are NaN and -1.  Expert ids outside [0, n_experts) match no expert; the trace is expected to be
 * one the router produced (top_k distinct experts per token).
 */
typedef struct melinoe_proxy_config {
    int32_t layer;
    int32_t cache_slots;
    double gamma;
} melinoe_proxy_config;
int melinoe_trace_miss_proxies(void *cuda_stream, const int32_t *trace_dev, int n_layers, int n_tokens, int top_k,
                               int n_experts, const melinoe_proxy_config *configs_dev, int n_configs,
                               double *soft_mean_dev, int64_t *hard_total_dev);

/* Cold start: all slots empty, stamps and totals zero.  Synchronises the handle first. */
int melinoe_moe_reset_cache(melinoe_moe_t *h);

/*
 * Post-deployment prefetch of Section 3.2 (Eq. 5: the Top-C experts the activation predictor names
 * are loaded into the cache before generation begins; the predictor itself is not part of this
 * library, the caller supplies the set).  Up to cache_slots expert ids, host memory; each id is one
 * cache request of its own, in the order given, as if it were the only expert of a call: a
 * resident expert is re-stamped (counted as a hit), a missing one takes the lowest empty slot,
 * else the policy's victim (counted as a miss; under the count policy every id's count is raised
 * by one without a decay step).
 * The call queues its work on the handle's copy stream, behind everything already queued on the
 * handle, and returns: on a bf16 store the device can address, a planning kernel and a copy kernel
 * that reads the experts over the host link itself (the host is not involved); otherwise the host
 * waits for the planning kernel's list and issues one cudaMemcpyAsync per expert.  The next forward
 * call of the handle, on whatever stream, waits for the preload on the device before it starts.
 */
int melinoe_moe_preload(melinoe_moe_t *h, const int32_t *expert_ids_host, int n);

/*
 * The same for a batch (Section 4.3 "Effect of Batch Size": the predictor pools the most likely
 * experts across all sequences of the batch; the paper does not say how, the reading taken here is
 * a vote).  lists_host [n_seq][per_seq] int32: every sequence's own predicted set.  An expert's
 * vote is the number of sequences whose list contains it; the cache_slots experts with the most
 * votes (at least one), the lower id first among equals, are preloaded in that order.
 */
int melinoe_moe_preload_pooled(melinoe_moe_t *h, const int32_t *lists_host, int n_seq, int per_seq);

/*
 * Inspection (synchronise the stream first; these copy from the device and block).
 * last_routing: idx [T][top_k] int32 and gates [T][top_k] fp32 of the most recent call.
 * last_logits: the router logits (argument of the softmax in Eq. 1, bias included).
 * last_requests: the most recent call's cache requests in order; *n_out receives their count
 *   (capacity n_experts records).
 * last_gather: counts [n_experts], offsets [n_experts+1], perm [T*top_k] (flat pair indices
 *   t*top_k + j grouped by expert, ascending within an expert).
 * cache_state: expert_of_slot [cache_slots] (-1 = empty) and totals {hits, misses, evictions}.
 * Any output pointer may be NULL.
 */
int melinoe_moe_last_routing(melinoe_moe_t *h, int32_t *idx_host, float *gate_host);
int melinoe_moe_last_logits(melinoe_moe_t *h, float *logits_host /* [T][n_experts] fp32 */);
int melinoe_moe_last_requests(melinoe_moe_t *h, melinoe_moe_request *req_host, int *n_out);
int melinoe_moe_last_gather(melinoe_moe_t *h, int32_t *counts_host, int32_t *offsets_host,
                            int32_t *perm_host);
int melinoe_moe_cache_state(melinoe_moe_t *h, int32_t *expert_of_slot_host, uint64_t *totals_host);

/*
 * Kernel timing for benchmarks: when enabled, every forward call brackets its expert-FFN
 * launches with CUDA events on the caller's stream; melinoe_moe_ffn_time_ms returns, for the
 * calls since the last query, the summed FFN time (ms) and the number of FFN launches and
 * resets both.  Synchronises the recorded events.
 */
int melinoe_moe_enable_timing(melinoe_moe_t *h, int enable);
int melinoe_moe_ffn_time_ms(melinoe_moe_t *h, double *ms_out, int64_t *launches_out);
/* The same launches one by one, in launch order, without resetting anything: up to `capacity` times
 * (ms) into ms_out; *n_out receives the number of timed launches recorded since the last
 * melinoe_moe_ffn_time_ms.  With one FFN launch per call (calls of at most 8 tokens on a store the
 * device can address) entry i belongs to the i-th call, whose statistics say what it fetched. */
int melinoe_moe_ffn_launch_times_ms(melinoe_moe_t *h, float *ms_out, int capacity, int *n_out);
/* With timing enabled, every wave of miss transfers is bracketed by events on the copy stream
 * as well: summed copy-stream time (ms) and bytes moved host-to-device since the last query
 * (Eq. 4's N_miss * Time_transfer, measured).  Resets both. */
int melinoe_moe_transfer_time_ms(melinoe_moe_t *h, double *ms_out, uint64_t *bytes_out);

/*
 * Request trace of the handle's forward calls.  trace_buf: device memory (or page-locked host memory
 * the device can address), 16-byte aligned, borrowed; bytes: its size; max_tokens: tokens per call
 * whose routing is recorded.  The buffer is used as a ring of bytes / melinoe_moe_trace_record_bytes()
 * records: the n-th call after this call (n = 1, 2, ...) writes record (n - 1) mod capacity.  The
 * records of calls that have finished on the device are valid (synchronise the stream, or an event
 * behind the calls, before reading).  NULL switches the trace off.  melinoe_moe_trace_count returns
 * the number of calls recorded since the trace was set.  INVALID if the buffer holds no record.
 * A recorded routing trace (the idx arrays of consecutive calls) is what melinoe_trace_miss_proxies
 * evaluates.
 */
size_t melinoe_moe_trace_record_bytes(melinoe_moe_t *h, int max_tokens);
int melinoe_moe_set_trace(melinoe_moe_t *h, void *trace_buf, size_t bytes, int max_tokens);
int64_t melinoe_moe_trace_count(melinoe_moe_t *h);

/*
 * Per-layer cache sizes under one budget (the paper names per-layer cache budgets as future work in
 * its limitations; Section 3.1 / Definition C.1 give the miss counts this works on).  Pure host code.
 * hard_host [n_layers][n_sizes] int64: transfers of layer l with first_size + j slots (what
 * melinoe_trace_miss_proxies returns as hard totals for consecutive cache sizes).  Every layer starts
 * at first_size slots; the rest of budget (total slots over all layers) is handed out one slot at a
 * time to the layer whose next slot saves the most transfers, the lower layer first among equals,
 * until the budget is spent or no layer can grow.  slots_out [n_layers] receives the sizes.
 * INVALID if the budget does not cover first_size slots per layer.
 */
int melinoe_allocate_slots(const int64_t *hard_host, int n_layers, int n_sizes, int first_size, int64_t budget,
                           int32_t *slots_out);

/*
 * Kernel timeline for profiling (no counterpart in the paper).  trace_dev: device memory of at
 * least 8 * 8 bytes per SM of the device (melinoe_moe_timeline_ctas() * 64 bytes), 8-byte aligned,
 * borrowed; NULL switches tracing off.  Every launch of the decode FFN kernel then overwrites, per
 * CTA, eight 64-bit nanosecond stamps of the device's global timer: 0 entry, 1 set-up done (plan
 * read, rows dealt out), 2 first tile of weights landed, 3 last tile computed, 4 partial output added
 * and counted out, 5 (last CTA only) sums complete, 6 (last CTA only) output written, 7 exit.  Stamps of
 * steps a CTA skipped keep their old value.
 */
int melinoe_moe_set_timeline(melinoe_moe_t *h, void *trace_dev, size_t bytes);
int melinoe_moe_timeline_ctas(melinoe_moe_t *h);

/* 1 if the most recent forward call of the handle ran its expert FFN as the tensor-core grouped
 * GEMM (calls of more than 8 tokens on shapes with d_model % 256 == 0 and d_ff % 128 == 0), 0 if it
 * ran the decode kernel (in slices of 8 tokens where the call had more). */
int melinoe_moe_last_call_used_gemm(melinoe_moe_t *h);

/* Test hook, host side only: the nth host-issued expert copy from now (cudaMemcpyAsync of a miss
 * wave; n >= 1) is not issued and reports a CUDA failure instead, so that the error path of a
 * partly queued call can be exercised without any fault on the device.  0 switches it off. */
int melinoe_debug_fail_host_copy(int nth);

/* Number of kernels this library has launched in this process (all handles). */
int64_t melinoe_launch_count(void);

/* Last CUDA error code seen by the library in this process (0 = none). */
int melinoe_last_cuda_error(void);

const char *melinoe_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* MELINOE_MOE_H_ */
