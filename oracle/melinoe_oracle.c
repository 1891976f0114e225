/*
 * CPU oracle for the cached Mixture-of-Experts layer.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, scalar C restating what the path computes, written from the paper's
 * problem statement.  Only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may build, link or call this file; the CUDA library never does, and the two share
 * no code.
 *
 *   router            Eq. 1   p = softmax(W_r x), r = Top-K(p)
 *   layer output      Eq. 2   y = sum over selected experts of gate_i * E_i(x)
 *   expert FFN        Eq. 3   E_i(x) = W_d ( phi(W_g x) (.) W_u x ),  phi = SiLU
 *   offloading model  Section 2 "Expert Offloading Systems" and Section 3.2: a bounded
 *                     per-layer cache of resident experts, fetch on demand, eviction by
 *                     the cache policy: LRU, or the gamma-discounted count of
 *                     Definition C.1 (gamma = 1 is LFU, gamma -> 0+ reduces to LRU)
 *   miss count        Appendix C.1: number of cache misses = number of transfers
 *   4-bit store       Section 3.2: experts kept in 4-bit form in host memory (plain symmetric
 *                     group quantisation here, stated at moe_oracle_quantize_q4)
 *
 * Precision: the routing decision is an integer result, so the logits that decide it are
 * computed in fp32 in one fixed summation order (stated at moe_oracle_logits) that the GPU
 * path must reproduce bit for bit.  Everything else (gates, FFN, combine) is fp64 with no
 * intermediate rounding: it is Eq. 2-3 written out.
 *
 * The discounted counts decide an integer result (the victim), so they too are fp32 with a
 * fixed rounding order that the GPU path reproduces.
 *
 * Parity status: router indices, cache trace (both policies), gather lists and the FFN/combine are pinned
 * by the CPU tests (closed forms, brute force, library cross-checks, the paper's printed
 * transfer-time example).  Unpinned by design: exact bits of expf inside softmax gates
 * (the gates are compared within a tolerance, never bit for bit).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define MOE_ORACLE_MAX_E 4096

/* ---------------------------------------------------------------- bf16 ---------- */

static float bf16_to_f32(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

int moe_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------- 4-bit store --- */

/*
 * Group-quantised 4-bit experts (Section 3.2: expert weights are "maintained in HQQ INT4"; HQQ's
 * calibration is a third-party method and is not reproduced: this is plain symmetric
 * round-to-nearest quantisation, which is all the data path needs).  Reading:
 *  - a matrix row is cut into groups of 64 consecutive elements (cols % 64 == 0);
 *  - a group's scale is bf16( max|w| / 7 ), the division in fp32, rounded to nearest even;
 *  - code = clamp( rint(w / scale), -8, 7 ) + 8 with the division in fp32 and ties to even; a
 *    group whose scale is zero has code 8 everywhere;
 *  - the weight the layer computes with is bf16( scale * (code - 8) ), product in fp32 (exact),
 *    rounded to nearest even.
 */
static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* w [rows][cols] bf16 bits -> codes [rows][cols / 2] (low nibble = even column), scales [rows][cols / 64] bf16 bits */
int moe_oracle_quantize_q4(const uint16_t *w, int rows, int cols, uint8_t *codes, uint16_t *scales)
{
    if (rows <= 0 || cols <= 0 || cols % 64)
        return 1;
    for (int r = 0; r < rows; ++r)
        for (int g0 = 0; g0 < cols; g0 += 64) {
            const uint16_t *src = w + (size_t)r * cols + g0;
            float amax = 0.0f;
            for (int j = 0; j < 64; ++j) {
                float a = fabsf(bf16_to_f32(src[j]));
                if (a > amax)
                    amax = a;
            }
            uint16_t sb = f32_to_bf16_rne(amax / 7.0f);
            float s = bf16_to_f32(sb);
            scales[(size_t)r * (cols / 64) + g0 / 64] = sb;
            for (int j = 0; j < 64; ++j) {
                int q = 0;
                if (s > 0.0f) {
                    float t = rintf(bf16_to_f32(src[j]) / s);
                    if (t < -8.0f)
                        t = -8.0f;
                    if (t > 7.0f)
                        t = 7.0f;
                    q = (int)t;
                }
                uint8_t c = (uint8_t)(q + 8);
                uint8_t *dst = codes + ((size_t)r * cols + g0 + j) / 2;
                if (j & 1)
                    *dst = (uint8_t)((*dst & 0x0f) | (c << 4));
                else
                    *dst = (uint8_t)((*dst & 0xf0) | c);
            }
        }
    return 0;
}

int moe_oracle_dequantize_q4(const uint8_t *codes, const uint16_t *scales, int rows, int cols, uint16_t *w_out)
{
    if (rows <= 0 || cols <= 0 || cols % 64)
        return 1;
    for (int r = 0; r < rows; ++r)
        for (int j = 0; j < cols; ++j) {
            size_t at = (size_t)r * cols + j;
            int c = (j & 1) ? (codes[at / 2] >> 4) : (codes[at / 2] & 0x0f);
            float s = bf16_to_f32(scales[(size_t)r * (cols / 64) + j / 64]);
            w_out[at] = f32_to_bf16_rne(s * (float)(c - 8));
        }
    return 0;
}

/* ---------------------------------------------------------------- router -------- */

/*
 * Router logits, Eq. 1 (the argument of the softmax), plus an optional per-sequence bias.
 *
 * Inputs are bf16, so every product x_j * w_ej is exact in fp32.  The fp32 sum is taken in
 * this fixed order ("32 lanes of 8"): element j belongs to lane (j mod 256) / 8; each of the
 * 32 lanes adds its elements in increasing j into one fp32 accumulator starting from 0;
 * the 32 lane sums are then folded in five pairwise levels, s[l] <- s[l] + s[l xor m] for
 * m = 16, 8, 4, 2, 1 (every lane ends with the same value; lane 0 is taken); the fp32 bias
 * is added last.  d must be a multiple of 256.
 *
 * x [T][d], w_r [E][d] bf16 bits; bias [n_seq][E] fp32 or NULL; token_seq [T] or NULL
 * (NULL: every token uses bias row 0); logits [T][E] fp32 out.
 */
int moe_oracle_logits(const uint16_t *x, const uint16_t *w_r, const float *bias,
                      const int32_t *token_seq, int T, int d, int E, float *logits)
{
    if (d <= 0 || d % 256 != 0 || E <= 0 || T < 0)
        return 1;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const uint16_t *xt = x + (size_t)t * d;
        for (int e = 0; e < E; ++e) {
            const uint16_t *we = w_r + (size_t)e * d;
            float s[32], n[32];
            for (int l = 0; l < 32; ++l)
                s[l] = 0.0f;
            for (int j = 0; j < d; ++j) {
                int l = (j % 256) / 8;
                float prod = bf16_to_f32(xt[j]) * bf16_to_f32(we[j]);
                s[l] = s[l] + prod;
            }
            for (int m = 16; m >= 1; m >>= 1) {
                for (int l = 0; l < 32; ++l)
                    n[l] = s[l] + s[l ^ m];
                for (int l = 0; l < 32; ++l)
                    s[l] = n[l];
            }
            float v = s[0];
            if (bias) {
                int q = token_seq ? token_seq[t] : 0;
                v = v + bias[(size_t)q * E + e];
            }
            logits[(size_t)t * E + e] = v;
        }
    }
    return 0;
}

/*
 * Top-K of Eq. 1 taken on the fp32 logits (softmax is strictly increasing, so the selected
 * set is the same as Top-K of p, and no exponential takes part in an integer decision).
 * K passes of arg-max scanning e = 0..E-1 with a strict ">", so the lowest index wins a
 * tie; idx[t][0..K) is in descending-logit order.
 *
 * Gates: renormalised over the selected experts, gate_j = exp(l_j - m) / sum_i exp(l_i - m)
 * with m the largest selected logit (the K gates of a token sum to 1).  With raw_softmax != 0
 * the gate is instead the full-softmax probability p_i exactly as printed in Eq. 2.
 */
int moe_oracle_topk(const float *logits, int T, int E, int K, int raw_softmax,
                    int32_t *idx, double *gate)
{
    if (K <= 0 || K > E || E > MOE_ORACLE_MAX_E)
        return 1;
    for (int t = 0; t < T; ++t) {
        const float *l = logits + (size_t)t * E;
        unsigned char taken[MOE_ORACLE_MAX_E];
        memset(taken, 0, (size_t)E);
        for (int j = 0; j < K; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e) {
                if (taken[e])
                    continue;
                if (best < 0 || l[e] > l[best])
                    best = e;
            }
            taken[best] = 1;
            idx[(size_t)t * K + j] = best;
        }
        double m = (double)l[idx[(size_t)t * K]];
        double denom = 0.0;
        if (raw_softmax) {
            for (int e = 0; e < E; ++e)
                denom += exp((double)l[e] - m);
        } else {
            for (int j = 0; j < K; ++j)
                denom += exp((double)l[idx[(size_t)t * K + j]] - m);
        }
        for (int j = 0; j < K; ++j)
            gate[(size_t)t * K + j] = exp((double)l[idx[(size_t)t * K + j]] - m) / denom;
    }
    return 0;
}

/* ---------------------------------------------------------------- gather -------- */

/*
 * Token-to-expert lists implied by Eq. 2: for every expert the (token, rank) pairs routed to
 * it, in increasing flat pair index p = t*K + j.  counts [E], offsets [E+1], perm [T*K]
 * (perm[offsets[e] + i] = flat index of the i-th pair of expert e).
 */
int moe_oracle_gather(const int32_t *idx, int T, int K, int E,
                      int32_t *counts, int32_t *offsets, int32_t *perm)
{
    if (E <= 0 || E > MOE_ORACLE_MAX_E || T < 0 || K <= 0)
        return 1;
    for (int e = 0; e < E; ++e)
        counts[e] = 0;
    for (int p = 0; p < T * K; ++p) {
        if (idx[p] < 0 || idx[p] >= E)
            return 1;
        counts[idx[p]]++;
    }
    offsets[0] = 0;
    for (int e = 0; e < E; ++e)
        offsets[e + 1] = offsets[e] + counts[e];
    int32_t fill[MOE_ORACLE_MAX_E];
    for (int e = 0; e < E; ++e)
        fill[e] = 0;
    for (int p = 0; p < T * K; ++p) {
        int e = idx[p];
        perm[offsets[e] + fill[e]] = p;
        fill[e]++;
    }
    return 0;
}

/* ---------------------------------------------------------------- cache --------- */

/*
 * Expert cache of one layer (Section 2, "Expert Offloading Systems"; Section 3.2: experts
 * are fetched on demand, "evicting cached experts as dictated by the cache policy").
 *
 * The paper never states LRU operationally, so this is the reading used here:
 *  - a per-cache 64-bit counter; every request takes stamp = ++counter;
 *  - hit: the expert's slot is re-stamped;
 *  - miss: the victim is the lowest-index empty slot if there is one, else the slot with
 *    the smallest stamp (stamps are unique, so there are no ties); the expert is placed
 *    there and stamped; one miss = one host-to-device transfer (Appendix C.1);
 *  - one forward call issues one request per DISTINCT expert that its tokens selected:
 *    first the experts resident at call entry in ascending expert id, then the others in
 *    ascending expert id.  (Hits first lets their compute overlap the transfers, and never
 *    evicts a needed resident expert while another victim exists.)
 *
 * Second policy: the gamma-discounted count of Definition C.1 (gamma = 1 is LFU, the policy of
 * the paper's experiments; gamma -> 0+ is LRU, by the remark under the definition).  Reading:
 *  - one forward call is one time step: before its requests are served, every expert's count
 *    becomes gamma * count + r, r = 1 for the experts the call requests and 0 for the others
 *    (the count recurrence of Definition C.1), in fp32, product rounded before the sum;
 *  - requests, hits, stamps and empty slots exactly as above; only the victim differs: the
 *    occupied slot whose expert has the smallest count, the smaller stamp deciding ties (so
 *    the policy falls back to LRU order where counts are equal);
 *  - a preloaded expert's count is raised by one without a decay step (the definition leaves
 *    the initial count vector to the prefetch; C preloaded experts give it L1 norm C).
 * Definition C.1's cache is the Top-C of the counts; a demand-fetched cache can only change
 * where a miss occurs (the "lazy update" of the remark), which is what this does.
 */
typedef struct moe_oracle_cache {
    int C, E;
    uint64_t counter;
    int32_t *expert_of_slot; /* [C], -1 = empty */
    uint64_t *stamp;         /* [C] */
    int32_t *slot_of_expert; /* [E], -1 = not resident */
    uint64_t hits, misses, evictions;
    int policy;              /* 0 = LRU, 1 = gamma-discounted count */
    float gamma;
    float *count;            /* [E] */
} moe_oracle_cache;

typedef struct moe_oracle_request {
    int32_t expert, slot, hit, evicted; /* evicted = expert thrown out, or -1 */
} moe_oracle_request;

void moe_oracle_cache_reset(moe_oracle_cache *c)
{
    c->counter = 0;
    c->hits = c->misses = c->evictions = 0;
    for (int s = 0; s < c->C; ++s) {
        c->expert_of_slot[s] = -1;
        c->stamp[s] = 0;
    }
    for (int e = 0; e < c->E; ++e) {
        c->slot_of_expert[e] = -1;
        c->count[e] = 0.0f;
    }
}

/* policy 0 = LRU, 1 = gamma-discounted count (0 <= gamma <= 1).  Keeps the cache contents. */
int moe_oracle_cache_set_policy(moe_oracle_cache *c, int policy, float gamma)
{
    if (!c || (policy != 0 && policy != 1) || !(gamma >= 0.0f && gamma <= 1.0f))
        return -1;
    c->policy = policy;
    c->gamma = gamma;
    return 0;
}

moe_oracle_cache *moe_oracle_cache_create(int C, int E)
{
    if (C <= 0 || E <= 0)
        return NULL;
    moe_oracle_cache *c = (moe_oracle_cache *)calloc(1, sizeof *c);
    if (!c)
        return NULL;
    c->C = C;
    c->E = E;
    c->expert_of_slot = (int32_t *)malloc(sizeof(int32_t) * (size_t)C);
    c->stamp = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)C);
    c->slot_of_expert = (int32_t *)malloc(sizeof(int32_t) * (size_t)E);
    c->count = (float *)malloc(sizeof(float) * (size_t)E);
    c->policy = 0;
    c->gamma = 0.0f;
    moe_oracle_cache_reset(c);
    return c;
}

void moe_oracle_cache_destroy(moe_oracle_cache *c)
{
    if (!c)
        return;
    free(c->expert_of_slot);
    free(c->stamp);
    free(c->slot_of_expert);
    free(c->count);
    free(c);
}

static void cache_one_request(moe_oracle_cache *c, int e, moe_oracle_request *out)
{
    out->expert = e;
    out->evicted = -1;
    uint64_t st = ++c->counter;
    int s = c->slot_of_expert[e];
    if (s >= 0) {
        out->hit = 1;
        out->slot = s;
        c->stamp[s] = st;
        c->hits++;
        return;
    }
    out->hit = 0;
    c->misses++;
    int victim = -1;
    for (int i = 0; i < c->C; ++i)
        if (c->expert_of_slot[i] < 0) {
            victim = i;
            break;
        }
    if (victim < 0) {
        for (int i = 0; i < c->C; ++i) {
            if (victim < 0) {
                victim = i;
            } else if (c->policy == 1) {
                const float ci = c->count[c->expert_of_slot[i]], cv = c->count[c->expert_of_slot[victim]];
                if (ci < cv || (ci == cv && c->stamp[i] < c->stamp[victim]))
                    victim = i;
            } else if (c->stamp[i] < c->stamp[victim]) {
                victim = i;
            }
        }
        out->evicted = c->expert_of_slot[victim];
        c->slot_of_expert[out->evicted] = -1;
        c->evictions++;
    }
    c->expert_of_slot[victim] = e;
    c->slot_of_expert[e] = victim;
    c->stamp[victim] = st;
    out->slot = victim;
}

/*
 * One forward call's worth of requests.  idx holds n_idx expert ids (the call's T*K routing
 * indices, duplicates allowed).  Writes at most E records in request order and returns their
 * number, or -1 on a bad index.
 */
int moe_oracle_cache_call(moe_oracle_cache *c, const int32_t *idx, int n_idx,
                          moe_oracle_request *out)
{
    unsigned char *needed = (unsigned char *)calloc((size_t)c->E, 1);
    unsigned char *was_resident = (unsigned char *)calloc((size_t)c->E, 1);
    int n = 0;
    for (int i = 0; i < n_idx; ++i) {
        if (idx[i] < 0 || idx[i] >= c->E) {
            n = -1;
            goto done;
        }
        needed[idx[i]] = 1;
    }
    for (int e = 0; e < c->E; ++e)
        was_resident[e] = (unsigned char)(c->slot_of_expert[e] >= 0);
    if (c->policy == 1)
        for (int e = 0; e < c->E; ++e) {
            const float decayed = c->gamma * c->count[e];   /* rounded before the sum */
            c->count[e] = decayed + (needed[e] ? 1.0f : 0.0f);
        }
    for (int e = 0; e < c->E; ++e)
        if (needed[e] && was_resident[e])
            cache_one_request(c, e, &out[n++]);
    for (int e = 0; e < c->E; ++e)
        if (needed[e] && !was_resident[e])
            cache_one_request(c, e, &out[n++]);
done:
    free(needed);
    free(was_resident);
    return n;
}

/* Fill the cache ahead of the first token (Eq. 5's preloading step): one request per id, in
 * order, no decay step; under the count policy each id's count grows by one. */
int moe_oracle_cache_preload(moe_oracle_cache *c, const int32_t *ids, int n, moe_oracle_request *out)
{
    for (int i = 0; i < n; ++i) {
        if (ids[i] < 0 || ids[i] >= c->E)
            return -1;
        if (c->policy == 1)
            c->count[ids[i]] += 1.0f;
        cache_one_request(c, ids[i], &out[i]);
    }
    return n;
}

/*
 * Pooled prefetch set of a batch (Section 4.3 "Effect of Batch Size": the predictor pools the most
 * likely experts across the sequences of the batch; the paper gives no rule, the reading taken is
 * a vote).  lists[n_seq][per_seq]: every sequence's own predicted set.  vote(e) = number of
 * sequences whose list contains e.  The result is the C experts with the largest non-zero vote,
 * by decreasing vote, the lower id first among equal votes; returns how many were written to out,
 * or -1 on a bad id.  Written as a selection sort over the votes, nothing cleverer.
 */
int moe_oracle_pool_prefetch(const int32_t *lists, int n_seq, int per_seq, int E, int C, int32_t *out)
{
    int *vote = (int *)calloc((size_t)E, sizeof(int));
    unsigned char *in_list = (unsigned char *)calloc((size_t)E, 1);
    int n = 0;
    for (int q = 0; q < n_seq; ++q) {
        for (int e = 0; e < E; ++e)
            in_list[e] = 0;
        for (int j = 0; j < per_seq; ++j) {
            const int e = lists[(size_t)q * per_seq + j];
            if (e < 0 || e >= E) {
                n = -1;
                goto done;
            }
            in_list[e] = 1;
        }
        for (int e = 0; e < E; ++e)
            vote[e] += in_list[e];
    }
    while (n < C) {
        int best = -1;
        for (int e = 0; e < E; ++e)
            if (vote[e] > 0 && (best < 0 || vote[e] > vote[best]))
                best = e;                      /* strict >: the lowest id wins among equal votes */
        if (best < 0)
            break;
        out[n++] = best;
        vote[best] = 0;
    }
done:
    free(vote);
    free(in_list);
    return n;
}

void moe_oracle_cache_counts(const moe_oracle_cache *c, float *count)
{
    for (int e = 0; e < c->E; ++e)
        count[e] = c->count[e];
}

void moe_oracle_cache_state(const moe_oracle_cache *c, int32_t *expert_of_slot,
                            uint64_t *stamp, uint64_t *totals /* hits, misses, evictions */)
{
    for (int s = 0; s < c->C; ++s) {
        if (expert_of_slot)
            expert_of_slot[s] = c->expert_of_slot[s];
        if (stamp)
            stamp[s] = c->stamp[s];
    }
    if (totals) {
        totals[0] = c->hits;
        totals[1] = c->misses;
        totals[2] = c->evictions;
    }
}

/* ---------------------------------------------------------------- FFN + combine - */

static double silu(double a)
{
    return a / (1.0 + exp(-a));
}

/*
 * Eq. 3 for one token and one expert, fp64 throughout:
 *   g = W_g x, u = W_u x, h = SiLU(g) (.) u, z = W_d h.
 * W_g, W_u [F][d] and W_d [d][F] are bf16 bits in the paper's row-major shapes.
 * hbuf is scratch of F doubles.
 */
static void expert_ffn(const uint16_t *wg, const uint16_t *wu, const uint16_t *wd,
                       const uint16_t *x, int d, int F, double *hbuf, double *z)
{
#pragma omp parallel for schedule(static)
    for (int f = 0; f < F; ++f) {
        const uint16_t *rg = wg + (size_t)f * d;
        const uint16_t *ru = wu + (size_t)f * d;
        double g = 0.0, u = 0.0;
        for (int j = 0; j < d; ++j) {
            double xj = (double)bf16_to_f32(x[j]);
            g += (double)bf16_to_f32(rg[j]) * xj;
            u += (double)bf16_to_f32(ru[j]) * xj;
        }
        hbuf[f] = silu(g) * u;
    }
#pragma omp parallel for schedule(static)
    for (int r = 0; r < d; ++r) {
        const uint16_t *rd = wd + (size_t)r * F;
        double acc = 0.0;
        for (int f = 0; f < F; ++f)
            acc += (double)bf16_to_f32(rd[f]) * hbuf[f];
        z[r] = acc;
    }
}

/*
 * Eq. 2 for a list of tokens: y_t = sum_j gate[t][j] * E_{idx[t][j]}(x_t), plus every shared
 * expert with gate 1 (shared experts are not in the paper; they are always resident, apply
 * to every token and never touch the cache).
 *
 * wg/wu/wd: arrays of E (+ n_shared after them) pointers to the expert matrices; a NULL
 * entry for an expert that some listed token needs is an error (return 2).
 * tokens [n_sel]: which rows of x / idx / gate to evaluate (NULL: rows 0..n_sel-1).
 * y [n_sel][d] fp64 out.  Independent of any cache state by construction.
 */
int moe_oracle_ffn_combine(const uint16_t *x, const int32_t *idx, const double *gate,
                           const uint16_t *const *wg, const uint16_t *const *wu,
                           const uint16_t *const *wd, int d, int F, int E, int K,
                           int n_shared, const int32_t *tokens, int n_sel, double *y)
{
    double *hbuf = (double *)malloc(sizeof(double) * (size_t)F);
    double *z = (double *)malloc(sizeof(double) * (size_t)d);
    if (!hbuf || !z) {
        free(hbuf);
        free(z);
        return 3;
    }
    int rc = 0;
    for (int i = 0; i < n_sel && rc == 0; ++i) {
        int t = tokens ? tokens[i] : i;
        double *yt = y + (size_t)i * d;
        for (int r = 0; r < d; ++r)
            yt[r] = 0.0;
        for (int j = 0; j < K + n_shared; ++j) {
            int e = j < K ? idx[(size_t)t * K + j] : E + (j - K);
            double w = j < K ? gate[(size_t)t * K + j] : 1.0;
            if (e < 0 || e >= E + n_shared || !wg[e] || !wu[e] || !wd[e]) {
                rc = 2;
                break;
            }
            expert_ffn(wg[e], wu[e], wd[e], x + (size_t)t * d, d, F, hbuf, z);
            for (int r = 0; r < d; ++r)
                yt[r] += w * z[r];
        }
    }
    free(hbuf);
    free(z);
    return rc;
}
