"""Pins for the CPU oracle: everything here runs without a GPU.

Each test checks the oracle against something other than itself: a value the paper prints,
a closed form, a textbook property, brute force on tiny inputs, or a library routine on a
special case.
"""
import json
import os

import numpy as np
import pytest

import gen
import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


def _bf16(a):
    return gen.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


# ------------------------------------------------------------------ generator sanity


def test_bf16_round_trip_and_rne():
    # exactly representable values survive; ties go to even mantissa
    v = np.array([1.0, -2.5, 0.02, 4096.0, 3.0e-5], dtype=np.float32)
    b = gen.f32_to_bf16_bits(v)
    back = gen.bf16_bits_to_f32(b)
    assert np.all(np.abs(back - v) <= np.abs(v) * 2.0 ** -8)
    one_plus_half_ulp = np.array([1.0 + 2.0 ** -8], dtype=np.float32)       # tie -> even (1.0)
    one_plus_3half_ulp = np.array([1.0 + 3 * 2.0 ** -8], dtype=np.float32)  # tie -> even (1 + 2^-6)
    assert gen.bf16_bits_to_f32(gen.f32_to_bf16_bits(one_plus_half_ulp))[0] == 1.0
    assert gen.bf16_bits_to_f32(gen.f32_to_bf16_bits(one_plus_3half_ulp))[0] == np.float32(1.0 + 2.0 ** -6)


def test_generators_are_order_independent():
    a = gen.hidden_states(7, 3, "decode", 5, 4, 256)
    _ = gen.hidden_states(7, 2, "decode", 5, 4, 256)
    b = gen.hidden_states(7, 3, "decode", 5, 4, 256)
    assert np.array_equal(a, b)
    assert not np.array_equal(a, gen.hidden_states(7, 3, "decode", 6, 4, 256))


def test_uniform_routing_share_matches_paper_figure():
    g = _gold("uniform_share.json")
    # alpha -> infinity gives an exactly flat preference: any `top` experts carry top/E
    E, top = g["n_experts"], g["top"]
    pi = np.full(E, 1.0 / E)
    assert abs(np.sort(pi)[::-1][:top].sum() - g["share"]) < 1e-12
    # a large-alpha draw is close to it, a small-alpha draw far above it
    flat = np.exp(gen.router_bias(1, 0, 0, 1000.0, E).astype(np.float64))
    peaked = np.exp(gen.router_bias(1, 0, 0, 0.1, E).astype(np.float64))
    assert abs(flat.sum() - 1) < 1e-4 and abs(np.sort(flat)[::-1][:top].sum() - g["share"]) < 0.02
    assert np.sort(peaked)[::-1][:top].sum() > 0.6


# ------------------------------------------------------------------ a1: router (Eq. 1)


def test_logit_summation_order_hand_worked():
    g = _gold("logit_order.json")
    d = g["d"]
    x = np.zeros((1, d), np.float32)
    w = np.zeros((1, d), np.float32)
    for j, v in g["x_nonzero"].items():
        x[0, int(j)] = v
    for j, v in g["w_nonzero"].items():
        w[0, int(j)] = v
    lg = oracle.logits(_bf16(x), _bf16(w))
    assert lg.shape == (1, 1) and lg[0, 0] == np.float32(g["expected_logit"])
    # the plain left-to-right fp32 sum of the same products gives the other printed value
    acc = np.float32(0)
    for j in range(d):
        acc = np.float32(acc + np.float32(x[0, j] * w[0, j]))
    assert acc == np.float32(g["left_to_right_would_give"])


def test_logits_close_to_exact_dot_product():
    rs = np.random.default_rng(0)
    x = _bf16(rs.standard_normal((5, 512)))
    w = _bf16(rs.standard_normal((7, 512)) * 0.02)
    bias = rs.standard_normal((2, 7)).astype(np.float32)
    seq = np.array([0, 1, 1, 0, 1], np.int32)
    lg = oracle.logits(x, w, bias, seq)
    exact = gen.bf16_bits_to_f32(x).astype(np.float64) @ gen.bf16_bits_to_f32(w).astype(np.float64).T
    exact += bias.astype(np.float64)[seq]
    # fp32 summation of 512 exact products: error far below 1e-4 relative to the operand scale
    assert np.max(np.abs(lg - exact)) < 5e-6
    # without token_seq every token uses bias row 0
    lg0 = oracle.logits(x, w, bias, None)
    exact0 = exact - bias.astype(np.float64)[seq] + bias.astype(np.float64)[0]
    assert np.max(np.abs(lg0 - exact0)) < 5e-6


def test_logits_reject_bad_d():
    with pytest.raises(ValueError):
        oracle.logits(np.zeros((1, 128), np.uint16), np.zeros((2, 128), np.uint16))


def test_topk_against_stable_sort_brute_force():
    rs = np.random.default_rng(1)
    for E, k in ((8, 2), (64, 8), (16, 16), (5, 1)):
        lg = rs.standard_normal((50, E)).astype(np.float32)
        lg[3, :] = 0.25                      # all equal
        lg[4, : E // 2] = 1.0                # a tie block at the top
        lg[5] = np.round(lg[5] * 2) / 2      # many ties
        idx, gate = oracle.topk(lg, k)
        for t in range(lg.shape[0]):
            order = np.argsort(-lg[t].astype(np.float64), kind="stable")[:k]
            assert np.array_equal(idx[t], order)
            e = np.exp(lg[t, order].astype(np.float64) - lg[t, order[0]])
            assert np.allclose(gate[t], e / e.sum(), rtol=1e-12)
        assert np.allclose(gate.sum(axis=1), 1.0, atol=1e-12)
        for t in range(lg.shape[0]):
            assert len(set(idx[t].tolist())) == k and idx[t].min() >= 0 and idx[t].max() < E
            assert np.all(np.diff(lg[t, idx[t]]) <= 0)
    # all-equal logits: indices 0..k-1 and gates 1/k
    idx, gate = oracle.topk(np.zeros((1, 8), np.float32), 3)
    assert idx.tolist() == [[0, 1, 2]] and np.allclose(gate, 1 / 3)


def test_topk_raw_softmax_matches_eq2_weights():
    rs = np.random.default_rng(2)
    lg = rs.standard_normal((4, 8)).astype(np.float32)
    idx, gate = oracle.topk(lg, 2, raw_softmax=True)
    p = np.exp(lg.astype(np.float64))
    p /= p.sum(axis=1, keepdims=True)
    assert np.allclose(gate, np.take_along_axis(p, idx, axis=1), rtol=1e-12)
    assert np.all(gate.sum(axis=1) < 1.0)


def test_zero_router_selects_topk_of_bias():
    E, k, d = 16, 4, 256
    rs = np.random.default_rng(3)
    x = _bf16(rs.standard_normal((3, d)))
    bias = rs.permutation(E).astype(np.float32)[None, :]
    idx, gate, lg = oracle.route(x, np.zeros((E, d), np.uint16), k, bias)
    want = np.argsort(-bias[0], kind="stable")[:k]
    assert np.all(idx == want[None, :])
    assert np.array_equal(lg, np.repeat(bias, 3, axis=0))


# ------------------------------------------------------------------ a4: gather


def test_gather_is_stable_counting_sort():
    rs = np.random.default_rng(4)
    T, k, E = 37, 3, 10
    idx = np.stack([rs.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    counts, offsets, perm = oracle.gather(idx, E)
    flat = idx.reshape(-1)
    assert np.array_equal(counts, np.bincount(flat, minlength=E))
    assert np.array_equal(offsets, np.concatenate([[0], np.cumsum(counts)]))
    assert np.array_equal(perm, np.argsort(flat, kind="stable"))
    # an expert nobody selected has an empty list
    idx2 = np.zeros((4, 1), np.int32)
    c2, o2, p2 = oracle.gather(idx2, 3)
    assert c2.tolist() == [4, 0, 0] and o2.tolist() == [0, 4, 4, 4] and p2.tolist() == [0, 1, 2, 3]


# ------------------------------------------------------------------ a2/a3: cache trace


def _lru_closed_form(call_sets, C):
    """Textbook LRU from the raw history: after any request sequence the resident set is the
    last min(C, #distinct) distinct experts requested; a request hits iff fewer than C other
    distinct experts were requested since its previous request (stack distance < C)."""
    history = []      # flat request sequence in the stated order
    hits = []
    for s in call_sets:
        # resident set at call entry, recomputed from history alone
        seen, resident = [], []
        for e in reversed(history):
            if e not in seen:
                seen.append(e)
        resident = seen[:C]
        first = sorted(e for e in s if e in resident)
        rest = sorted(e for e in s if e not in resident)
        for e in first + rest:
            if e in history:
                last = len(history) - 1 - history[::-1].index(e)
                between = len(set(history[last + 1:]) - {e})
                hits.append((e, between < C))
            else:
                hits.append((e, False))
            history.append(e)
    seen = []
    for e in reversed(history):
        if e not in seen:
            seen.append(e)
    return hits, set(seen[:C])


def test_lru_hand_worked_trace():
    g = _gold("lru_trace.json")
    c = oracle.ExpertCache(g["cache_slots"], g["n_experts"])
    for call, want in zip(g["calls"], g["requests"]):
        got = c.call(np.array(call, np.int32))
        assert got.tolist() == want


@pytest.mark.parametrize("C,E,k,T", [(4, 8, 2, 1), (3, 6, 1, 1), (16, 64, 8, 1), (6, 16, 2, 8), (2, 8, 2, 1)])
def test_lru_matches_stack_distance_closed_form(C, E, k, T):
    rs = np.random.default_rng(C * 100 + E)
    cache = oracle.ExpertCache(C, E)
    call_sets, got = [], []
    pref = rs.dirichlet(np.full(E, 0.5))
    for _ in range(120):
        idx = np.stack([rs.choice(E, size=k, replace=False, p=pref) for _ in range(T)]).astype(np.int32)
        req = cache.call(idx)
        # duplicates inside a call collapse to one request per distinct expert
        assert sorted(req[:, 0].tolist()) == sorted(set(idx.reshape(-1).tolist()))
        call_sets.append(set(idx.reshape(-1).tolist()))
        got += [(int(r[0]), bool(r[2])) for r in req]
    want, resident = _lru_closed_form(call_sets, C)
    assert got == want
    eos, stamps, tot = cache.state()
    assert set(int(e) for e in eos if e >= 0) == resident
    assert tot["hits"] == sum(h for _, h in want) and tot["misses"] == sum(not h for _, h in want)
    live = stamps[eos >= 0]
    assert len(set(live.tolist())) == live.size          # stamps unique


def test_lru_slot_bookkeeping_is_consistent():
    rs = np.random.default_rng(11)
    C, E = 5, 12
    cache = oracle.ExpertCache(C, E)
    slot_now = {}
    for _ in range(200):
        idx = rs.choice(E, size=3, replace=False).astype(np.int32)[None, :]
        for e, s, hit, ev in cache.call(idx).tolist():
            if hit:
                assert slot_now[e] == s and ev == -1
            else:
                assert e not in slot_now
                if ev >= 0:
                    assert slot_now.pop(ev) == s
                else:
                    # an empty slot is taken lowest index first
                    assert s == min(set(range(C)) - set(slot_now.values()))
                slot_now[e] = s
        eos, _, _ = cache.state()
        assert {int(e): i for i, e in enumerate(eos) if e >= 0} == slot_now


def test_lru_inclusion_property():
    rs = np.random.default_rng(5)
    E = 16
    calls = [rs.choice(E, size=1).astype(np.int32)[None, :] for _ in range(400)]
    prev_res, prev_miss = None, None
    for C in range(1, E + 1):
        cache = oracle.ExpertCache(C, E)
        for idx in calls:
            cache.call(idx)
        eos, _, tot = cache.state()
        res = set(int(e) for e in eos if e >= 0)
        if prev_res is not None:
            assert prev_res <= res and tot["misses"] <= prev_miss
        prev_res, prev_miss = res, tot["misses"]


def test_full_cache_only_compulsory_misses():
    rs = np.random.default_rng(6)
    E, k = 8, 2
    cache = oracle.ExpertCache(E, E)
    seen = set()
    for _ in range(100):
        idx = rs.choice(E, size=k, replace=False).astype(np.int32)[None, :]
        for e, s, hit, ev in cache.call(idx).tolist():
            assert ev == -1 and bool(hit) == (e in seen)
            seen.add(e)
    _, _, tot = cache.state()
    assert tot["misses"] == len(seen) and tot["evictions"] == 0


def test_cyclic_scan_thrashes_lru():
    C = 4
    for n, all_miss in ((C + 1, True), (C, False)):
        cache = oracle.ExpertCache(C, 8)
        recs = [cache.call(np.array([[i % n]], np.int32))[0] for i in range(40)]
        hits = [int(r[2]) for r in recs]
        if all_miss:
            assert sum(hits) == 0
        else:
            assert hits == [0] * n + [1] * (40 - n)


def test_lru_equals_discounted_topc_cache_for_small_gamma():
    """Definition C.1 with gamma < 1/2, zero-initialised counts and K = 1: Top-C of the
    discounted counts is the C most recently requested experts (gamma -> 0+ gives LRU)."""
    rs = np.random.default_rng(7)
    E, C, gamma = 10, 4, 0.25
    cache = oracle.ExpertCache(C, E)
    count = np.zeros(E)
    for t in range(300):
        e = int(rs.integers(E))
        # hard cache state before the request, from the counts alone
        nz = [i for i in np.argsort(-count, kind="stable") if count[i] > 0][:C]
        rec = cache.call(np.array([[e]], np.int32))[0]
        assert bool(rec[2]) == (e in nz)          # miss  <=>  <r, 1 - c_hat> = 1
        r = np.zeros(E)
        r[e] = 1.0
        count = gamma * count + r
        eos, _, _ = cache.state()
        nz_after = set(int(i) for i in np.argsort(-count, kind="stable") if count[i] > 0)
        top = set(list(int(i) for i in np.argsort(-count, kind="stable") if count[i] > 0)[:C])
        assert set(int(x) for x in eos if x >= 0) == top and top <= nz_after


def test_count_policy_hand_worked_traces():
    """Definition C.1's discounted count as the eviction key: traces worked by hand."""
    for g in _gold("count_policy_trace.json")["cases"]:
        c = oracle.ExpertCache(g["cache_slots"], g["n_experts"], "count", g["gamma"])
        for call, want in zip(g["calls"], g["requests"]):
            assert c.call(np.array(call, np.int32)).tolist() == want, g["comment"]


@pytest.mark.parametrize("C,E,k,T", [(4, 8, 2, 1), (16, 64, 8, 1), (6, 16, 2, 8), (2, 8, 2, 1)])
def test_count_policy_with_vanishing_gamma_is_lru(C, E, k, T):
    """Remark under Definition C.1: gamma -> 0+ gives LRU updates.  With a gamma so small that a
    count is 1 for the experts of the latest call and (in fp32) below that for all others, older
    ones tying at zero, the trace must be the LRU trace, request for request."""
    rs = np.random.default_rng(C + 7 * E)
    lru = oracle.ExpertCache(C, E)
    cnt = oracle.ExpertCache(C, E, "count", 1e-30)
    pref = rs.dirichlet(np.full(E, 0.5))
    for _ in range(150):
        idx = np.stack([rs.choice(E, size=k, replace=False, p=pref) for _ in range(T)]).astype(np.int32)
        assert cnt.call(idx).tolist() == lru.call(idx).tolist()


@pytest.mark.parametrize("gamma", [1.0, 0.9, 0.5])
def test_count_policy_evicts_a_minimal_discounted_count(gamma):
    """Every victim has the smallest discounted count among the experts resident at that moment,
    the counts taken from the closed form sum_s gamma^(t - s) r_e(s) over the request history
    (fp64, no recurrence), the resident set tracked from the request records alone."""
    rs = np.random.default_rng(int(gamma * 100))
    C, E, k = 5, 14, 2
    cache = oracle.ExpertCache(C, E, "count", gamma)
    history = []                      # request vectors r(s), one per call
    slot_expert = {}
    pref = rs.dirichlet(np.full(E, 0.7))
    n_evictions = 0
    for t in range(250):
        idx = rs.choice(E, size=k, replace=False, p=pref).astype(np.int32)
        r = np.zeros(E)
        r[idx] = 1.0
        history.append(r)
        w = gamma ** np.arange(len(history) - 1, -1, -1, dtype=np.float64)
        count = (w[:, None] * np.array(history)).sum(axis=0)
        for e, slot, hit, ev in cache.call(idx[None, :]).tolist():
            if hit:
                assert slot_expert[slot] == e
                continue
            if ev >= 0:
                n_evictions += 1
                assert slot_expert[slot] == ev
                others = [x for s_, x in slot_expert.items() if s_ != slot]
                assert count[ev] <= min(count[x] for x in others) * (1 + 1e-5) + 1e-12
            else:
                assert slot not in slot_expert
            slot_expert[slot] = e
        assert np.allclose(cache.counts(), count, rtol=1e-4, atol=1e-30)
    assert n_evictions > 50


def test_count_policy_preload_gives_the_definitions_initial_counts():
    """Definition C.1 starts from a count vector of L1 norm C set by the prefetch: C preloaded experts
    carry count 1 each, sit in the cache, and hit on the first call."""
    C, E = 4, 12
    cache = oracle.ExpertCache(C, E, "count", 0.9)
    rec = cache.preload([7, 2, 9, 4])
    assert rec[:, 2].tolist() == [0, 0, 0, 0] and rec[:, 1].tolist() == [0, 1, 2, 3]
    cnt = cache.counts()
    assert cnt.sum() == C and set(np.nonzero(cnt)[0].tolist()) == {2, 4, 7, 9}
    first = cache.call(np.array([[2, 9]], np.int32))
    assert first[:, 2].tolist() == [1, 1]
    assert np.allclose(cache.counts()[[2, 9, 4, 7]], [1.9, 1.9, 0.9, 0.9])


def test_q4_hand_worked_groups():
    for g in _gold("q4_groups.json")["groups"]:
        row = np.zeros(64, np.float32)
        row[:len(g["head"])] = g["head"]
        codes, scales = oracle.quantize_q4(_bf16(row)[None, :])
        assert gen.bf16_bits_to_f32(scales)[0, 0] == g["scale"], g["comment"]
        nib = np.stack([codes[0] & 15, codes[0] >> 4], axis=1).reshape(-1)
        n = len(g["head"])
        assert nib[:n].tolist() == g["codes_head"] and np.all(nib[n:] == 8), g["comment"]
        deq = gen.bf16_bits_to_f32(oracle.dequantize_q4(codes, scales))[0]
        assert deq[:n].tolist() == g["dequant_head"] and np.all(deq[n:] == 0.0), g["comment"]


def test_q4_error_bound_range_and_grid_points():
    rs = np.random.default_rng(5)
    w = _bf16(rs.normal(0.0, 0.02, (24, 256)).astype(np.float32))
    codes, scales = oracle.quantize_q4(w)
    wf = gen.bf16_bits_to_f32(w).astype(np.float64)
    sf = np.repeat(gen.bf16_bits_to_f32(scales).astype(np.float64), 64, axis=1)
    deq = gen.bf16_bits_to_f32(oracle.dequantize_q4(codes, scales)).astype(np.float64)
    nib = np.stack([codes & 15, codes >> 4], axis=2).reshape(24, 256).astype(np.int64) - 8
    assert nib.min() >= -8 and nib.max() <= 7
    # rounding to the nearest code: half a step, plus half an ulp of bf16 on the product, plus the
    # clamp at +-7 where the rounded-down scale makes max|w| / scale a little more than 7
    step_err = np.abs(wf - sf * nib)
    assert np.all(step_err <= sf * (0.5 + 7 * 2.0 ** -8) + 1e-12)
    assert np.all(np.abs(deq - sf * nib) <= np.abs(sf * nib) * 2.0 ** -8 + 1e-30)
    # the largest element of every group sits on the outermost code
    wg, ng = np.abs(wf).reshape(24, 4, 64), np.abs(nib).reshape(24, 4, 64)
    assert np.all(np.take_along_axis(ng, wg.argmax(axis=2)[..., None], axis=2) >= 7)
    # weights that are already scale * integer with a power-of-two scale come back exactly
    grid = (rs.integers(-7, 8, (6, 128)) * 2.0 ** -6).astype(np.float32)
    grid[:, 0] = 7 * 2.0 ** -6
    grid[:, 64] = -7 * 2.0 ** -6
    c2, s2 = oracle.quantize_q4(_bf16(grid))
    assert np.array_equal(gen.bf16_bits_to_f32(oracle.dequantize_q4(c2, s2)), grid)
    # an all-zero group: scale 0, code 8, weight 0
    c3, s3 = oracle.quantize_q4(np.zeros((2, 64), np.uint16))
    assert np.all(s3 == 0) and np.all(c3 == 0x88) and np.all(oracle.dequantize_q4(c3, s3) == 0)
    with pytest.raises(ValueError):
        oracle.quantize_q4(np.zeros((2, 96), np.uint16))


def test_miss_proxies_closed_forms():
    """Section 3.1's soft cache and Definition C.1's hard cache on traces whose answer is known."""
    E, C, K = 12, 4, 2
    # the same K experts every token: once the soft cache is full its whole mass C sits on them, so the
    # proxy is K (1 - C / K) = K - C; the hard cache misses them once
    same = np.tile(np.array([[3, 7]]), (60, 1))
    soft, hard = oracle.miss_proxies(same, E, C, 0.9)
    assert soft[0] == K and np.allclose(soft[-10:], K - C)
    assert hard.tolist() == [2] + [0] * 59
    # gamma = 0 with K < C: the state is the previous request (its norm K never reaches C, so it is never
    # rescaled), soft and hard proxy are both K - |overlap with the previous token|
    rs = np.random.default_rng(9)
    tr = np.stack([rs.choice(E, size=K, replace=False) for _ in range(80)])
    soft0, hard0 = oracle.miss_proxies(tr, E, C, 0.0)
    for t in range(1, 80):
        overlap = len(set(tr[t].tolist()) & set(tr[t - 1].tolist()))
        assert soft0[t] == K - overlap and hard0[t] == K - overlap
    # gamma = 1: the fill ends after C / K tokens with c0 = the sum of their requests (norm exactly C);
    # from then on Z_n c_n = c0 + the requests since, Z_n = 1 + n K / C
    soft1, _ = oracle.miss_proxies(tr, E, C, 1.0)
    n0 = C // K
    acc = np.zeros(E)
    for t in range(80):
        r = np.zeros(E)
        r[tr[t]] = 1.0
        if t >= n0:
            c_t = acc / (1.0 + (t - n0) * K / C)
            assert abs(soft1[t] - float((r * (1.0 - c_t)).sum())) < 1e-12
        acc += r
    # the norm of the soft state stays at C after the fill: sum_i (1 - c_i) r_i <= K and the mean proxy
    # over a uniform trace is K (1 - C / E) up to sampling noise
    big = np.stack([rs.choice(E, size=K, replace=False) for _ in range(4000)])
    soft_u, _ = oracle.miss_proxies(big, E, C, 0.9)
    assert abs(soft_u[100:].mean() - K * (1 - C / E)) < 0.03


@pytest.mark.parametrize("C,E", [(4, 10), (6, 16)])
def test_hard_miss_proxy_is_the_lru_miss_count_for_small_gamma(C, E):
    """K = 1 and gamma < 1/2: Top-C of the discounted counts is the C most recent experts, so the
    hard proxy equals the misses of the LRU cache oracle on the same trace."""
    rs = np.random.default_rng(C)
    tr = rs.integers(0, E, size=(400, 1))
    _, hard = oracle.miss_proxies(tr, E, C, 0.25)
    cache = oracle.ExpertCache(C, E)
    lru = [int(1 - cache.call(tr[t:t + 1])[0, 2]) for t in range(400)]
    assert hard.tolist() == lru


def test_miss_bytes_match_papers_transfer_example():
    g = _gold("transfer_time.json")
    cfg = gen.config_by_name("mixtral")
    assert (cfg.d_model, cfg.d_ff) == (g["d_model"], g["d_ff"])
    assert cfg.expert_bytes == 3 * g["d_model"] * g["d_ff"] * g["bytes_per_value"] == g["expert_bytes"]
    cache = oracle.ExpertCache(2, 8)
    for e in (0, 1, 2, 0):
        cache.call(np.array([[e]], np.int32))
    _, _, tot = cache.state()
    assert tot["misses"] == 4                      # 0,1,2 compulsory; 0 was evicted by 2
    ms = cfg.expert_bytes / (g["link_GBps"] * 1e9) * 1e3
    assert g["printed_ms_low"] <= ms <= g["printed_ms_high"]


# ------------------------------------------------------------------ a5/a6: FFN + combine (Eq. 2-3)


def _experts(seed, E, d, F):
    return [gen.expert_weights(seed, 0, e, d, F) for e in range(E)]


def test_single_expert_layer_is_a_plain_swiglu_mlp():
    torch = pytest.importorskip("torch")
    d, F, T = 256, 96, 3
    ex = _experts(21, 1, d, F)
    x = gen.hidden_states(21, 0, "decode", 0, T, d)
    w_r = gen.router_weights(21, 0, 1, d)
    out = oracle.layer_forward(x, w_r, ex, 1, F)
    assert np.all(out["idx"] == 0) and np.allclose(out["gate"], 1.0)
    tx = torch.from_numpy(gen.bf16_bits_to_f32(x)).double()
    wg, wu, wd = (torch.from_numpy(gen.bf16_bits_to_f32(m)).double() for m in ex[0])
    ref = (torch.nn.functional.silu(tx @ wg.T) * (tx @ wu.T)) @ wd.T
    assert np.allclose(out["y"], ref.numpy(), rtol=1e-10, atol=1e-14)


def test_layer_equals_dense_sum_over_selected_experts():
    d, F, E, k, T = 256, 64, 6, 3, 4
    ex = _experts(22, E, d, F)
    x = gen.hidden_states(22, 0, "decode", 0, T, d)
    w_r = gen.router_weights(22, 0, E, d)
    bias = np.stack([gen.router_bias(22, 0, s, 0.5, E) for s in range(2)])
    seq = np.array([0, 1, 0, 1], np.int32)
    out = oracle.layer_forward(x, w_r, ex, k, F, bias=bias, token_seq=seq)
    xf = gen.bf16_bits_to_f32(x).astype(np.float64)
    for t in range(T):
        y = np.zeros(d)
        for j in range(k):
            e = int(out["idx"][t, j])
            wg, wu, wd = (gen.bf16_bits_to_f32(m).astype(np.float64) for m in ex[e])
            g, u = wg @ xf[t], wu @ xf[t]
            y += out["gate"][t, j] * (wd @ (g / (1.0 + np.exp(-g)) * u))
        assert np.allclose(out["y"][t], y, rtol=1e-10, atol=1e-14)
    # token subset evaluation returns the same rows
    sub = oracle.ffn_combine(x, out["idx"], out["gate"], ex, F, tokens=[3, 1])
    assert np.array_equal(sub, out["y"][[3, 1]])


def test_shared_experts_add_with_unit_gate():
    d, F, E, k, T = 256, 32, 4, 2, 2
    ex = _experts(23, E + 2, d, F)
    x = gen.hidden_states(23, 0, "decode", 0, T, d)
    w_r = gen.router_weights(23, 0, E, d)
    idx, gate, _ = oracle.route(x, w_r, k)
    routed = oracle.ffn_combine(x, idx, gate, ex[:E], F)
    both = oracle.ffn_combine(x, idx, gate, ex, F, n_shared=2)
    ones = np.ones((T, 1))
    s0 = oracle.ffn_combine(x, np.zeros((T, 1), np.int32), ones, [ex[E]], F)
    s1 = oracle.ffn_combine(x, np.zeros((T, 1), np.int32), ones, [ex[E + 1]], F)
    assert np.allclose(both, routed + s0 + s1, rtol=1e-12, atol=1e-15)


def test_output_independent_of_cache_size_and_history():
    d, F, E, k = 256, 32, 8, 2
    ex = _experts(24, E, d, F)
    w_r = gen.router_weights(24, 0, E, d)
    xs = [gen.hidden_states(24, 0, "decode", s, 1, d) for s in range(6)]
    ys = {}
    for C in (2, 4, 8):
        cache = oracle.ExpertCache(C, E)
        ys[C] = [oracle.layer_forward(x, w_r, ex, k, F, cache=cache) for x in xs]
    for s in range(6):
        for C in (4, 8):
            assert np.array_equal(ys[C][s]["y"], ys[2][s]["y"])
            assert np.array_equal(ys[C][s]["idx"], ys[2][s]["idx"])
    assert ys[8][-1]["requests"] is not None


def test_missing_expert_is_reported():
    d, F = 256, 16
    ex = _experts(25, 2, d, F)
    x = gen.hidden_states(25, 0, "decode", 0, 1, d)
    with pytest.raises(ValueError):
        oracle.ffn_combine(x, np.array([[1]], np.int32), np.ones((1, 1)), [ex[0], None], F)


def test_pooled_prefetch_set_hand_worked_and_against_a_sort():
    """Pooled prefetch of a batch: the hand-worked sets, then random batches against a plain sort of
    (-votes, id) computed with collections.Counter; every chosen expert is named by some sequence."""
    import collections
    import json
    g = json.load(open(os.path.join(GOLD, "pooled_prefetch.json")))
    for c in g["cases"]:
        got = oracle.pool_prefetch(np.array(c["lists"], np.int32), g["n_experts"], c["cache_slots"])
        assert got.tolist() == c["expect"]
    rs = np.random.default_rng(5)
    for _ in range(50):
        E, n_seq, m, C = int(rs.integers(4, 40)), int(rs.integers(1, 9)), int(rs.integers(1, 9)), int(rs.integers(1, 12))
        lists = rs.integers(0, E, size=(n_seq, m)).astype(np.int32)
        votes = collections.Counter(e for row in lists for e in set(row.tolist()))
        want = [e for e, _ in sorted(votes.items(), key=lambda kv: (-kv[1], kv[0]))][:C]
        assert oracle.pool_prefetch(lists, E, C).tolist() == want
    with pytest.raises(ValueError):
        oracle.pool_prefetch(np.array([[0, 11]], np.int32), 10, 4)
