"""GPU-vs-oracle parity through the C ABI (run with -m gpu on a B200)."""
import os

import numpy as np
import pytest

import gen
import oracle

pytestmark = pytest.mark.gpu


def _pair(*a, **kw):
    from parity_util import Pair
    return Pair(*a, **kw)


def _bias(seed, E, alpha, n_seq):
    return np.stack([gen.router_bias(seed, 0, s, alpha, E) for s in range(n_seq)])


def test_tiny_config_32_decode_tokens_cold_start():
    """Config 1: d=256, F=512, 8 experts, top-2, 4 slots, 32 single-token calls."""
    c = gen.config_by_name("tiny")
    P = _pair(c.d_model, c.d_ff, c.n_experts, c.top_k, c.cache_slots[0], seed=c.seed)
    P.set_bias(_bias(c.seed, c.n_experts, c.alphas[0], 1), None)
    misses = 0
    for step in range(c.decode_steps):
        x = gen.hidden_states(c.seed, 0, "decode", step, 1, c.d_model)
        _, o = P.step(x)
        misses += o["stats"]["misses"]
    assert misses >= 2          # cold start: the first call misses both experts
    P.close()


@pytest.mark.parametrize("d,F,E,k,C", [
    (512, 200, 16, 4, 5),       # ragged d_ff (25 units), waves when T*k > C
    (1024, 64, 8, 2, 2),        # cache as small as top-k
    (2048, 96, 12, 3, 12),      # everything resident after warm-up
    (3072, 40, 6, 2, 3),
    (4096, 72, 5, 2, 4),        # widest rows (two ring entries per 8 rows)
])
def test_shapes_and_token_counts(d, F, E, k, C):
    P = _pair(d, F, E, k, C, seed=100 + d // 256)
    n_seq = 3
    P.set_bias(_bias(7, E, 0.5, n_seq), None)
    step = 0
    for T in (1, 3, 8, 1, 19, 70, 2, 1):
        seq = (np.arange(T) * n_seq // max(T, 1)).astype(np.int32)
        P.set_bias(P.bias, seq)
        x = gen.hidden_states(100 + d, 0, "decode", step, T, d)
        P.step(x)
        step += 1
    eos, tot = P.gpu.layer.cache_state()
    assert tot["hits"] + tot["misses"] > 0
    P.close()


def test_wide_model_with_many_tokens_keeps_its_token_operands_in_tensor_memory():
    """d_model 4096 with 5 to 8 tokens per call: the decode kernel writes the hidden states' tensor-core
    operands into tensor memory once and reads them from there (the shared memory goes to taller weight
    tiles).  Calls whose missed experts the kernel fetches itself (token-expert pairs <= slots), with a
    shared expert, between calls of fewer tokens that take the shared-memory form; then the same bits
    again from a warm cache (the sum over the SMs is exact, so residency must not change the output)."""
    d, F, E, k, C = 4096, 48, 20, 2, 16
    P = _pair(d, F, E, k, C, seed=77, n_shared=1)
    P.set_bias(_bias(9, E, 0.5, 4), None)
    outs = {}
    for rnd in range(2):
        for step, T in enumerate((8, 5, 2, 7, 6, 1, 8)):
            P.set_bias(P.bias, (np.arange(T) % 4).astype(np.int32))
            res, o = P.step(gen.hidden_states(77, 0, "decode", step, T, d))
            if rnd == 0:
                outs[step] = res["out_bits"].copy()
            else:
                assert np.array_equal(outs[step], res["out_bits"]), "output bits depend on the cache state"
    assert not P.gpu.layer.last_call_used_gemm()
    P.close()


def test_largest_supported_sizes_and_empty_call():
    """d_model, n_experts and top_k at their limits; T * k = 64 is the largest call the fused
    decode planner takes, T = 3 already goes through the general kernels; T = 0 is a no-op."""
    from paper_2602_11192_b200 import MelinoeError, MoELayer
    with pytest.raises(MelinoeError) as ei:
        MoELayer(8192, 64, 8, 2, 2)                 # wider than the decode kernel's accumulators cover
    assert ei.value.status == 6
    import torch
    from paper_2602_11192_b200.runner import current_stream_ptr
    d, F, E, k, C = 4096, 64, 64, 32, 32
    P = _pair(d, F, E, k, C, seed=41)
    for step, T in enumerate((1, 2, 3, 9, 1)):
        P.step(gen.hidden_states(41, 0, "decode", step, T, d), tokens=[0, T - 1] if T > 1 else None)
    x = torch.zeros((1, d), dtype=torch.int16, device="cuda")
    y = torch.full((1, d), 7, dtype=torch.int16, device="cuda")
    before = P.gpu.layer.cache_state()
    P.gpu.layer.forward(current_stream_ptr(), x, 0, y)
    torch.cuda.synchronize()
    assert int(y.min()) == 7 and int(y.max()) == 7          # nothing written
    after = P.gpu.layer.cache_state()
    assert np.array_equal(before[0], after[0]) and before[1] == after[1]
    P.close()


def test_full_cache_has_only_compulsory_misses():
    E, k = 8, 2
    P = _pair(256, 64, E, k, E, seed=3)
    seen = set()
    for step in range(24):
        x = gen.hidden_states(3, 0, "decode", step, 1, 256)
        _, o = P.step(x)
        for e, s, hit, ev in o["req"].tolist():
            assert ev == -1 and bool(hit) == (e in seen)
            seen.add(e)
    _, tot = P.gpu.layer.cache_state()
    assert tot["misses"] == len(seen) and tot["evictions"] == 0
    P.close()


def test_output_does_not_depend_on_cache_size_or_history():
    d, F, E, k = 512, 64, 8, 2
    xs = [gen.hidden_states(5, 0, "decode", s, 2, d) for s in range(6)]
    outs = {}
    for C in (2, 5, 8):
        P = _pair(d, F, E, k, C, seed=5)
        outs[C] = [P.step(x)[0]["out_bits"] for x in xs]
        # warm second pass over the same inputs: same outputs
        again = [P.step(x)[0]["out_bits"] for x in xs]
        for a, b in zip(outs[C], again):
            assert np.array_equal(a, b)
        P.close()
    for C in (5, 8):
        for a, b in zip(outs[C], outs[2]):
            assert np.array_equal(a, b)


def test_shared_experts_and_batch():
    d, F, E, k, C = 512, 48, 10, 3, 4
    P = _pair(d, F, E, k, C, seed=9, n_shared=2)
    P.set_bias(_bias(9, E, 0.3, 4), np.arange(4, dtype=np.int32))
    for step in range(5):
        x = gen.hidden_states(9, 0, "decode", step, 4, d)
        P.step(x)
    P.set_bias(P.bias, (np.arange(37) % 4).astype(np.int32))
    P.step(gen.hidden_states(9, 0, "prefill", 0, 37, d))
    P.close()


def test_prefill_then_decode_with_waves():
    """More distinct experts than slots in one call: the misses come in waves."""
    d, F, E, k, C = 512, 64, 16, 4, 4
    P = _pair(d, F, E, k, C, seed=11)
    x = gen.hidden_states(11, 0, "prefill", 0, 40, d)
    _, o = P.step(x)
    assert o["stats"]["n_distinct"] > C and o["stats"]["groups"] >= 3
    for step in range(6):
        P.step(gen.hidden_states(11, 0, "decode", step, 1, d))
    P.close()


@pytest.mark.parametrize("d,F,E,k,C,n_shared,Ts", [
    (512, 256, 8, 2, 8, 0, (40, 300, 9)),        # everything fits the cache: one compute group after warm-up
    (256, 128, 16, 4, 5, 0, (130, 64)),          # more distinct experts than slots: miss waves
    (1024, 384, 6, 2, 3, 2, (257, 20)),          # shared experts, ragged last m-tile
    (512, 256, 4, 2, 4, 0, (600, 385, 40)),      # many tokens per expert, ragged
    (1024, 384, 4, 2, 2, 1, (700,)),             # many tokens per expert with a shared expert and miss waves
    (256, 256, 2, 2, 2, 0, (1100, 520)),         # every token to both experts: nine m-tiles (CTA pairs, the last one half empty)
])
def test_prefill_grouped_gemm(d, F, E, k, C, n_shared, Ts):
    """Calls of more than 8 tokens run the tensor-core grouped GEMM (d_ff a multiple of 128)."""
    P = _pair(d, F, E, k, C, seed=200 + d // 256, n_shared=n_shared)
    n_seq = 4
    bias = _bias(21, E, 0.5, n_seq)
    step = 0
    for T in Ts:
        P.set_bias(bias, (np.arange(T) % n_seq).astype(np.int32))
        x = gen.hidden_states(300 + d, 0, "prefill", step, T, d)
        # the oracle evaluates a spread of tokens (first, last and every 7th): the FFN is per token
        tokens = sorted(set([0, 1, T - 2, T - 1] + list(range(0, T, 7))))
        P.step(x, tokens=tokens)
        assert P.gpu.layer.last_call_used_gemm()
        step += 1
    # and decode-sized calls on the same handle afterwards (streaming kernel), sharing the cache state
    P.set_bias(bias, np.zeros(2, np.int32))
    P.step(gen.hidden_states(300 + d, 0, "decode", 0, 2, d))
    assert not P.gpu.layer.last_call_used_gemm()
    P.close()


def test_prefill_router_breaks_ties_towards_the_lowest_expert_id():
    """More than 8 tokens go through the general router kernel: with a zero router matrix the logits are
    the bias alone, and a bias with equal entries makes ties that must go to the lowest ids (Eq. 1 with
    the tie rule of the oracle's strict-greater arg-max); all-equal logits select experts 0 .. k-1."""
    d, F, E, k, C = 512, 64, 12, 3, 6
    P = _pair(d, F, E, k, C, seed=81)
    P.w_r = np.zeros_like(P.w_r)
    P.gpu.set_router(P.w_r)
    bias = np.zeros((3, E), np.float32)
    bias[0, [2, 5, 7, 9, 11]] = 1.0            # five tied winners: 2, 5, 7 are taken
    bias[1, :] = 0.25                          # everything equal: 0, 1, 2
    bias[2, [10, 4]] = 3.0                     # two clear winners, then the lowest of the tied rest: 4, 10, 0
    for T in (20, 9, 33):
        seq = (np.arange(T) % 3).astype(np.int32)
        P.set_bias(bias, seq)
        _, o = P.step(gen.hidden_states(81, 0, "prefill", T, T, d), tokens=[0, 1, 2, T - 1])
        for t in range(T):
            want = {0: [2, 5, 7], 1: [0, 1, 2], 2: [4, 10, 0]}[int(seq[t])]
            assert o["idx"][t].tolist() == want
    # the same ties through the decode router (at most 8 tokens)
    P.set_bias(bias, np.arange(3, dtype=np.int32))
    _, o = P.step(gen.hidden_states(81, 0, "decode", 0, 3, d))
    assert o["idx"].tolist() == [[2, 5, 7], [0, 1, 2], [4, 10, 0]]
    P.close()


def test_a_failed_host_copy_leaves_the_handle_usable():
    """Error path of a partly queued call.  The failure is made on the host: a hook makes the first
    host-issued expert copy of the call report an error instead of being issued (nothing faults or
    waits on the device).  The call returns the error, later calls return it too until the cache is
    reset, the stream can be synchronised, and after the reset the layer works again."""
    import torch
    from paper_2602_11192_b200 import MelinoeError, lib
    from paper_2602_11192_b200.runner import current_stream_ptr, to_dev_bf16
    d, F, E, k, C = 512, 128, 8, 2, 4
    P = _pair(d, F, E, k, C, seed=83)
    T = 40                                              # grouped-GEMM path: the host issues the copies
    x = gen.hidden_states(83, 0, "prefill", 0, T, d)
    xd = to_dev_bf16(x)
    out = torch.zeros((T, d), dtype=torch.int16, device="cuda")
    lib().melinoe_debug_fail_host_copy(1)
    with pytest.raises(MelinoeError) as ei:
        P.gpu.layer.forward(current_stream_ptr(), xd, T, out)
    assert ei.value.status == 3
    lib().melinoe_debug_fail_host_copy(0)
    torch.cuda.synchronize()                            # whatever was queued runs to its end
    with pytest.raises(MelinoeError) as ei:
        P.gpu.layer.forward(current_stream_ptr(), xd, T, out)
    assert ei.value.status == 3                         # sticky
    with pytest.raises(MelinoeError):
        P.gpu.layer.cache_state()
    P.reset()                                           # clears the error; both sides start cold again
    P.step(x, tokens=[0, 7, T - 1])
    P.step(gen.hidden_states(83, 0, "decode", 0, 2, d))
    P.close()


def test_request_trace_records_calls_without_synchronising():
    """The request trace: 24 calls (decode-sized ones through the fused planner, two larger ones through the
    general planner) are queued back to back with no synchronisation in between; afterwards the ring holds
    the last 16 calls' records, each equal to what the oracle says of that call: routing indices, gates,
    request records in order, hit and miss counts."""
    import torch
    from paper_2602_11192_b200.budget import read_trace
    from paper_2602_11192_b200.runner import current_stream_ptr, to_dev_bf16
    d, F, E, k, C = 512, 64, 12, 2, 4
    P = _pair(d, F, E, k, C, seed=87)
    L = P.gpu.layer
    max_tok, cap = 8, 16
    rb = L.trace_record_bytes(max_tok)
    assert rb == (32 + 16 * E + 8 * max_tok * k + 15) // 16 * 16
    buf = torch.zeros(cap * rb, dtype=torch.uint8, device="cuda")
    L.set_trace(buf, buf.numel(), max_tok)
    Ts = [1, 3, 8, 1, 20, 2, 1, 5] * 3
    xs = [gen.hidden_states(87, 0, "decode", i, T, d) for i, T in enumerate(Ts)]
    outs = [torch.empty((T, d), dtype=torch.int16, device="cuda") for T in Ts]
    xd = [to_dev_bf16(x) for x in xs]
    s = current_stream_ptr()
    for x, o, T in zip(xd, outs, Ts):
        L.forward(s, x, T, o)                       # nothing waits here
    torch.cuda.synchronize()
    assert L.trace_count() == len(Ts)
    recs = read_trace(buf.cpu().numpy(), cap, E, k, max_tok)
    want = []
    for x in xs:
        idx, gate, _ = oracle.route(x, P.w_r, k)
        want.append((idx, gate, P.cache.call(idx)))
    for n in range(len(Ts) - cap, len(Ts)):
        r = recs[n % cap]
        idx, gate, req = want[n]
        nt = min(Ts[n], max_tok)
        assert r["call_no"] == n + 1 and r["n_tokens"] == Ts[n] and r["status"] == 0
        assert np.array_equal(r["idx"], idx[:nt]) and np.allclose(r["gate"], gate[:nt], rtol=1e-5, atol=1e-7)
        assert np.array_equal(r["req"], req)
        assert r["hits"] == int(req[:, 2].sum()) and r["misses"] == len(req) - int(req[:, 2].sum())
    L.set_trace(None, 0, 0)
    L.forward(s, xd[0], Ts[0], outs[0])
    torch.cuda.synchronize()
    assert L.trace_count() == len(Ts)               # switched off: nothing more is recorded
    P.close()


def test_forward_host_matches_forward_and_is_deterministic():
    import torch
    from paper_2602_11192_b200.runner import current_stream_ptr
    d, F, E, k, C = 512, 64, 8, 2, 3
    P = _pair(d, F, E, k, C, seed=13)
    xs = [gen.hidden_states(13, 0, "decode", s, 3, d) for s in range(5)]
    a = [P.step(x)[0]["out_bits"] for x in xs]
    P.reset()
    hx = torch.empty((3, d), dtype=torch.int16, pin_memory=True)
    hy = torch.empty((3, d), dtype=torch.int16, pin_memory=True)
    hs = torch.zeros(12, dtype=torch.int32, pin_memory=True)
    for i, x in enumerate(xs):
        hx.copy_(torch.from_numpy(x.view(np.int16)))
        P.gpu.layer.forward_host(current_stream_ptr(), hx, 3, hy, hs)
        torch.cuda.synchronize()
        assert np.array_equal(hy.numpy().view(np.uint16), a[i])
        assert int(hs[0]) == 0 and int(hs[1]) == 3
        P.cache.call(oracle.route(x, P.w_r, k)[0])
    # pageable host buffers take the staged route and give the same bits
    P.gpu.layer.reset_cache()
    py, ps = np.empty((3, d), np.int16), np.zeros(12, np.int32)
    for i, x in enumerate(xs):
        px = np.ascontiguousarray(x.view(np.int16))
        P.gpu.layer.forward_host(current_stream_ptr(), px, 3, py, ps)
        torch.cuda.synchronize()
        assert np.array_equal(py.view(np.uint16), a[i])
        assert int(ps[0]) == 0 and int(ps[1]) == 3
    P.close()


def test_preload_fills_the_cache_before_the_first_token():
    d, F, E, k, C = 256, 32, 8, 2, 4
    P = _pair(d, F, E, k, C, seed=15)
    x = gen.hidden_states(15, 0, "decode", 0, 1, d)
    idx, _, _ = oracle.route(x, P.w_r, k)
    P.preload(sorted(idx[0].tolist()))
    _, o = P.step(x)
    assert o["stats"]["misses"] == 0 and o["stats"]["hits"] == k
    eos, tot = P.gpu.layer.cache_state()
    assert tot["misses"] == k and set(eos[:k].tolist()) == set(idx[0].tolist())
    P.close()


@pytest.mark.parametrize("policy", ["lru", "count"])
def test_preload_is_queued_and_matches_the_oracle(policy):
    """Preloads in the middle of a stream of calls (on a warm cache: ids that are resident, ids that
    evict, a full list of cache_slots ids), queued without any host synchronisation between them and
    the calls around them; slot table, totals, counts and the following calls' traces and outputs
    agree with the oracle; then the pooled variant for a batch."""
    d, F, E, k, C = 512, 64, 12, 2, 5
    P = _pair(d, F, E, k, C, seed=17)
    if policy == "count":
        P.set_policy("count", 0.9)
    step = 0
    for ids in ([3, 7], [7, 1, 9, 3, 0], [11], [2, 2, 5]):
        P.preload(ids)
        for _ in range(2):
            P.step(gen.hidden_states(17, 0, "decode", step, 3, d))
            step += 1
    lists = np.array([[4, 6, 8], [6, 8, 10], [8, 1, 4], [0, 8, 6]], np.int32)
    want = oracle.pool_prefetch(lists, E, C)
    assert want.tolist() == [8, 6, 4, 0, 1]
    P.gpu.layer.preload_pooled(lists)
    P.cache.preload(want)
    P.step(gen.hidden_states(17, 0, "decode", step, 4, d))
    eos, _ = P.gpu.layer.cache_state()
    P.close()


@pytest.mark.parametrize("gamma", [1.0, 0.9, 0.5])
def test_count_policy_trace_matches_the_oracle(gamma):
    """Definition C.1's discounted-count eviction (gamma = 1: LFU): requests, victims, compute
    groups' results and the fp32 counts agree with the oracle call by call, decode and prefill."""
    d, F, E, k, C = 256, 64, 16, 2, 4
    P = _pair(d, F, E, k, C, seed=31)
    P.set_policy("count", gamma)
    bias = np.stack([gen.router_bias(31, 0, s, 0.3, E) for s in range(4)])
    n_evict = 0
    for step in range(40):
        T = (1, 3, 8)[step % 3]
        P.set_bias(bias, (np.arange(T) % 4).astype(np.int32))
        _, out = P.step(gen.hidden_states(31, 0, "decode", step, T, d))
        n_evict += int((out["req"][:, 3] >= 0).sum())
    assert n_evict > 20
    P.set_bias(bias, (np.arange(40) % 4).astype(np.int32))
    P.step(gen.hidden_states(31, 0, "prefill", 0, 40, d))     # many misses in one call: one wave each at worst
    # back to LRU on the same cache contents: the trace follows the LRU oracle again
    P.set_policy("lru")
    P.set_bias(bias, np.zeros(1, np.int32))
    for step in range(6):
        P.step(gen.hidden_states(31, 0, "decode", 100 + step, 1, d))
    P.close()


def test_count_policy_with_shared_experts_and_batches():
    """The count policy on a stack with always-resident shared experts (their requests sit between
    the hits and the miss waves in the launch order) and token batches."""
    d, F, E, k, C = 256, 64, 12, 3, 4
    P = _pair(d, F, E, k, C, seed=35, n_shared=2)
    P.set_policy("count", 0.9)
    for step, T in enumerate((4, 1, 8, 2, 30, 1, 5)):
        P.step(gen.hidden_states(35, 0, "decode", step, T, d))
    P.close()


def test_count_policy_preload_and_lfu_keeps_the_hot_experts():
    d, F, E, k, C = 256, 32, 8, 2, 4
    P = _pair(d, F, E, k, C, seed=33)
    P.set_policy("count", 1.0)
    P.preload([5, 1, 6, 2])
    assert np.array_equal(P.gpu.layer.cache_counts(E), P.cache.counts())
    for step in range(12):
        P.step(gen.hidden_states(33, 0, "decode", step, 2, d))
    with pytest.raises(Exception):
        P.gpu.layer.set_policy("count", 1.5)
    P.close()


def test_q4_host_store_matches_the_oracle_and_a_bf16_store_of_the_same_weights():
    """4-bit host store: the misses move 4-bit blobs, the layer computes with the weights the format
    defines.  Against the oracle on its own dequantised weights (tolerance), and bit for bit against
    a second layer whose bf16 store holds those dequantised weights."""
    from paper_2602_11192_b200.runner import LayerSetup
    d, F, E, k, C = 512, 128, 12, 2, 4
    P = _pair(d, F, E, k, C, seed=51, store="q4")
    assert P.bytes_per_miss == 3 * (d * F // 2 + d * F // 32)
    ref = LayerSetup(d, F, E, k, C)
    ref.set_experts(P.weights, [])
    ref.set_router(P.w_r)
    n_miss = 0
    for step, T in enumerate((1, 2, 8, 1, 20, 3, 1, 1)):
        x = gen.hidden_states(51, 0, "decode", step, T, d)
        res, out = P.step(x)
        n_miss += out["stats"]["misses"]
        assert np.array_equal(res["out_bits"], ref.forward_np(x)["out_bits"])
    assert n_miss > 10
    # preload goes through the same expansion
    P.reset()
    ref.layer.reset_cache()
    P.preload([3, 7])
    ref.layer.preload(np.array([3, 7], np.int32))
    x = gen.hidden_states(51, 0, "decode", 99, 4, d)
    res, _ = P.step(x)
    assert np.array_equal(res["out_bits"], ref.forward_np(x)["out_bits"])
    ref.close()
    P.close()


@pytest.mark.parametrize("d,F,E,k,C,n_shared", [(512, 128, 12, 2, 4, 0), (1024, 72, 16, 4, 8, 1), (2048, 64, 16, 8, 8, 0),
                                                (4096, 40, 8, 2, 4, 0)])
def test_q4_slots_match_the_oracle(d, F, E, k, C, n_shared):
    """4-bit cache slots: host link and HBM carry 4-bit blobs only, the FFN kernel expands the codes in
    registers.  Routing, cache trace and statistics bit for bit, activations element-wise, against the
    oracle on the weights the format defines; calls of 1..8 tokens (fetched by the kernel itself), of
    more tokens than slots allow (copies issued by the host) and of several launches; both entry points."""
    P = _pair(d, F, E, k, C, seed=61, n_shared=n_shared, store="q4slots")
    from paper_2602_11192_b200 import melinoe_moe_expert_bytes_q4
    assert P.bytes_per_miss == melinoe_moe_expert_bytes_q4(d, F) and P.gpu.layer.slots == "q4"
    n_miss = 0
    for step, T in enumerate((1, 1, 2, 8, 5, 1, 19, 3, 1, 4)):
        x = gen.hidden_states(61, 0, "decode", step, T, d)
        entry = "static" if T <= 8 and T * k <= 64 and step % 2 == 1 else "forward"
        res, out = P.step(x, entry=entry)
        n_miss += out["stats"]["misses"]
        assert not P.gpu.layer.last_call_used_gemm()
    assert n_miss > 6
    P.set_policy("count", 0.9)
    P.reset()
    P.preload(list(range(min(C, 3))))
    for step in range(6):
        P.step(gen.hidden_states(61, 0, "decode", 50 + step, 1 + step % 3, d))
    # a bf16 store cannot be registered on this handle, nor 4-bit slots made for a width the kernel does not split
    with pytest.raises(Exception):
        P.gpu.layer.register_host_experts([0] * E, 3 * d * F * 2)
    P.close()
    from paper_2602_11192_b200 import MoELayer
    with pytest.raises(Exception):
        MoELayer(1536, 64, 8, 2, 4, slots="q4")


def test_parity_without_programmatic_launch():
    """The decode kernels are launched with programmatic stream serialisation by default; the
    same parity must hold with the attribute switched off (the switch is read once per process,
    hence the child process)."""
    import os
    import subprocess
    import sys
    here = os.path.dirname(os.path.abspath(__file__))
    code = (
        "import sys; sys.path.insert(0, %r); sys.path.insert(0, %r)\n"
        "import numpy as np, gen\n"
        "from parity_util import Pair\n"
        "P = Pair(512, 64, 16, 2, 4, seed=61)\n"
        "for step, T in enumerate((1, 4, 1, 8, 2, 1, 12, 1)):\n"
        "    P.step(gen.hidden_states(61, 0, 'decode', step, T, 512))\n"
        "P.close()\n"
        "print('child ok')\n" % (os.path.dirname(here), here))
    env = dict(os.environ, MELINOE_MOE_NO_PDL="1")
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "child ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


def _child(code_body, env_extra):
    import os
    import subprocess
    import sys
    here = os.path.dirname(os.path.abspath(__file__))
    code = ("import sys; sys.path.insert(0, %r); sys.path.insert(0, %r)\n"
            "import numpy as np, gen\nfrom parity_util import Pair\n" % (os.path.dirname(here), here)) + code_body + "print('child ok')\n"
    r = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, **env_extra), capture_output=True, text=True,
                       timeout=600)
    assert r.returncode == 0 and "child ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


def test_parity_with_every_transfer_issued_by_the_host():
    """MELINOE_MOE_HOST_COPIES: decode calls, too, wait for their plan on the host and fetch with
    cudaMemcpyAsync (the switch is read once per process, hence the child process)."""
    _child("P = Pair(512, 64, 16, 2, 4, seed=62)\n"
           "for step, T in enumerate((1, 2, 1, 8, 2, 1, 12, 1)):\n"
           "    P.step(gen.hidden_states(62, 0, 'decode', step, T, 512))\n"
           "P.close()\n", {"MELINOE_MOE_HOST_COPIES": "1"})


def test_parity_of_the_single_cta_gemm_on_a_call_of_many_tokens():
    """MELINOE_MOE_GEMM_SINGLE: a call that would pair CTAs (300 tokens per expert) through the
    cta_group::1 form of the grouped GEMM."""
    _child("P = Pair(512, 256, 4, 2, 4, seed=63)\n"
           "x = gen.hidden_states(63, 0, 'prefill', 0, 600, 512)\n"
           "P.step(x, tokens=sorted(set([0, 1, 598, 599] + list(range(0, 600, 7)))))\n"
           "assert P.gpu.layer.last_call_used_gemm()\n"
           "P.close()\n", {"MELINOE_MOE_GEMM_SINGLE": "1"})


def test_trace_miss_proxies_match_the_oracle():
    """Soft (Section 3.1) and hard (Definition C.1) miss proxies of recorded traces, every cache size
    at once: hard misses exact, soft proxy to fp64 rounding; then a budget split over the layers."""
    from paper_2602_11192_b200.budget import miss_curves, allocate_slots
    rs = np.random.default_rng(71)
    L, T, K, E = 3, 300, 2, 12
    trace = np.empty((L, T, K), np.int32)
    for l, alpha in enumerate((0.05, 0.5, 50.0)):             # from concentrated to uniform routing
        pref = rs.dirichlet(np.full(E, alpha)) + 1e-6
        pref /= pref.sum()
        for t in range(T):
            trace[l, t] = rs.choice(E, size=K, replace=False, p=pref)
    sizes = list(range(K, E + 1))
    for gamma in (1.0, 0.9, 0.0):
        soft, hard = miss_curves(trace, E, gamma, sizes)
        for l in range(L):
            for j, c in enumerate(sizes):
                so, ho = oracle.miss_proxies(trace[l], E, c, gamma)
                assert hard[l, j] == int(ho.sum()), (gamma, l, c)
                assert abs(soft[l, j] - so.mean()) <= 1e-10 * max(1.0, abs(so.mean())), (gamma, l, c)
        assert np.all(np.diff(hard, axis=1) <= 0)            # a larger gamma-cache never transfers more
    _, hard = miss_curves(trace, E, 0.9, sizes)
    slots = allocate_slots(hard, sizes, 3 * K + 9)
    assert sum(slots) == 3 * K + 9 and slots[0] <= slots[1]   # concentrated routing needs the fewest slots
    # a configuration that names nothing is marked, not evaluated
    import torch
    from paper_2602_11192_b200 import binding as B
    from paper_2602_11192_b200.runner import current_stream_ptr
    cfg = (B.ProxyConfig * 2)(B.ProxyConfig(7, 4, 0.9), B.ProxyConfig(0, 0, 0.9))
    cfg_dev = torch.frombuffer(bytearray(bytes(cfg)), dtype=torch.uint8).cuda()
    so = torch.zeros(2, dtype=torch.float64, device="cuda")
    ha = torch.zeros(2, dtype=torch.int64, device="cuda")
    B.melinoe_trace_miss_proxies(current_stream_ptr(), torch.from_numpy(trace).cuda(), L, T, K, E, cfg_dev, 2, so, ha)
    torch.cuda.synchronize()
    assert bool(torch.isnan(so).all()) and ha.tolist() == [-1, -1]


def test_argument_and_state_errors():
    import torch
    from paper_2602_11192_b200 import MoELayer, MelinoeError, melinoe_moe_expert_bytes
    from paper_2602_11192_b200.runner import current_stream_ptr
    for bad in ((250, 64, 8, 2, 4), (256, 63, 8, 2, 4), (256, 64, 65, 2, 4), (256, 64, 8, 3, 2), (256, 64, 8, 2, 9)):
        with pytest.raises(MelinoeError):
            MoELayer(*bad)
    L = MoELayer(256, 64, 4, 2, 2)
    x = torch.zeros((1, 256), dtype=torch.int16, device="cuda")
    y = torch.zeros((1, 256), dtype=torch.int16, device="cuda")
    with pytest.raises(MelinoeError) as ei:
        L.forward(current_stream_ptr(), x, 1, y)
    assert ei.value.status == 2                       # router / experts not set
    eb = melinoe_moe_expert_bytes(256, 64)
    pageable = torch.zeros((4, eb), dtype=torch.uint8)
    with pytest.raises(MelinoeError) as ei:
        L.register_host_experts([pageable.data_ptr() + i * eb for i in range(4)], eb)
    assert ei.value.status == 1                       # pageable memory is rejected, never staged
    pinned = torch.zeros((4, eb), dtype=torch.uint8, pin_memory=True)
    with pytest.raises(MelinoeError):
        L.register_host_experts([pinned.data_ptr() + i * eb for i in range(4)], eb - 2)
    L.register_host_experts([pinned.data_ptr() + i * eb for i in range(4)], eb, keep=pinned)
    w = torch.zeros((4, 256), dtype=torch.int16, device="cuda")
    L.set_router(w)
    L.forward(current_stream_ptr(), x, 0, y)          # zero tokens: no-op
    L.forward(current_stream_ptr(), x, 1, y)
    torch.cuda.synchronize()
    assert int(y.abs().max()) == 0                    # all-zero weights give exactly zero
    idx, gate = L.last_routing(1)
    assert idx.tolist() == [[0, 1]] and np.allclose(gate, 0.5)   # all-equal logits: lowest ids, equal gates
    L.destroy()
