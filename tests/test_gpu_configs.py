"""Parity at the benchmark's sizes: the synthetic stacks of the five workload shapes, driven the
way bench.py drives them (one handle per layer, device-resident inputs), against the oracle.

Routing indices, gates, request traces and statistics are compared for every call (they are
cheap to recompute on the CPU); activations are compared on a sample of (layer, token) pairs,
which is sound because a token's output depends only on its inputs and routing, never on the
cache state.  The largest shapes run with 4 of their layers (each layer is an independent
handle with its own weights, router, bias and cache; full width and call shapes are kept) and
32 of their decode steps; every call's sampled tokens (up to 8 per call, first and last
included) are compared element by element as well as by norm.
"""
import numpy as np
import pytest

import gen
import oracle
from parity_util import _q4_roundtrip, elementwise_excess

pytestmark = pytest.mark.gpu

REL_TOL = 2e-2          # the specified bound at full size


def _run_stack(name, n_layers, alpha, C, decode_steps, sample_layers, prefill=True, y_tokens=8, store="bf16"):
    import torch
    from paper_2602_11192_b200.workload import Stack, bits_of, stats_rows
    cfg = gen.config_by_name(name)
    st = Stack(cfg, alpha, C, n_layers=n_layers, store=store)
    L, B, k, E, d = st.L, cfg.batch, cfg.top_k, cfg.n_experts, cfg.d_model
    caches = [oracle.ExpertCache(C, E) for _ in range(L)]
    weights = {}
    for l in sample_layers:
        wg, wu, wd = st.layer_weights(l)
        ws = [(bits_of(wg[e]), bits_of(wu[e]), bits_of(wd[e])) for e in range(E + cfg.n_shared)]
        if store == "q4slots":
            ws = [_q4_roundtrip(w) for w in ws]        # the weights the 4-bit format defines
        weights[l] = (ws, (wg, wu, wd))

    def check(phase, step, T, seq):
        x = st.hidden_bits(phase, step)                                  # [L][T][d]
        xd = torch.from_numpy(x.view(np.int16)).cuda()
        out = torch.empty_like(xd)
        stats = torch.zeros((L, 12), dtype=torch.int32, device="cuda")
        st.set_phase(phase)
        st.forward_all(xd, out, stats)
        torch.cuda.synchronize()
        out_bits = out.cpu().numpy().view(np.uint16)
        sr = stats_rows(stats)
        worst = 0.0
        for l in range(L):
            idx_o, gate_o, lg_o = oracle.route(x[l], st.w_r[l], k, st.bias[l], seq)
            req_o = caches[l].call(idx_o)
            layer = st.layers[l].layer
            idx_g, gate_g = layer.last_routing(T)
            assert np.array_equal(idx_g, idx_o), "routing differs: %s layer %d %s step %d" % (name, l, phase, step)
            assert np.allclose(gate_g, gate_o, rtol=1e-5, atol=1e-7)
            assert np.array_equal(layer.last_requests(), req_o), "trace differs: %s layer %d" % (name, l)
            hits = int(req_o[:, 2].sum())
            assert sr["status"][l] == 0 and sr["n_distinct"][l] == len(req_o)
            assert sr["hits"][l] == hits and sr["misses"][l] == len(req_o) - hits
            assert layer.last_call_used_gemm() == (T > 8 and cfg.d_ff % 128 == 0 and store == "bf16")
            if l in weights:
                toks = sorted(set(np.linspace(0, T - 1, min(T, y_tokens)).astype(int).tolist()))
                y = oracle.ffn_combine(x[l], idx_o, gate_o, weights[l][0], cfg.d_ff, cfg.n_shared, toks)
                yg = gen.bf16_bits_to_f32(out_bits[l][toks]).astype(np.float64)
                err = np.linalg.norm(yg - y, axis=1) / np.maximum(np.linalg.norm(y, axis=1), 1e-30)
                assert np.all(np.isfinite(yg)) and err.max() <= REL_TOL, "rel err %.3e" % err.max()
                ex = elementwise_excess(out_bits[l][toks], y)
                assert ex <= 1.0, "%s layer %d: an output element is off by %.2f times its bound" % (name, l, ex)
                worst = max(worst, float(err.max()))
        return worst

    if prefill and cfg.prefill_tokens:
        check("prefill", 0, B * cfg.prefill_tokens, st.prefill_seq)
    for s in range(decode_steps):
        check("decode", s, B, st.decode_seq)
    tot = [st.layers[l].layer.cache_state()[1] for l in range(L)]
    for l in range(L):
        _, _, t_o = caches[l].state()
        assert tot[l] == t_o
    st.close()


def test_olmoe_full_stack_as_benchmarked():
    """configs[1]: all 16 layers, 16 slots per layer, the prompt and the first decode steps."""
    _run_stack("olmoe", None, 0.1, 16, decode_steps=12, sample_layers=(0, 7, 15))


@pytest.mark.parametrize("alpha", [1.0, 10.0])
def test_olmoe_other_routing_concentrations(alpha):
    """configs[1], alpha = 1 and 10 (near-uniform routing thrashes the cache): 4 of the 16 layers, the
    prompt and 32 decode steps."""
    _run_stack("olmoe", 4, alpha, 16, decode_steps=32, sample_layers=(0, 3))


@pytest.mark.parametrize("C,alpha", [(2, 0.2), (2, 2.0), (4, 0.2), (4, 2.0)])
def test_mixtral_shape(C, alpha):
    """configs[2]: d 4096, d_ff 14336, 8 experts, top-2, 2 and 4 slots, alpha 0.2 and 2.0; 4 of the 32
    layers, the 256-token prompt and 32 decode steps."""
    _run_stack("mixtral", 4, alpha, C, decode_steps=32, sample_layers=(1,), y_tokens=8)


def test_phi35_shape_batch_of_eight():
    """configs[3]: d 4096, d_ff 6400, 16 experts, top-2, 6 slots, 8 sequences: 4096-token prefill
    through the grouped GEMM, then 32 decode steps of 8 tokens; 4 of the 32 layers."""
    _run_stack("phi35", 4, 0.3, 6, decode_steps=32, sample_layers=(2,), y_tokens=8)


@pytest.mark.parametrize("alpha", [0.1, 1.0])
def test_deepseek_shape_with_shared_experts(alpha):
    """configs[4]: d 2048, d_ff 1408, 64 routed + 2 shared experts, top-6, 12 slots, 4 sequences:
    8192-token prefill, then 32 decode steps of 4 tokens; 4 of the 28 layers."""
    _run_stack("deepseek", 4, alpha, 12, decode_steps=32, sample_layers=(3,), y_tokens=8)


@pytest.mark.parametrize("name,n_layers,alpha,C,steps,prefill", [
    ("olmoe", 4, 0.1, 16, 32, True),          # d 2048; the 128-token prompt runs as 16 launches of 8 tokens
    ("mixtral", 2, 0.2, 4, 16, False),        # d 4096, one token
    ("phi35", 2, 0.3, 6, 16, False),          # d 4096, eight tokens (both token groups of the down product)
    ("deepseek", 2, 0.1, 12, 16, False),      # shared experts (4-bit as well), four tokens
])
def test_four_bit_slots_at_full_width(name, n_layers, alpha, C, steps, prefill):
    """The workload shapes with 4-bit cache slots (codes expanded inside the FFN kernel): routing, traces and
    statistics bit for bit, activations element-wise against the oracle on the weights the format defines."""
    _run_stack(name, n_layers, alpha, C, decode_steps=steps, sample_layers=(n_layers - 1,), prefill=prefill, store="q4slots")


def test_per_layer_budget_end_to_end_makes_fewer_transfers():
    """Per-layer cache budgets from a recorded trace, end to end on the OLMoE shape: four layers whose
    routing runs from concentrated to near-uniform decode 96 tokens with 16 slots each while their request
    traces are recorded on the device (no synchronisation per call); the routing traces go through the
    miss-proxy evaluator (Definition C.1's hard cache) for every cache size, the library splits the same
    total of 64 slots over the layers, and a second stack with those sizes decodes the same tokens.  Both
    runs' request records equal the oracle's, and the budgeted stack makes fewer transfers."""
    import torch
    from paper_2602_11192_b200.budget import allocate_slots, miss_curves, read_trace
    from paper_2602_11192_b200.workload import Stack
    cfg = gen.config_by_name("olmoe")
    L, steps, E, k = 4, 96, cfg.n_experts, cfg.top_k
    alphas = (0.05, 0.3, 3.0, 30.0)

    def run(slots):
        st = Stack(cfg, 1.0, slots, n_layers=L)
        st.bias = [np.stack([gen.router_bias(cfg.seed, l, 0, alphas[l], E)]) for l in range(L)]
        st.set_phase("decode")
        bufs = []
        for ls in st.layers:
            rb = ls.layer.trace_record_bytes(1)
            b = torch.zeros(steps * rb, dtype=torch.uint8, device="cuda")
            ls.layer.set_trace(b, b.numel(), 1)
            bufs.append(b)
        out = torch.empty((L, 1, cfg.d_model), dtype=torch.int16, device="cuda")
        xs = [st.hidden_bits("decode", s) for s in range(steps)]
        xd = [torch.from_numpy(x.view(np.int16)).cuda() for x in xs]
        for s in range(steps):
            st.forward_all(xd[s], out, None)
        torch.cuda.synchronize()
        recs = [read_trace(b.cpu().numpy(), steps, E, k, 1) for b in bufs]
        # against the oracle, request by request
        Cs = [slots] * L if np.isscalar(slots) else list(slots)
        for l in range(L):
            cache = oracle.ExpertCache(Cs[l], E)
            for s in range(steps):
                idx, _, _ = oracle.route(xs[s][l], st.w_r[l], k, st.bias[l], np.zeros(1, np.int32))
                assert np.array_equal(recs[l][s]["idx"], idx)
                assert np.array_equal(recs[l][s]["req"], cache.call(idx)), (l, s)
        trace = np.stack([np.stack([r["idx"][0] for r in recs[l]]) for l in range(L)])[:, :, None, :].reshape(L, steps, k)
        misses = [sum(r["misses"] for r in recs[l]) for l in range(L)]
        st.close()
        return trace, misses

    trace, uniform = run(16)
    sizes = list(range(k, 41))
    _, hard = miss_curves(trace, E, 0.5, sizes)
    slots = allocate_slots(hard, sizes, 16 * L)
    assert sum(slots) == 16 * L and min(slots) >= k
    assert len(set(slots)) > 1                      # layers with different routing get different sizes
    _, budgeted = run(slots)
    assert sum(budgeted) < sum(uniform), (slots, budgeted, uniform)


def test_repeated_runs_with_heavy_miss_traffic_are_bit_identical():
    """Two cold-start runs of the same OLMoE-shaped steps (near-uniform routing: several transfers
    per layer and token, miss waves, slot reuse inside a call) give the same output bits and the
    same statistics: nothing in the transfer / compute overlap is left to chance."""
    import torch
    from paper_2602_11192_b200.workload import Stack, stats_rows
    cfg = gen.config_by_name("olmoe")
    L, steps = 2, 60
    runs = []
    for rep in range(2):
        st = Stack(cfg, 10.0, cfg.cache_slots[0], n_layers=L)
        out = torch.empty((L, 1, cfg.d_model), dtype=torch.int16, device="cuda")
        stats = torch.zeros((steps, L, 12), dtype=torch.int32, device="cuda")
        outs = []
        for s in range(steps):
            x = torch.from_numpy(st.hidden_bits("decode", s).view(np.int16)).cuda()
            st.forward_all(x, out, stats[s])
            outs.append(out.clone())
        torch.cuda.synchronize()
        r = stats_rows(stats)
        assert int(r["status"].max()) == 0 and int(r["misses"].sum()) > 3 * L * steps
        runs.append((torch.stack(outs).cpu().numpy(), stats.cpu().numpy()[:, :, :8]))
        st.close()
    assert np.array_equal(runs[0][0], runs[1][0]) and np.array_equal(runs[0][1], runs[1][1])

