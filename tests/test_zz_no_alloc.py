"""The allocation-free entry point, melinoe_moe_forward_static.

Some users of this library cannot let a forward call allocate: a serving process that has
given all remaining device memory to its KV cache would see a stray cudaMalloc fail (or stall
the whole device while it synchronises).  For them the library offers the same call on a fixed
scratch array that lives in its device image.  These tests drive that entry point through the C
ABI: against melinoe_moe_forward on the same layer and inputs, on two calls in a row (the second
call finds the scratch as the first one left it), and against the CPU oracle (routing, cache
trace, statistics, activations) under both eviction policies, with device memory watched for any
allocation.

Kept in a file that pytest collects last, so a failure here cannot hide the other tests of a
run that stops at the first failure.
"""
import numpy as np
import pytest

import gen

pytestmark = pytest.mark.gpu

REL_TOL = 8e-3   # the tolerance of the other GPU tests (per-token relative L2 error)


def _rel_err(a_bits, b_bits):
    a = gen.bf16_bits_to_f32(a_bits).astype(np.float64)
    b = gen.bf16_bits_to_f32(b_bits).astype(np.float64)
    return np.linalg.norm(a - b, axis=1) / np.maximum(np.linalg.norm(b, axis=1), 1e-30)


@pytest.mark.parametrize("d,F,E,k,C,T,n_shared", [
    (512, 200, 8, 2, 4, 1, 0),      # d_ff that is not a multiple of the tile height
    (1024, 64, 8, 2, 8, 4, 1),      # several tokens, a shared expert
])
def test_static_scratch_forward_matches_forward(d, F, E, k, C, T, n_shared):
    import torch
    from paper_2602_11192_b200 import MelinoeError, lib
    from paper_2602_11192_b200.runner import LayerSetup, current_stream_ptr, to_dev_bf16

    assert lib().melinoe_moe_static_scratch_bytes() < 16 * 2 ** 20
    seed = 40 + d // 256
    ws = [gen.expert_weights(seed, 0, e, d, F) for e in range(E + n_shared)]
    L = LayerSetup(d, F, E, k, C, n_shared)
    L.set_experts(ws[:E], ws[E:])
    L.set_router(gen.router_weights(seed, 0, E, d))
    stream = current_stream_ptr()
    xs = [to_dev_bf16(gen.hidden_states(seed, 0, "decode", s, T, d)) for s in range(2)]

    # reference: the ordinary entry point, cold cache
    want = []
    for x in xs:
        out = torch.empty((T, d), dtype=torch.int16, device="cuda")
        L.layer.forward(stream, x, T, out)
        torch.cuda.synchronize()
        want.append(out.cpu().numpy().view(np.uint16))

    # the static-scratch entry point on the same handle, again from a cold cache, twice in a row
    L.layer.reset_cache()
    stats = torch.zeros(12, dtype=torch.int32, device="cuda")
    for x, w in zip(xs, want):
        out = torch.full((T, d), 0x7FC0, dtype=torch.int16, device="cuda")     # NaN pattern: must be overwritten
        L.layer.forward_static(stream, x, T, out, stats)
        torch.cuda.synchronize()
        got = out.cpu().numpy().view(np.uint16)
        st = stats.cpu().numpy()
        assert int(st[0]) == 0 and int(st[1]) == T
        assert np.all(np.isfinite(gen.bf16_bits_to_f32(got)))
        err = _rel_err(got, w)
        assert err.max() <= REL_TOL, "static-scratch output differs: rel err %.3e" % err.max()

    # sizes beyond the static scratch are refused with a clear status, not served by allocating
    big = torch.zeros((9, d), dtype=torch.int16, device="cuda")
    with pytest.raises(MelinoeError) as ei:
        L.layer.forward_static(stream, big, 9, big)
    assert ei.value.status == 6
    L.close()


@pytest.mark.parametrize("policy,gamma", [("lru", 0.0), ("count", 1.0), ("count", 0.5)])
def test_static_scratch_forward_against_the_oracle_without_allocating(policy, gamma):
    """Every call through the static entry point, from the very first call of a fresh handle, checked
    against the oracle like any other call: routing bits, cache trace, statistics, activations element
    by element.  The cache is smaller than what a call can request, so experts are evicted inside calls
    (under the count policy a call may evict an expert it has itself just fetched).  Free device memory
    is read before and after: the calls allocate nothing."""
    import torch
    from parity_util import Pair
    d, F, E, k, C = 512, 64, 12, 3, 4
    P = Pair(d, F, E, k, C, seed=91)
    if policy != "lru":
        P.set_policy(policy, gamma)
    bias = np.stack([gen.router_bias(91, 0, s, 0.4, E) for s in range(4)])
    torch.cuda.synchronize()
    xs = [(T, gen.hidden_states(91, 0, "decode", step, T, d)) for step, T in enumerate((1, 4, 2, 8, 1, 3, 8, 1, 2, 1))]
    n_evict = 0
    free0 = None
    for i, (T, x) in enumerate(xs):
        P.set_bias(bias, (np.arange(T) % 4).astype(np.int32))
        _, o = P.step(x, entry="static")
        n_evict += o["stats"]["evictions"]
        if i == 0:
            free0 = torch.cuda.mem_get_info()[0]        # after the first call: torch's own pools are warm
    assert n_evict >= 8
    assert torch.cuda.mem_get_info()[0] == free0, "device memory changed across static-scratch calls"
    P.close()


def test_two_handles_share_the_static_scratch_back_to_back():
    """Two layers of different widths alternate on the one static array, on one stream: each call finds
    what the other left there and must not depend on it."""
    from parity_util import Pair
    A = Pair(512, 200, 8, 2, 3, seed=93)
    B = Pair(1024, 64, 6, 2, 2, seed=94)
    for step in range(4):
        A.step(gen.hidden_states(93, 0, "decode", step, 2, 512), entry="static")
        B.step(gen.hidden_states(94, 0, "decode", step, 5, 1024), entry="static")
    A.close()
    B.close()
