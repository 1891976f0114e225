"""The allocation-free entry point, melinoe_moe_forward_static, against melinoe_moe_forward.

Some users of this library cannot let a forward call allocate: a serving process that has
given all remaining device memory to its KV cache would see a stray cudaMalloc fail (or stall
the whole device while it synchronises).  For them the library offers the same call on a fixed
scratch array that lives in its device image.  This test drives both entry points through the C
ABI on the same layer and inputs and requires the same outputs, on two calls in a row (the
second call finds the scratch as the first one left it).

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
    (512, 200, 8, 2, 4, 1, 0),      # ragged d_ff: the zero padding behind h rows matters
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
