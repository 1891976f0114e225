"""Helpers for the GPU-vs-oracle parity tests: build the same layer on both sides from the
seeded generators and compare call by call."""
from __future__ import annotations

import numpy as np

import gen
import oracle

REL_TOL = 2e-2      # per-token ||y_gpu - y_ref|| / ||y_ref||, the bound the layer is specified to
TIGHT_TOL = 8e-3    # what bf16 rounding of h and of the output actually allows (2 x 2^-9 rms-ish)
GATE_RTOL = 1e-5
# Element-wise bound on an output: |y_gpu - y_ref| <= ELEM_A * |y_ref| + ELEM_B * rms(y_ref of the token).
# bf16 keeps 8 significant bits, so one rounding moves a value by at most 2^-8 of itself.  ELEM_A is that
# bound for the final rounding of y (with 1 % to spare for the fp32 sums behind it).  ELEM_B covers the one
# other rounding on the path, gate * h to bf16: its error is uniform within half a unit in the last place,
# a relative standard deviation of 2^-8 * 0.7355 / sqrt(3) = 1.66e-3 for a mantissa spread log-uniformly
# over a binade; it enters y_i as sum_f W_d[i, f] * dh_f, whose standard deviation is 1.66e-3 times the
# root of sum_f (W_d[i, f] * h_f)^2, i.e. about 1.66e-3 * rms(y) for weights that are independent of h;
# 1.2e-2 is seven standard deviations.  A wrong output column, a token given another token's expert, a
# missing expert or a dropped block of hidden units moves elements by the order of rms(y) itself.
ELEM_A = 1.01 * 2.0 ** -8
ELEM_B = 1.2e-2


def make_weights(seed, layer, E, d, F, n_shared=0):
    return [gen.expert_weights(seed, layer, e, d, F) for e in range(E + n_shared)]


def _q4_roundtrip(w):
    """The weights a 4-bit store defines: W_g and W_u quantised along their rows, W_d along its columns
    (the quantisation groups follow the d_model axis in all three)."""
    wg, wu, wd = w
    q = lambda m: oracle.dequantize_q4(*oracle.quantize_q4(np.ascontiguousarray(m)))
    return q(wg), q(wu), np.ascontiguousarray(q(wd.T).T)


def rel_err_per_token(y_gpu_bits: np.ndarray, y_ref: np.ndarray) -> np.ndarray:
    yg = gen.bf16_bits_to_f32(y_gpu_bits).astype(np.float64)
    num = np.linalg.norm(yg - y_ref, axis=1)
    den = np.linalg.norm(y_ref, axis=1)
    return num / np.maximum(den, 1e-30)


def elementwise_excess(y_gpu_bits: np.ndarray, y_ref: np.ndarray) -> float:
    """Largest |y_gpu - y_ref| / (ELEM_A |y_ref| + ELEM_B rms(y_ref of the token)) over all elements: <= 1 passes."""
    yg = gen.bf16_bits_to_f32(y_gpu_bits).astype(np.float64)
    rms = np.sqrt(np.mean(y_ref * y_ref, axis=1, keepdims=True))
    bound = ELEM_A * np.abs(y_ref) + ELEM_B * rms + 1e-30
    return float(np.max(np.abs(yg - y_ref) / bound))


class Pair:
    """The CUDA layer and the oracle side by side on identical weights."""

    def __init__(self, d, F, E, k, C, seed=0, layer=0, n_shared=0, store="bf16"):
        from paper_2602_11192_b200.runner import LayerSetup
        from paper_2602_11192_b200 import melinoe_moe_expert_bytes_q4
        self.d, self.F, self.E, self.k, self.C, self.n_shared = d, F, E, k, C, n_shared
        self.weights = make_weights(seed, layer, E, d, F, n_shared)
        self.w_r = gen.router_weights(seed, layer, E, d)
        self.gpu = LayerSetup(d, F, E, k, C, n_shared, slots="q4" if store == "q4slots" else "bf16")
        self.bytes_per_miss = 3 * d * F * 2
        if store in ("q4", "q4slots"):
            # the library quantises the original weights; the oracle computes with what the 4-bit
            # format defines as the layer's weights (its own quantise + dequantise)
            assert n_shared == 0 or store == "q4slots"
            self.gpu.set_experts_q4(self.weights[:E], self.weights[E:])
            self.weights = [_q4_roundtrip(w) for w in self.weights]
            self.bytes_per_miss = melinoe_moe_expert_bytes_q4(d, F)
        else:
            self.gpu.set_experts(self.weights[:E], self.weights[E:])
        self.gpu.set_router(self.w_r)
        self.cache = oracle.ExpertCache(C, E)
        self.bias = None
        self.seq = None

    def set_bias(self, bias, seq):
        self.bias, self.seq = bias, seq
        self.gpu.set_bias(bias, seq)

    def set_policy(self, policy, gamma=0.0):
        self.gpu.layer.set_policy(policy, gamma)
        self.cache.set_policy(policy, gamma)

    def preload(self, ids):
        self.gpu.layer.preload(np.asarray(ids, np.int32))
        self.cache.preload(ids)

    def reset(self):
        self.gpu.layer.reset_cache()
        self.cache.reset()

    def step(self, x_bits, check_y=True, tokens=None, tol=TIGHT_TOL, entry="forward"):
        """One forward call on both sides; asserts parity; returns (gpu result, oracle result).
        entry: "forward" or "static" (melinoe_moe_forward_static)."""
        T = x_bits.shape[0]
        res = self.gpu.forward_np(x_bits, entry=entry)
        L = self.gpu.layer
        idx_g, gate_g = L.last_routing(T)
        lg_g = L.last_logits(T)
        req_g = L.last_requests()
        cnt_g, off_g, perm_g = L.last_gather(T)
        eos_g, tot_g = L.cache_state()

        idx_o, gate_o, lg_o = oracle.route(x_bits, self.w_r, self.k, self.bias, self.seq)
        req_o = self.cache.call(idx_o)
        cnt_o, off_o, perm_o = oracle.gather(idx_o, self.E)
        eos_o, _, tot_o = self.cache.state()

        assert np.array_equal(lg_g.view(np.uint32), lg_o.view(np.uint32)), "router logits differ in bits"
        assert np.array_equal(idx_g, idx_o), "routing indices differ"
        assert np.allclose(gate_g, gate_o, rtol=GATE_RTOL, atol=1e-7), "gates differ"
        assert np.allclose(gate_g.sum(axis=1), 1.0, atol=1e-5)
        assert np.array_equal(req_g, req_o), "cache trace differs:\n%s\n%s" % (req_g, req_o)
        assert np.array_equal(cnt_g, cnt_o) and np.array_equal(off_g, off_o) and np.array_equal(perm_g, perm_o)
        assert np.array_equal(eos_g, eos_o) and tot_g == tot_o
        # the discounted counts decide evictions: same bits on both sides
        assert np.array_equal(L.cache_counts(self.E).view(np.uint32), self.cache.counts().view(np.uint32))
        st = res["stats"]
        assert st["status"] == 0 and st["n_tokens"] == T and st["n_distinct"] == len(req_o)
        assert st["hits"] == int(req_o[:, 2].sum()) and st["misses"] == len(req_o) - int(req_o[:, 2].sum())
        assert st["evictions"] == int((req_o[:, 3] >= 0).sum())
        assert st["bytes_h2d"] == st["misses"] * self.bytes_per_miss
        out = {"idx": idx_o, "gate": gate_o, "req": req_o, "stats": st}
        if check_y:
            y_ref = oracle.ffn_combine(x_bits, idx_o, gate_o, self.weights, self.F, self.n_shared, tokens)
            yb = res["out_bits"] if tokens is None else res["out_bits"][np.asarray(tokens)]
            err = rel_err_per_token(yb, y_ref)
            assert np.all(np.isfinite(gen.bf16_bits_to_f32(res["out_bits"]))), "non-finite output"
            assert err.max() <= tol, "activation rel err %.3e > %.1e" % (err.max(), tol)
            ex = elementwise_excess(yb, y_ref)
            assert ex <= 1.0, "an output element is off by %.2f times its bound" % ex
            out["err"] = err
        return res, out

    def close(self):
        self.gpu.close()
