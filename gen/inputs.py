"""Counter-based, seeded generators for every tensor the MoE-layer path consumes.

Recipe (stand-in for real prompts driven through trained OLMoE / Mixtral /
Phi-3.5-MoE / DeepSeekMoE checkpoints, which are not available offline):

* router matrix W_r [E][d] and expert matrices W_g [F][d], W_u [F][d], W_d [d][F]:
  i.i.d. N(0, 0.02^2), rounded to bf16 (round-to-nearest-even);
* hidden states [T][d]: i.i.d. N(0, 1) rounded to bf16, drawn independently per
  (layer, phase, step): layer inputs are teacher-forced, they never depend on a
  previous layer's output, so routing is a pure function of the seeded inputs;
* per-(sequence, layer) router bias b = ln(max(pi, 1e-12)) with pi ~ Dirichlet(alpha * 1_E):
  small alpha concentrates a sequence's routing on few experts, which is the effect
  that the paper's fine-tuning has (Section 2, "Fine-Tuning to Achieve
  Cache-Friendliness"); large alpha approaches uniform routing.

Every draw comes from numpy's Philox generator keyed by (seed, tag, indices), so any
(layer, token, expert) block can be regenerated on its own.  bf16 tensors are carried
as uint16 bit patterns (numpy has no bf16 dtype).
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

__all__ = [
    "f32_to_bf16_bits", "bf16_bits_to_f32", "rng_for", "router_weights", "hidden_states",
    "router_bias", "expert_weights", "MoEConfig", "CONFIGS", "config_by_name",
    "fill_expert_store_fast",
]


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def rng_for(seed: int, tag: str, *idx: int) -> np.random.Generator:
    """A Philox stream keyed by (seed, tag, idx...): independent of call order."""
    h = hashlib.blake2b(digest_size=16)
    h.update(repr((int(seed), str(tag), tuple(int(i) for i in idx))).encode())
    key = np.frombuffer(h.digest(), dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _normal_bf16(g: np.random.Generator, shape, std: float) -> np.ndarray:
    x = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return f32_to_bf16_bits(x)


def router_weights(seed: int, layer: int, n_experts: int, d_model: int) -> np.ndarray:
    """W_r [E][d] as bf16 bits, N(0, 0.02^2)."""
    return _normal_bf16(rng_for(seed, "router", layer), (n_experts, d_model), 0.02)


def hidden_states(seed: int, layer: int, phase: str, step: int, n_tokens: int, d_model: int) -> np.ndarray:
    """hidden [T][d] as bf16 bits, N(0,1); phase is 'prefill' or 'decode'."""
    return _normal_bf16(rng_for(seed, "hidden:" + phase, layer, step), (n_tokens, d_model), 1.0)


def router_bias(seed: int, layer: int, seq: int, alpha: float, n_experts: int) -> np.ndarray:
    """ln Dirichlet(alpha) preference of one sequence at one layer, fp32 [E].

    Gamma(alpha) draws are taken in log space (ln G(a) = ln G(a+1) + ln(U)/a) so that
    small alpha does not underflow; the result is clamped below at ln(1e-12).
    """
    g = rng_for(seed, "bias:%r" % float(alpha), layer, seq)
    lg = np.log(g.standard_gamma(alpha + 1.0, size=n_experts)) + np.log(1.0 - g.random(n_experts)) / alpha
    lpi = lg - (np.max(lg) + np.log(np.sum(np.exp(lg - np.max(lg)))))
    return np.maximum(lpi, np.log(1e-12)).astype(np.float32)


def expert_weights(seed: int, layer: int, expert: int, d_model: int, d_ff: int
                   ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """(W_g [F][d], W_u [F][d], W_d [d][F]) as bf16 bits, N(0, 0.02^2): the paper's shapes (Eq. 3)."""
    g = rng_for(seed, "expert", layer, expert)
    wg = _normal_bf16(g, (d_ff, d_model), 0.02)
    wu = _normal_bf16(g, (d_ff, d_model), 0.02)
    wd = _normal_bf16(g, (d_model, d_ff), 0.02)
    return wg, wu, wd


def fill_expert_store_fast(seed: int, layer: int, n_experts: int, d_model: int, d_ff: int):
    """Paper-layout expert matrices for one whole layer, generated with torch's seeded RNG.

    Returns three torch CPU tensors of dtype bfloat16: W_g [E][F][d], W_u [E][F][d],
    W_d [E][d][F], N(0, 0.02^2).  Used for the large stacks (tens of GB), where the numpy
    Philox path is too slow; the draw happens on the GPU when one is present and on the
    CPU otherwise, so values are reproducible per device type, not across them.  Expert
    values never influence routing or the cache trace.
    """
    import torch
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    gen = torch.Generator(device=dev)
    gen.manual_seed((int(seed) * 1000003 + int(layer)) & 0x7FFFFFFFFFFF)
    outs = []
    for shape in ((n_experts, d_ff, d_model), (n_experts, d_ff, d_model), (n_experts, d_model, d_ff)):
        t = torch.empty(shape, dtype=torch.float32, device=dev).normal_(0.0, 0.02, generator=gen)
        outs.append(t.to(torch.bfloat16).cpu())
    return tuple(outs)


@dataclass(frozen=True)
class MoEConfig:
    """One synthetic stack: shapes, cache size, call shapes, bias concentrations."""
    name: str
    seed: int
    n_layers: int
    d_model: int
    d_ff: int
    n_experts: int
    top_k: int
    cache_slots: Tuple[int, ...]
    alphas: Tuple[float, ...]
    batch: int            # independent sequences decoded together
    prefill_tokens: int   # prompt tokens per sequence (0: no prefill call)
    decode_steps: int
    n_shared: int = 0     # always-resident shared experts

    @property
    def expert_bytes(self) -> int:
        return 3 * self.d_model * self.d_ff * 2


CONFIGS: Dict[str, MoEConfig] = {
    c.name: c for c in (
        MoEConfig("tiny", 0, 1, 256, 512, 8, 2, (4,), (0.3,), 1, 0, 32),
        MoEConfig("olmoe", 2, 16, 2048, 1024, 64, 8, (16,), (0.1, 1.0, 10.0), 1, 128, 256),
        MoEConfig("mixtral", 3, 32, 4096, 14336, 8, 2, (2, 4), (0.2, 2.0), 1, 256, 512),
        MoEConfig("phi35", 4, 32, 4096, 6400, 16, 2, (6,), (0.3,), 8, 512, 256),
        MoEConfig("deepseek", 5, 28, 2048, 1408, 64, 6, (12,), (0.1, 1.0), 4, 2048, 512, n_shared=2),
    )
}


def config_by_name(name: str) -> MoEConfig:
    return CONFIGS[name]
