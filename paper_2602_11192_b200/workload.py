"""Synthetic MoE stacks: one library handle per layer over a pinned host expert store.

Builds the stacks that the benchmark, the smoke check and the full-size tests drive.  Input
data comes from the seeded generators in `gen`; every step of the layer runs in the CUDA
library.  torch is used for device / pinned memory and streams only.
"""
from __future__ import annotations

import time
from typing import Dict, List, Optional

import numpy as np
import torch

import gen

from . import binding as B
from .runner import LayerSetup, current_stream_ptr, to_dev_bf16

__all__ = ["Stack", "bits_of", "stats_rows"]


def bits_of(t: torch.Tensor) -> np.ndarray:
    """uint16 bit patterns of a CPU bf16 tensor (no copy)."""
    return t.view(torch.int16).numpy().view(np.uint16)


class Stack:
    """All layers of one synthetic stack for one (alpha, cache_slots) run.

    hidden states are teacher-forced (drawn per layer and step, never fed from the previous
    layer), so routing and the cache trace are functions of the seeded inputs alone.
    """

    def __init__(self, cfg: gen.MoEConfig, alpha: float, cache_slots: int, n_layers: Optional[int] = None,
                 verbose: bool = False, policy: str = "lru", gamma: float = 0.0, store: str = "bf16"):
        self.cfg, self.alpha = cfg, float(alpha)
        self.L = cfg.n_layers if n_layers is None else int(n_layers)
        # one cache size for every layer, or one per layer (see budget.allocate_slots)
        self.C = [int(cache_slots)] * self.L if np.isscalar(cache_slots) else [int(c) for c in cache_slots]
        assert len(self.C) == self.L
        self.layers: List[LayerSetup] = []
        self.w_r: List[np.ndarray] = []
        self.bias: List[np.ndarray] = []
        t0 = time.time()
        for l in range(self.L):
            # store: "bf16"; "q4" = 4-bit host store expanded into bf16 slots; "q4slots" = 4-bit store and 4-bit slots
            ls = LayerSetup(cfg.d_model, cfg.d_ff, cfg.n_experts, cfg.top_k, self.C[l], cfg.n_shared,
                            slots="q4" if store == "q4slots" else "bf16")
            wg, wu, wd = gen.fill_expert_store_fast(cfg.seed, l, cfg.n_experts + cfg.n_shared, cfg.d_model, cfg.d_ff)
            if store in ("q4", "q4slots"):
                ls.set_experts_stacked_q4(wg[:cfg.n_experts], wu[:cfg.n_experts], wd[:cfg.n_experts])
            else:
                ls.set_experts_stacked(wg[:cfg.n_experts], wu[:cfg.n_experts], wd[:cfg.n_experts])
            if cfg.n_shared:
                ls.set_shared_stacked(wg[cfg.n_experts:], wu[cfg.n_experts:], wd[cfg.n_experts:])
            del wg, wu, wd
            w_r = gen.router_weights(cfg.seed, l, cfg.n_experts, cfg.d_model)
            ls.set_router(w_r)
            if policy != "lru":
                ls.layer.set_policy(policy, gamma)
            bias = np.stack([gen.router_bias(cfg.seed, l, s, self.alpha, cfg.n_experts) for s in range(cfg.batch)])
            self.w_r.append(w_r)
            self.bias.append(bias)
            self.layers.append(ls)
            if verbose:
                print("  layer %d/%d ready (%.1f s)" % (l + 1, self.L, time.time() - t0), flush=True)
        self.decode_seq = np.arange(cfg.batch, dtype=np.int32)
        self.prefill_seq = np.repeat(np.arange(cfg.batch, dtype=np.int32), max(cfg.prefill_tokens, 1))
        self.set_phase("decode")
        max_t = max(cfg.batch, cfg.batch * cfg.prefill_tokens)
        for ls in self.layers:
            ls.layer.reserve(max_t)

    # -- inputs
    def set_phase(self, phase: str) -> None:
        seq = self.decode_seq if phase == "decode" else self.prefill_seq
        for ls, b in zip(self.layers, self.bias):
            ls.set_bias(b, seq)

    def layer_weights(self, l: int):
        """Paper-layout matrices of layer l again (same seed, same device type): (W_g, W_u, W_d) torch bf16."""
        c = self.cfg
        return gen.fill_expert_store_fast(c.seed, l, c.n_experts + c.n_shared, c.d_model, c.d_ff)

    def hidden_bits(self, phase: str, step: int) -> np.ndarray:
        """[L][T][d] bf16 bits of one step's layer inputs."""
        c = self.cfg
        T = c.batch if phase == "decode" else c.batch * c.prefill_tokens
        return np.stack([gen.hidden_states(c.seed, l, phase, step, T, c.d_model) for l in range(self.L)])

    def set_policy(self, policy: str, gamma: float = 0.0) -> None:
        for ls in self.layers:
            ls.layer.set_policy(policy, gamma)

    def reset(self) -> None:
        for ls in self.layers:
            ls.layer.reset_cache()

    # -- the calls
    def forward_all(self, x_dev: torch.Tensor, out_dev: torch.Tensor, stats_dev: Optional[torch.Tensor]) -> None:
        """One step: x_dev / out_dev [L][T][d] (int16 storage), stats_dev [L][12] int32 or None."""
        self._loop(False, x_dev, out_dev, stats_dev)

    def forward_all_host(self, x_host: torch.Tensor, out_host: torch.Tensor, stats_host: Optional[torch.Tensor]) -> None:
        """Same step through the host-buffer entry point (pinned buffers)."""
        self._loop(True, x_host, out_host, stats_host)

    def _loop(self, host: bool, x: torch.Tensor, out: torch.Tensor, stats: Optional[torch.Tensor]) -> None:
        assert x.is_contiguous() and out.is_contiguous() and x.shape[0] == self.L and out.shape == x.shape
        s = current_stream_ptr()
        T = int(x.shape[1])
        xp, op = x.data_ptr(), out.data_ptr()
        step = T * self.cfg.d_model * 2
        sp = 0 if stats is None else stats.data_ptr()
        if stats is not None:
            assert stats.is_contiguous() and stats.dtype == torch.int32 and tuple(stats.shape) == (self.L, 12)
        for l, ls in enumerate(self.layers):
            st = (sp + l * 48) if sp else None
            if host:
                ls.layer.forward_host(s, xp + l * step, T, op + l * step, st)
            else:
                ls.layer.forward(s, xp + l * step, T, op + l * step, st)

    def close(self) -> None:
        for ls in self.layers:
            ls.close()
        self.layers = []


def stats_rows(stats: torch.Tensor) -> Dict[str, np.ndarray]:
    """Decode a [..., 12] int32 tensor of melinoe_moe_stats records into named arrays."""
    s = stats.cpu().numpy().reshape(-1, 12)
    return {"status": s[:, 0], "n_tokens": s[:, 1], "n_distinct": s[:, 2], "hits": s[:, 3], "misses": s[:, 4],
            "evictions": s[:, 5], "groups": s[:, 6]}
