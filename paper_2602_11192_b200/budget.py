"""Per-layer cache sizes under one budget, from recorded routing traces.

`miss_curves` asks the library for the transfers a gamma-cache of every size would have made on each
layer's trace (Definition C.1's hard cache, evaluated on the device); `allocate_slots` is host
logic: it hands out the budget one slot at a time to the layer whose transfers drop most.
torch is used for device memory only.
"""
from __future__ import annotations

import ctypes as C
from typing import List, Sequence

import numpy as np
import torch

from . import binding as B
from .runner import current_stream_ptr

__all__ = ["miss_curves", "allocate_slots"]


def miss_curves(trace: np.ndarray, n_experts: int, gamma: float, sizes: Sequence[int]):
    """trace [L][T][K] int32 -> (soft [L][len(sizes)] fp64, hard [L][len(sizes)] int64)."""
    trace = np.ascontiguousarray(trace, dtype=np.int32)
    L, T, K = trace.shape
    cfg = (B.ProxyConfig * (L * len(sizes)))()
    for l in range(L):
        for j, c in enumerate(sizes):
            cfg[l * len(sizes) + j] = B.ProxyConfig(l, int(c), float(gamma))
    cfg_dev = torch.frombuffer(bytearray(bytes(cfg)), dtype=torch.uint8).cuda()
    tr_dev = torch.from_numpy(trace).cuda()
    soft = torch.empty(L * len(sizes), dtype=torch.float64, device="cuda")
    hard = torch.empty(L * len(sizes), dtype=torch.int64, device="cuda")
    B.melinoe_trace_miss_proxies(current_stream_ptr(), tr_dev, L, T, K, n_experts, cfg_dev, L * len(sizes), soft, hard)
    torch.cuda.synchronize()
    return soft.cpu().numpy().reshape(L, -1), hard.cpu().numpy().reshape(L, -1)


def allocate_slots(hard: np.ndarray, sizes: Sequence[int], budget: int) -> List[int]:
    """hard[l][j] = transfers of layer l with sizes[j] slots (sizes ascending, step 1).  Starts every
    layer at sizes[0] and spends the rest of `budget` (total slots over all layers) greedily on the
    layer whose next slot saves the most transfers; ties go to the lower layer.  Returns the
    slots per layer."""
    hard = np.asarray(hard)
    L, n = hard.shape
    assert n == len(sizes) and all(sizes[j + 1] == sizes[j] + 1 for j in range(n - 1))
    at = [0] * L
    left = int(budget) - L * int(sizes[0])
    if left < 0:
        raise ValueError("the budget does not cover the smallest size on every layer")
    while left > 0:
        best, gain = -1, -1
        for l in range(L):
            if at[l] + 1 < n:
                g = int(hard[l][at[l]] - hard[l][at[l] + 1])
                if g > gain:
                    best, gain = l, g
        if best < 0:
            break
        at[best] += 1
        left -= 1
    return [int(sizes[a]) for a in at]
