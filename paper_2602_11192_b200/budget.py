"""Per-layer cache sizes under one budget, from recorded routing traces.

`miss_curves` asks the library for the transfers a gamma-cache of every size would have made on each
layer's trace (Definition C.1's hard cache, evaluated on the device); `allocate_slots` asks it to hand
out the budget one slot at a time to the layer whose transfers drop most; `read_trace` unpacks the
records of a request trace.  Argument marshalling only; torch is used for device memory only.
"""
from __future__ import annotations

import ctypes as C
from typing import List, Sequence

import numpy as np
import torch

from . import binding as B
from .runner import current_stream_ptr

__all__ = ["miss_curves", "allocate_slots", "read_trace"]


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
    """hard[l][j] = transfers of layer l with sizes[j] slots (sizes ascending, step 1).  The library hands
    the budget (total slots over all layers) out greedily (melinoe_allocate_slots); returns the slots per
    layer."""
    hard = np.ascontiguousarray(hard, dtype=np.int64)
    L, n = hard.shape
    assert n == len(sizes) and all(sizes[j + 1] == sizes[j] + 1 for j in range(n - 1))
    out = np.zeros(L, dtype=np.int32)
    rc = B.lib().melinoe_allocate_slots(hard.ctypes.data, L, n, int(sizes[0]), int(budget), out.ctypes.data)
    if rc:
        raise ValueError("the budget does not cover the smallest size on every layer")
    return [int(v) for v in out]


def read_trace(buf: np.ndarray, n_records: int, n_experts: int, top_k: int, max_tokens: int):
    """Unpack the first n_records records of a request-trace buffer (bytes, as copied from the device).
    Returns a list of dicts: call_no, n_tokens, n_requests, hits, misses, status, req [n_requests][4],
    idx [min(n_tokens, max_tokens)][top_k], gate likewise."""
    raw = np.ascontiguousarray(buf).view(np.uint8).reshape(-1)
    req_off = 32
    idx_off = req_off + 16 * n_experts
    gate_off = idx_off + 4 * max_tokens * top_k
    rb = (gate_off + 4 * max_tokens * top_k + 15) // 16 * 16
    out = []
    for i in range(n_records):
        r = raw[i * rb:(i + 1) * rb]
        hdr = r[:32].view(np.int32)
        n_tok, n_req = int(hdr[2]), int(hdr[3])
        nt = min(n_tok, max_tokens)
        out.append({"call_no": int(r[:8].view(np.uint64)[0]), "n_tokens": n_tok, "n_requests": n_req, "hits": int(hdr[4]),
                    "misses": int(hdr[5]), "status": int(hdr[6]),
                    "req": r[req_off:req_off + 16 * n_req].view(np.int32).reshape(n_req, 4).copy(),
                    "idx": r[idx_off:idx_off + 4 * nt * top_k].view(np.int32).reshape(nt, top_k).copy(),
                    "gate": r[gate_off:gate_off + 4 * nt * top_k].view(np.float32).reshape(nt, top_k).copy()})
    return out
