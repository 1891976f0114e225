"""Times the prefill expert FFN (tensor-core grouped GEMM) of one synthetic layer.

    python -m paper_2602_11192_b200.prefill_probe [phi35|deepseek|olmoe|mixtral] [--tokens N] [--reps R]

One layer of the named stack with every expert resident (cache = all experts, warmed by one
call), one prefill call of the stack's prompt shape per repetition; reports the FFN time
measured by the library's per-launch events and the implied bf16 throughput
(6 * d_model * d_ff flop per (token, expert) pair).  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402
from paper_2602_11192_b200.workload import Stack, stats_rows  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("workload", nargs="?", default="phi35")
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--reps", type=int, default=5)
    a = ap.parse_args()
    cfg = gen.config_by_name(a.workload)
    T = a.tokens or cfg.batch * cfg.prefill_tokens
    st = Stack(cfg, cfg.alphas[-1], cfg.n_experts, n_layers=1)
    L = st.layers[0]
    L.layer.reserve(T)
    seq = (np.arange(T) * cfg.batch // T).astype(np.int32)
    L.set_bias(st.bias[0], seq)
    x = torch.from_numpy(gen.hidden_states(cfg.seed, 0, "prefill", 0, T, cfg.d_model).view(np.int16)).cuda()
    out = torch.empty_like(x)
    stats = torch.zeros((1, 12), dtype=torch.int32, device="cuda")
    s = int(torch.cuda.current_stream().cuda_stream)
    L.layer.forward(s, x, T, out, stats)          # cold: fetches every needed expert
    torch.cuda.synchronize()
    L.layer.enable_timing(True)
    best = None
    for _ in range(a.reps):
        L.layer.forward(s, x, T, out, stats)
        torch.cuda.synchronize()
        ms, n = L.layer.ffn_time_ms()
        best = ms if best is None else min(best, ms)
    r = stats_rows(stats)
    pairs = T * (cfg.top_k + cfg.n_shared)
    flop = 6.0 * cfg.d_model * cfg.d_ff * pairs
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak = float(peaks.get("bf16_tflops", 1590.0))
    print(json.dumps({
        "workload": a.workload, "tokens": T, "pairs": pairs, "used_gemm": L.layer.last_call_used_gemm(),
        "ffn_ms": best, "launches_per_call": int(n), "tflops": flop / (best * 1e-3) / 1e12,
        "peak_tflops": peak, "frac": flop / (best * 1e-3) / 1e12 / peak, "peak_source": "measured" if peaks else "fallback",
        "misses_last_call": int(r["misses"][0]), "distinct_experts": int(r["n_distinct"][0])}))
    st.close()


if __name__ == "__main__":
    main()
