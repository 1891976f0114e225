#!/usr/bin/env python
"""Benchmark of the cached MoE layer stack: decode tokens/s on the OLMoE-shaped workload.

One step = one decode token through every layer of the stack (16 forward calls, each
running router, planning, miss transfers, expert FFN and combine).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched through torch.distributed.run) every rank drives an independent replica
of the stack on its own GPU; there is no data-path collective, only the timing barrier.
"""
from __future__ import annotations

import argparse
import faulthandler
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the decode FFN kernel divided by the launch's
# algorithmic bytes (8 experts x 12.58 MB), from an ncu capture of a two-layer case of this workload (100.75 MB
# read + 3.5 MB written against 100.66 MB); traffic grows in proportion to the experts streamed.  To be set to
# None when the kernel changes, until the counters have been taken again.
DRAM_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.036

METRIC = "decode tokens/s (OLMoE-shaped, cache-limited)"
UNIT = "tokens/s"
WORKLOAD = "olmoe"


def phase(msg: str, limit_s: int = 600) -> None:
    """Progress line on stderr and a watchdog: a phase that takes longer than limit_s dumps every
    thread's stack and ends the process instead of holding the GPU."""
    sys.stderr.write("[bench %7.1f s] %s\n" % (time.time() - T_START, msg))
    sys.stderr.flush()
    faulthandler.cancel_dump_traceback_later()
    faulthandler.dump_traceback_later(limit_s, exit=True)


T_START = time.time()


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--alpha", type=float, default=None, help="headline router-bias concentration (default: the workload's first)")
    ap.add_argument("--layers", type=int, default=None, help="use fewer layers (debugging only; marks the line)")
    ap.add_argument("--store", default="bf16", choices=["bf16", "q4", "q4slots"],
                    help="expert format of the headline run (profiling aid; anything but bf16 marks the line): "
                         "q4 = 4-bit host store expanded into bf16 slots, q4slots = 4-bit store and 4-bit slots")
    ap.add_argument("--slots", type=int, default=None, help="cache slots per layer of the headline run (marks the line)")
    ap.add_argument("--shape", default=None, choices=["mixtral", "phi35", "deepseek"],
                    help="profiling aid: run only that workload shape's record (decode, FFN analysis, prefill GEMM) on "
                         "--layers layers (default 1), print it and exit; not a benchmark line")
    ap.add_argument("--timeline", action="store_true",
                    help="profiling aid: per-CTA time stamps of the decode FFN kernel (melinoe_moe_set_timeline) on a "
                         "--layers (default 2) layer stack with --slots slots (default: every expert resident), "
                         "printed as medians and maxima over the CTAs; not a benchmark line")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the other alphas and the resident-cache run")
    return ap.parse_args()


def workload_config(cfg, alpha, C, n_layers):
    return {
        "workload": "OLMoE-shaped stack: %d layers, d_model=%d, d_ff=%d, %d experts, top-%d, cache %d experts/layer, "
                    "batch %d, %d-token prompt then decode; router bias Dirichlet alpha=%g; seed %d"
                    % (n_layers, cfg.d_model, cfg.d_ff, cfg.n_experts, cfg.top_k, C, cfg.batch, cfg.prefill_tokens,
                       alpha, cfg.seed),
        "step": "one decode token through all %d layers" % n_layers,
        "l2": "inputs larger than L2: %.0f MB of expert weights are streamed per step, %.0f MB of slots per layer"
              % (n_layers * cfg.top_k * cfg.expert_bytes / 1e6, C * cfg.expert_bytes / 1e6),
        "parallelism": "replicas",
    }


# --------------------------------------------------------------------------- clocks

class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.path = os.path.join("/tmp", "bench_clocks_%d_%d.csv" % (os.getpid(), gpu_index))

    def start(self):
        try:
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.fh, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [v.strip() for v in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# --------------------------------------------------------------------------- ranks

def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The slowest rank's time: every rank runs an independent replica, the job is as slow as the
    slowest of them.  dist is torch.distributed (initialised) or None for a single process."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(tokens_per_rank: int, world: int, ms: float) -> float:
    """Whole-job tokens/s of `world` replicas that each processed tokens_per_rank tokens in ms."""
    return tokens_per_rank * world / (ms * 1e-3)


# --------------------------------------------------------------------------- our arm

REPEATS = 5          # every timed region is measured this many times: median and best are reported


class Runner:
    """One synthetic stack plus its decode inputs: prepares (cold start, prompt, warm-up) and times regions."""

    def __init__(self, torch, M, gen, cfg, alpha, C, L, K, W, store="bf16", dist=None):
        from paper_2602_11192_b200.workload import Stack
        self.torch, self.M, self.gen, self.cfg, self.dist = torch, M, gen, cfg, dist
        self.L, self.K, self.W = L, K, W
        self.stack = Stack(cfg, alpha, C, n_layers=L, store=store)
        d = cfg.d_model
        n_steps = W + K
        dec = np.stack([self.stack.hidden_bits("decode", s) for s in range(n_steps)])          # [S][L][B][d]
        self.dec_host = torch.from_numpy(dec.view(np.int16)).pin_memory()
        self.dec_dev = self.dec_host.cuda()
        self.pre_dev = None
        if cfg.prefill_tokens:
            self.pre_dev = torch.from_numpy(self.stack.hidden_bits("prefill", 0).view(np.int16)).cuda()
            self.pre_out = torch.empty_like(self.pre_dev)
        self.out_dev = torch.empty((L, cfg.batch, d), dtype=torch.int16, device="cuda")
        self.out_host = torch.empty((L, cfg.batch, d), dtype=torch.int16).pin_memory()
        self.stats_dev = torch.zeros((n_steps, L, 12), dtype=torch.int32, device="cuda")
        self.stats_host = torch.zeros((L, 12), dtype=torch.int32).pin_memory()

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def prepare(self, alpha, timing_prefill=False):
        """Cold start, prompt, then the warm-up decode steps are left to the caller."""
        st, cfg, gen = self.stack, self.cfg, self.gen
        if alpha != st.alpha:
            st.alpha = alpha
            st.bias = [np.stack([gen.router_bias(cfg.seed, l, s, alpha, cfg.n_experts) for s in range(cfg.batch)])
                       for l in range(self.L)]
        st.reset()
        if self.pre_dev is not None:
            st.set_phase("prefill")
            if timing_prefill:
                for ls in st.layers:
                    ls.layer.enable_timing(True)
            st.forward_all(self.pre_dev, self.pre_out, None)
        st.set_phase("decode")
        self.torch.cuda.synchronize()

    def timed_device(self, alpha, with_kernel_timing=False):
        """W warm-up steps, then K timed steps with device-resident inputs.  Returns ms, launches, the
        timed steps' statistics and, with kernel timing, the per-launch FFN times (ms) in call order."""
        torch, M, st, W, K = self.torch, self.M, self.stack, self.W, self.K
        self.prepare(alpha)
        self.stats_dev.zero_()
        for s in range(W):
            st.forward_all(self.dec_dev[s], self.out_dev, self.stats_dev[s])
        torch.cuda.synchronize()
        if with_kernel_timing:
            for ls in st.layers:
                ls.layer.enable_timing(True)
        self.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = M.melinoe_launch_count()
        e0.record()
        for s in range(W, W + K):
            st.forward_all(self.dec_dev[s], self.out_dev, self.stats_dev[s])
        e1.record()
        torch.cuda.synchronize()
        self.barrier()
        ms = e0.elapsed_time(e1)
        launches = M.melinoe_launch_count() - n0
        per_launch = None
        self.copy_ms = self.copy_bytes = 0.0
        if with_kernel_timing:
            per_launch = []                                   # [layer] -> times of its K calls' launches
            for ls in st.layers:
                per_launch.append(ls.layer.ffn_launch_times_ms())
                ls.layer.ffn_time_ms()
                cm, cb = ls.layer.transfer_time_ms()          # host-issued transfers only (copy-stream events)
                self.copy_ms += cm
                self.copy_bytes += cb
                ls.layer.enable_timing(False)
        stats = stats_arrays(self.stats_dev[W:W + K])
        if int(stats["status"].max()) != 0:
            raise SystemExit("device-side status %d in the timed region" % int(stats["status"].max()))
        return ms, launches, stats, per_launch

    def timed_e2e(self, alpha):
        """The same steps through the host-buffer entry point, one stream synchronisation per step."""
        torch, st, W, K = self.torch, self.stack, self.W, self.K
        self.prepare(alpha)
        s_ptr = torch.cuda.current_stream()
        for s in range(W):
            st.forward_all_host(self.dec_host[s], self.out_host, self.stats_host)
            s_ptr.synchronize()
        self.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for s in range(W, W + K):
            st.forward_all_host(self.dec_host[s], self.out_host, self.stats_host)
            s_ptr.synchronize()
        e1.record()
        torch.cuda.synchronize()
        self.barrier()
        return e0.elapsed_time(e1)

    def close(self):
        self.stack.close()


def stats_arrays(stats_dev):
    """[K][L][12] int32 statistics -> dict of [K][L] arrays."""
    s = stats_dev.cpu().numpy()
    return {"status": s[..., 0], "n_tokens": s[..., 1], "n_distinct": s[..., 2], "hits": s[..., 3], "misses": s[..., 4],
            "evictions": s[..., 5], "groups": s[..., 6]}


def med_best(vals, higher_is_better=True):
    v = sorted(vals)
    return statistics.median(v), (v[-1] if higher_is_better else v[0])


def hit_summary(cfg, stats, K, L):
    h, m = int(stats["hits"].sum()), int(stats["misses"].sum())
    return {"hit_rate": h / max(h + m, 1), "misses_per_layer_per_token": m / (K * L * cfg.batch),
            "h2d_expert_bytes_per_step": m * cfg.expert_bytes / K}


def ffn_launch_analysis(cfg, stats, per_launch, hbm_peak, link_peak, expert_bytes=None):
    """Per-launch CUDA-event times of the decode FFN kernel against what each launch moved.
    One launch per call here (the kernel fetches missed experts itself), so launch i of layer l is call i.
    Launches whose experts were all resident are bound by HBM: bytes = experts x bytes per expert.  Launches
    that fetched experts are bound by the host link for those: bytes over the link / launch time."""
    B_e = cfg.expert_bytes if expert_bytes is None else expert_bytes
    res_bytes = res_ms = 0.0
    res_n = 0
    miss_bytes = miss_ms = 0.0
    miss_n = 0
    all_bytes = all_ms = 0.0
    K, L = stats["misses"].shape
    if any(len(per_launch[l]) != K for l in range(L)):
        # not one launch per call (calls whose transfers the host issues, one launch per compute group): no
        # per-call attribution, only the sum over all launches
        ms = float(sum(float(t.sum()) for t in per_launch))
        n = int(sum(len(t) for t in per_launch))
        by = float((stats["n_distinct"].astype(np.int64) + cfg.n_shared).sum()) * B_e
        g = by / (ms * 1e-3) / 1e9
        return {"resident": None, "fetching": None,
                "all": {"launches": n, "avg_launch_us": 1e3 * ms / max(n, 1), "gbs": g, "frac_of_hbm": g / hbm_peak,
                        "note": "one launch per compute group (the host issues this shape's transfers): experts streamed "
                                "from their slots x bytes per expert / summed launch times"}}
    for l in range(L):
        t = per_launch[l]
        for i in range(K):
            experts = int(stats["n_distinct"][i, l]) + cfg.n_shared
            m = int(stats["misses"][i, l])
            all_bytes += experts * B_e
            all_ms += float(t[i])
            if m == 0:
                res_bytes += experts * B_e
                res_ms += float(t[i])
                res_n += 1
            else:
                miss_bytes += m * B_e
                miss_ms += float(t[i])
                miss_n += 1
    out = {"resident": None, "fetching": None, "all": None}
    if res_n:
        g = res_bytes / (res_ms * 1e-3) / 1e9
        out["resident"] = {"launches": res_n, "avg_launch_us": 1e3 * res_ms / res_n, "bytes_per_launch": res_bytes / res_n,
                           "gbs": g, "frac_of_hbm": g / hbm_peak}
    if miss_n:
        g = miss_bytes / (miss_ms * 1e-3) / 1e9
        out["fetching"] = {"launches": miss_n, "avg_launch_us": 1e3 * miss_ms / miss_n, "link_bytes_per_launch": miss_bytes / miss_n,
                           "link_gbs": g, "frac_of_link": g / link_peak if link_peak else None}
    g = all_bytes / (all_ms * 1e-3) / 1e9
    out["all"] = {"launches": res_n + miss_n, "avg_launch_us": 1e3 * all_ms / max(res_n + miss_n, 1), "gbs": g,
                  "frac_of_hbm": g / hbm_peak}
    return out


def host_link_gbs(torch):
    """Pinned host -> device copy of 512 MiB on a side stream: the link's own rate."""
    n = 512 << 20
    hb = torch.empty(n, dtype=torch.uint8).pin_memory()
    db = torch.empty(n, dtype=torch.uint8, device="cuda")
    st_ = torch.cuda.Stream()
    best = 0.0
    with torch.cuda.stream(st_):
        for _ in range(4):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st_)
            db.copy_(hb, non_blocking=True)
            b.record(st_)
            st_.synchronize()
            best = max(best, n / (a.elapsed_time(b) * 1e-3) / 1e9)
    del hb, db
    return best


def preload_record(torch, R, cfg, alpha, C, L, n_steps):
    """First n_steps decode tokens from an empty cache (no prompt), plain and after melinoe_moe_preload of
    each layer's C most preferred experts of the sequence (Eq. 5 with the bias standing in for the predictor)."""
    st = R.stack
    out = {}
    for mode in ("cold", "preloaded"):
        st.reset()
        st.set_phase("decode")
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        if mode == "preloaded":
            for l, ls in enumerate(st.layers):
                pref = np.argsort(-st.bias[l].max(axis=0), kind="stable")[:C].astype(np.int32)
                ls.layer.preload(pref)
        t1 = time.perf_counter()
        torch.cuda.synchronize()
        t2 = time.perf_counter()
        R.stats_dev.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for s in range(n_steps):
            st.forward_all(R.dec_dev[s], R.out_dev, R.stats_dev[s])
        e1.record()
        torch.cuda.synchronize()
        sa = stats_arrays(R.stats_dev[:n_steps])
        out[mode] = {"decode_ms": e0.elapsed_time(e1), "misses": int(sa["misses"].sum()),
                     "misses_per_layer_per_token": float(sa["misses"].sum()) / (n_steps * L * cfg.batch)}
        if mode == "preloaded":
            out[mode]["preload_queue_ms"] = (t1 - t0) * 1e3
            out[mode]["preload_ms"] = (t2 - t0) * 1e3
            out[mode]["preloaded_bytes"] = int(L * C * cfg.expert_bytes)
    out["tokens"] = n_steps
    out["saved_ms"] = out["cold"]["decode_ms"] - out["preloaded"]["decode_ms"]
    out["note"] = ("%d decode tokens from an empty cache; preload = every layer's %d most preferred experts of the sequence's "
                   "router bias, queued with melinoe_moe_preload (returns at once: preload_queue_ms is the host time of the "
                   "%d calls, preload_ms the time until the copies have landed)" % (n_steps, C, L))
    return out


def shape_record(torch, M, gen, name, n_layers, K, W, hbm_peak, link_peak, peaks, store="bf16"):
    """Decode throughput, FFN roofline and (where the prompt runs the grouped GEMM) the prefill GEMM's
    rate of one of the other workload shapes, at its full width with a reduced number of layers."""
    cfg = gen.config_by_name(name)
    C, alpha = cfg.cache_slots[0], cfg.alphas[0]
    eb = M.melinoe_moe_expert_bytes_q4(cfg.d_model, cfg.d_ff) if store == "q4slots" else cfg.expert_bytes
    R = Runner(torch, M, gen, cfg, alpha, C, n_layers, K, W, store=store)
    rec = {"store": store, "slot_bytes": eb, "workload": "%s-shaped: d_model=%d, d_ff=%d, %d experts (+%d shared), top-%d, cache %d/layer, batch %d, "
                       "%d-token prompts, alpha=%g" % (name, cfg.d_model, cfg.d_ff, cfg.n_experts, cfg.n_shared, cfg.top_k, C,
                                                       cfg.batch, cfg.prefill_tokens, alpha),
           "layers": n_layers, "reduced_layers": n_layers != cfg.n_layers, "decode_steps": K}
    vals = []
    for _ in range(3):
        ms, _, st, _ = R.timed_device(alpha)
        vals.append(cfg.batch * K / (ms * 1e-3))
    rec["tokens_per_s_median"], rec["tokens_per_s_best"] = med_best(vals)
    rec.update(hit_summary(cfg, st, K, n_layers))
    _, _, st2, per_launch = R.timed_device(alpha, with_kernel_timing=True)
    rec["ffn"] = ffn_launch_analysis(cfg, st2, per_launch, hbm_peak, link_peak, expert_bytes=eb)
    if R.copy_ms > 0:
        g = R.copy_bytes / (R.copy_ms * 1e-3) / 1e9
        rec["host_issued_transfers"] = {"gbs": g, "frac_of_link": g / link_peak, "bytes": R.copy_bytes,
                                        "note": "cudaMemcpyAsync waves on the copy stream, events around each wave"}
    # the prompt again with events around the grouped GEMM launches of every compute group
    if cfg.prefill_tokens and cfg.d_ff % 128 == 0 and cfg.batch * cfg.prefill_tokens > 8 and store != "q4slots":
        R.prepare(alpha, timing_prefill=True)
        ms_sum, n = 0.0, 0
        for ls in R.stack.layers:
            t = ls.layer.ffn_launch_times_ms()
            ms_sum += float(t.sum())
            n += len(t)
            ls.layer.ffn_time_ms()
            ls.layer.transfer_time_ms()
            ls.layer.enable_timing(False)
        T = cfg.batch * cfg.prefill_tokens
        pairs = T * (cfg.top_k + cfg.n_shared)
        flops = 6.0 * cfg.d_model * cfg.d_ff * pairs * n_layers
        tf = flops / (ms_sum * 1e-3) / 1e12
        rec["prefill_gemm"] = {"tokens": T, "token_expert_pairs_per_layer": pairs, "tflops": tf,
                               "frac_of_bf16_burst": tf / peaks.get("bf16_tflops", 1590.0),
                               "frac_of_bf16_sustained": tf / peaks.get("bf16_tflops_sustained", 1400.0),
                               "gemm_launch_pairs": n, "gemm_ms_per_layer": ms_sum / n_layers,
                               "note": "flops = 6 d_model d_ff per (token, expert) pair; time = CUDA events around the two "
                                       "GEMM launches of every compute group, transfers excluded"}
    R.close()
    # the same shape with every expert resident: the decode kernel in its HBM-bound regime
    Ra = Runner(torch, M, gen, cfg, alpha, cfg.n_experts, n_layers, K, W, store=store)
    Ra.timed_device(alpha)                                           # warm: the first pass fetches what the prompt did not
    _, _, st3, pl3 = Ra.timed_device(alpha, with_kernel_timing=True)
    a3 = ffn_launch_analysis(cfg, st3, pl3, hbm_peak, link_peak, expert_bytes=eb)
    rec["ffn_all_resident"] = a3["resident"] if a3 else None
    Ra.close()
    return rec


def timeline_record(torch, gen, cfg, alpha, C, n_layers, store, steps=24, warm=8):
    """Where a decode launch spends its time: the kernel stamps %globaltimer per CTA at entry, set-up done (plan
    seen), first tile landed, last tile done, partial sums added, (last CTA only: counter passed, output written),
    exit.  Stamps of the stack's last layer, microseconds after its first CTA entered, median and maximum over
    the CTAs, one row per decode step."""
    from paper_2602_11192_b200.workload import Stack
    st = Stack(cfg, alpha, C, n_layers=n_layers, store=store)
    lay = st.layers[-1].layer
    n_cta = lay.timeline_ctas()
    tr = torch.zeros((n_cta, 8), dtype=torch.int64, device="cuda")
    out = torch.empty((n_layers, cfg.batch, cfg.d_model), dtype=torch.int16, device="cuda")
    stats = torch.zeros((n_layers, 12), dtype=torch.int32, device="cuda")
    xs = [torch.from_numpy(st.hidden_bits("decode", s).view(np.int16)).cuda() for s in range(steps)]
    for s in range(warm):
        st.forward_all(xs[s], out, stats)
    torch.cuda.synchronize()
    lay.set_timeline(tr, n_cta * 64)
    rows = []
    for s in range(warm, steps):
        st.forward_all(xs[s], out, stats)
        torch.cuda.synchronize()
        t = tr.cpu().numpy().astype(np.int64)
        rel = (t - t[:, 0].min()) / 1e3
        live = [0, 1, 2, 3, 4, 7]                    # stamps every CTA writes
        rows.append({"misses": int(stats.cpu()[-1, 4]),
                     "median_us": [round(float(np.median(rel[:, i])), 2) for i in live],
                     "max_us": [round(float(rel[:, i].max()), 2) for i in range(8)]})
    st.close()
    return {"timeline": "decode FFN kernel, last of %d layers, %d slots, store %s" % (n_layers, C, store),
            "stamps_median": ["entry", "set-up done", "first tile landed", "last tile done", "partial sums added", "exit"],
            "stamps_max": ["entry", "set-up done", "first tile landed", "last tile done", "partial sums added",
                           "last CTA: counter passed", "last CTA: output written", "exit"],
            "steps": rows}


def run_ours(args):
    import torch
    import gen
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2602_11192_b200 import build as _build
    if rank == 0:
        _build.build()
    if dist is not None:
        dist.barrier()
    import paper_2602_11192_b200 as M

    cfg = gen.config_by_name(WORKLOAD)
    C = cfg.cache_slots[0] if args.slots is None else args.slots
    alpha0 = cfg.alphas[0] if args.alpha is None else args.alpha
    L = cfg.n_layers if args.layers is None else args.layers
    K, W = args.steps, args.warmup
    d = cfg.d_model
    B_e = cfg.expert_bytes if args.store != "q4slots" else M.melinoe_moe_expert_bytes_q4(cfg.d_model, cfg.d_ff)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_src = "measured" if "hbm_gbs" in peaks else "fallback"
    if args.timeline:
        print(json.dumps(timeline_record(torch, gen, cfg, alpha0, cfg.n_experts if args.slots is None else args.slots,
                                         args.layers or 2, args.store)), flush=True)
        return
    if args.shape is not None:
        rec = shape_record(torch, M, gen, args.shape, args.layers or 1, min(K, 64), W, hbm_peak, host_link_gbs(torch), peaks,
                           store=args.store)
        print(json.dumps({"shape_only": args.shape, "record": rec}), flush=True)
        return

    phase("building the stack: %d layers x %d experts x %.1f MB in pinned host memory" % (L, cfg.n_experts, B_e / 1e6))
    R = Runner(torch, M, gen, cfg, alpha0, C, L, K, W, store=args.store, dist=dist)

    gpu_index = local
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            gpu_index = int(vis.split(",")[local])
        except Exception:
            gpu_index = local
    sampler = ClockSampler(gpu_index)
    if rank == 0:
        sampler.start()
    phase("timed region x %d: %d warm-up + %d decode steps each, device-resident inputs" % (REPEATS, W, K))
    runs = []
    for _ in range(REPEATS):
        ms, launches, st, _ = R.timed_device(alpha0)
        runs.append(max_over_ranks(ms, dist, "cuda"))
    clocks = sampler.stop() if rank == 0 else None
    ms = statistics.median(runs)
    tokens = cfg.batch * K * world
    value = job_throughput(cfg.batch * K, world, ms)
    repeats = {"n": REPEATS, "tokens_per_s": [job_throughput(cfg.batch * K, world, m) for m in runs],
               "median": value, "best": job_throughput(cfg.batch * K, world, min(runs))}

    # ---- end to end: host buffers in, host buffers out, one synchronisation per decode step
    phase("end-to-end region x %d: host buffers, %.2f ms/step on the device path" % (REPEATS, ms / K))
    e2e_runs = [max_over_ranks(R.timed_e2e(alpha0), dist, "cuda") for _ in range(REPEATS)]
    e2e_ms = statistics.median(e2e_runs)
    e2e = {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT, "best": tokens / (min(e2e_runs) * 1e-3),
           "h2d_bytes_per_step": L * cfg.batch * d * 2,
           "d2h_bytes_per_step": L * (cfg.batch * d * 2 + 48),
           "note": "inputs from pinned host memory and outputs + statistics back to it inside the timed region, "
                   "one stream synchronisation per decode step; expert miss traffic (counted in hit_stats) is extra; "
                   "median of %d runs" % REPEATS}

    # ---- roofline of the dominant kernel (decode expert FFN): same region again with per-launch events
    phase("same region with per-launch events around the FFN kernel")
    link_peak = host_link_gbs(torch)
    _, _, st2, per_launch = R.timed_device(alpha0, with_kernel_timing=True)
    ana = ffn_launch_analysis(cfg, st2, per_launch, hbm_peak, link_peak, expert_bytes=B_e)
    res = ana["resident"] if ana and ana["resident"] else {"gbs": 0.0, "launches": 0, "avg_launch_us": None, "bytes_per_launch": 0.0}
    roofline = {"bound": "hbm", "kernel": "ffn_decode_kernel", "achieved": res["gbs"], "peak": hbm_peak, "unit": "GB/s",
                "frac": res["gbs"] / hbm_peak, "peak_source": peak_src,
                "traffic": (DRAM_TRAFFIC_PER_ALGORITHMIC_BYTE * res["bytes_per_launch"]) if DRAM_TRAFFIC_PER_ALGORITHMIC_BYTE else None,
                "launches": res["launches"], "avg_launch_us": res["avg_launch_us"], "bytes_per_launch": res["bytes_per_launch"],
                "all_launches": ana["all"] if ana else None,
                "target_frac": 0.70, "target_met": bool(res["gbs"] / hbm_peak >= 0.70),
                "note": "launches whose experts were all resident (HBM-bound): bytes = experts streamed x bytes per expert, "
                        "time = CUDA events around each launch; the launches that also fetched experts over the host link "
                        "are in miss_path, all launches together in all_launches"}
    fe = ana["fetching"] if ana else None
    miss_path = {"achieved_gbs": fe["link_gbs"] if fe else None, "peak_gbs": link_peak,
                 "frac": fe["frac_of_link"] if fe else None, "launches": fe["launches"] if fe else 0,
                 "avg_launch_us": fe["avg_launch_us"] if fe else None,
                 "note": "launches of the FFN kernel that read missed experts from pinned host memory themselves: expert "
                         "bytes over the link / whole launch time by CUDA events (the resident experts' compute runs on "
                         "other SMs meanwhile); peak = a 512 MiB pinned cudaMemcpyAsync measured in this run"}

    extra = {}
    if not args.no_extra and rank == 0 and world == 1:
        for a in cfg.alphas:
            if a == alpha0:
                continue
            phase("alpha=%g" % a)
            ms_a, _, st_a, _ = R.timed_device(a)
            extra["alpha=%g" % a] = dict(value=cfg.batch * K / (ms_a * 1e-3), **hit_summary(cfg, st_a, K, L))
        # the paper's other eviction policies on the same stream (its Table 13 compares transfers under
        # LRU and LFU): Definition C.1's discounted count, gamma = 1 (LFU) and gamma = 0.9
        for name, g in (("policy=lfu", 1.0), ("policy=count,gamma=0.9", 0.9)):
            phase(name)
            R.stack.set_policy("count", g)
            ms_p, _, st_p, _ = R.timed_device(alpha0)
            extra[name] = dict(value=cfg.batch * K / (ms_p * 1e-3), **hit_summary(cfg, st_p, K, L))
        R.stack.set_policy("lru")
        # cold start with and without a preload of every layer's Top-C of the sequence's router bias (the
        # stand-in for the paper's activation predictor): misses and time of the first decode tokens
        phase("cold start with and without preload")
        extra["preload"] = preload_record(torch, R, cfg, alpha0, C, L, min(64, W + K))
        R.close()
        # 4-bit host store (the paper keeps its experts in 4-bit form): a miss moves 3.76 times fewer bytes
        if cfg.d_ff % 64 == 0:
            Rq = Runner(torch, M, gen, cfg, alpha0, C, L, K, W, store="q4")
            qb = M.melinoe_moe_expert_bytes_q4(cfg.d_model, cfg.d_ff)
            for a in cfg.alphas[:2]:
                phase("4-bit host store, alpha=%g" % a)
                ms_q, _, st_q, _ = Rq.timed_device(a)
                extra["store=q4,alpha=%g" % a] = dict(value=cfg.batch * K / (ms_q * 1e-3), **hit_summary(cfg, st_q, K, L))
                extra["store=q4,alpha=%g" % a]["h2d_expert_bytes_per_step"] = float(st_q["misses"].sum()) * qb / K
            # the paper's own serving configuration: 4-bit experts and an LFU cache
            phase("4-bit host store with the LFU policy")
            Rq.stack.set_policy("count", 1.0)
            ms_q, _, st_q, _ = Rq.timed_device(alpha0)
            extra["store=q4,policy=lfu"] = dict(value=cfg.batch * K / (ms_q * 1e-3), **hit_summary(cfg, st_q, K, L))
            extra["store=q4,policy=lfu"]["h2d_expert_bytes_per_step"] = float(st_q["misses"].sum()) * qb / K
            Rq.close()
        # 4-bit cache slots (Appendix D.5, Table 12: at equal memory 4-bit experts let about 3.76 times as many stay
        # resident): the same number of slots, then the number of 4-bit slots that fit the bf16 slots' memory
        if cfg.d_model % 512 == 0:
            qb = M.melinoe_moe_expert_bytes_q4(cfg.d_model, cfg.d_ff)
            C_eq = int(min(cfg.n_experts, C * cfg.expert_bytes // qb))
            for name, Cq in (("slots=q4,same_count", C), ("slots=q4,equal_memory", C_eq)):
                phase("4-bit slots: %d per layer" % Cq)
                Rs = Runner(torch, M, gen, cfg, alpha0, Cq, L, K, W, store="q4slots")
                vals = []
                for _ in range(REPEATS):
                    ms_s, _, st_s, _ = Rs.timed_device(alpha0)
                    vals.append(cfg.batch * K / (ms_s * 1e-3))
                _, _, st_s2, pl_s = Rs.timed_device(alpha0, with_kernel_timing=True)
                ana_s = ffn_launch_analysis(cfg, st_s2, pl_s, hbm_peak, link_peak, expert_bytes=qb)
                med, best = med_best(vals)
                rec = {"value": med, "best": best, "cache_slots": Cq, "slot_bytes": qb, "slot_memory_bytes_per_layer": Cq * qb,
                       "bf16_slot_memory_bytes_per_layer": C * cfg.expert_bytes, **hit_summary(cfg, st_s, K, L)}
                rec["h2d_expert_bytes_per_step"] = float(st_s["misses"].sum()) * qb / K
                if ana_s and ana_s["resident"]:
                    r_ = ana_s["resident"]
                    rec["ffn_resident"] = {"launches": r_["launches"], "avg_launch_us": r_["avg_launch_us"], "gbs_4bit": r_["gbs"],
                                           "frac_of_hbm": r_["frac_of_hbm"],
                                           "bf16_equivalent_gbs": r_["gbs"] * cfg.expert_bytes / qb}
                if ana_s and ana_s["fetching"]:
                    rec["ffn_fetching"] = ana_s["fetching"]
                extra[name] = rec
                Rs.close()
        # everything resident (cache = all experts, warm): the hit path alone
        phase("all experts resident")
        Rf = Runner(torch, M, gen, cfg, alpha0, cfg.n_experts, L, K, W)
        vals = []
        for _ in range(REPEATS):
            ms_r, _, st_r, _ = Rf.timed_device(alpha0)
            vals.append(cfg.batch * K / (ms_r * 1e-3))
        _, _, st_r2, pl_r = Rf.timed_device(alpha0, with_kernel_timing=True)
        ana_r = ffn_launch_analysis(cfg, st_r2, pl_r, hbm_peak, link_peak)
        rr = ana_r["resident"] if ana_r and ana_r["resident"] else {"gbs": 0.0, "frac_of_hbm": 0.0, "launches": 0, "avg_launch_us": None}
        med, best = med_best(vals)
        extra["all_resident"] = {"value": med, "best": best, "ffn_gbs": rr["gbs"], "ffn_frac_of_hbm": rr["frac_of_hbm"],
                                 "ffn_launches": rr["launches"], "ffn_avg_launch_us": rr["avg_launch_us"],
                                 "us_per_layer": 1e6 / (med * L) * cfg.batch, **hit_summary(cfg, st_r, K, L)}
        Rf.close()
        # the other workload shapes at full width, fewer layers
        Ks = min(K, 64)
        for name, nl in (("mixtral", 2), ("phi35", 2), ("deepseek", 2)):
            phase("%s-shaped stack, %d layers" % (name, nl))
            extra["shape=" + name] = shape_record(torch, M, gen, name, nl, Ks, W, hbm_peak, link_peak, peaks)
    else:
        R.close()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        phase("CPU oracle on a sample of the same steps")
        cpu_baseline = cpu_oracle_sample(cfg, alpha0, C, L, W, K, budget_s=15.0)

    faulthandler.cancel_dump_traceback_later()
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": workload_config(cfg, alpha0, C, L),
            "clocks": clocks, "repeats": repeats, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "miss_path": miss_path, "cpu_baseline": cpu_baseline,
            "hit_stats": hit_summary(cfg, st, K, L), "other_runs": extra,
        }
        if args.layers is not None:
            line["config"]["reduced_layers"] = True
        if args.store != "bf16":
            line["config"]["store"] = args.store
        if args.slots is not None:
            line["config"]["slots_override"] = args.slots
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# --------------------------------------------------------------------------- CPU oracle legs

def oracle_layers(cfg, L):
    """Paper-layout weights of every layer as uint16 views, plus the router matrices."""
    import gen
    from paper_2602_11192_b200.workload import bits_of
    layers = []
    for l in range(L):
        wg, wu, wd = gen.fill_expert_store_fast(cfg.seed, l, cfg.n_experts + cfg.n_shared, cfg.d_model, cfg.d_ff)
        ws = [(bits_of(wg[e]), bits_of(wu[e]), bits_of(wd[e])) for e in range(cfg.n_experts + cfg.n_shared)]
        layers.append((ws, gen.router_weights(cfg.seed, l, cfg.n_experts, cfg.d_model), (wg, wu, wd)))
    return layers


def oracle_decode_steps(cfg, alpha, C, L, first_step, n_steps, max_seconds=None, layers=None):
    """Run the oracle over decode steps [first_step, first_step + n_steps) of all L layers, after
    replaying routing and cache decisions of the prompt and the earlier steps (cheap).  Returns
    (seconds spent in the timed steps, steps done)."""
    import gen
    import oracle
    if layers is None:
        layers = oracle_layers(cfg, L)
    caches = [oracle.ExpertCache(C, cfg.n_experts) for _ in range(L)]
    bias = [np.stack([gen.router_bias(cfg.seed, l, s, alpha, cfg.n_experts) for s in range(cfg.batch)]) for l in range(L)]
    dseq = np.arange(cfg.batch, dtype=np.int32)
    for l in range(L):
        if cfg.prefill_tokens:
            x = gen.hidden_states(cfg.seed, l, "prefill", 0, cfg.batch * cfg.prefill_tokens, cfg.d_model)
            pseq = np.repeat(dseq, cfg.prefill_tokens)
            caches[l].call(oracle.route(x, layers[l][1], cfg.top_k, bias[l], pseq)[0])
        for s in range(first_step):
            x = gen.hidden_states(cfg.seed, l, "decode", s, cfg.batch, cfg.d_model)
            caches[l].call(oracle.route(x, layers[l][1], cfg.top_k, bias[l], dseq)[0])
    xs = [[gen.hidden_states(cfg.seed, l, "decode", s, cfg.batch, cfg.d_model) for l in range(L)]
          for s in range(first_step, first_step + n_steps)]
    t0 = time.perf_counter()
    done = 0
    for s in range(n_steps):
        for l in range(L):
            oracle.layer_forward(xs[s][l], layers[l][1], layers[l][0], cfg.top_k, cfg.d_ff, caches[l], bias[l], dseq,
                                 cfg.n_shared)
        done += 1
        if max_seconds is not None and time.perf_counter() - t0 > max_seconds:
            break
    return time.perf_counter() - t0, done


def cpu_oracle_sample(cfg, alpha, C, L, W, K, budget_s):
    """The oracle on the timed decode steps and, where those take it less than the budget, on the steps
    of the same stream that follow them."""
    import oracle
    n = max(K, min(cfg.decode_steps - W, 512))
    secs, done = oracle_decode_steps(cfg, alpha, C, L, W, n, max_seconds=budget_s)
    return {"value": cfg.batch * done / secs, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": "%d decode steps of the same stream from the first timed one on (the %d timed steps first), all %d "
                      "layers each: %.0f s of CPU work" % (done, K, L, secs)}


def run_reference(args):
    import gen
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = gen.config_by_name(WORKLOAD)
    C = cfg.cache_slots[0]
    alpha0 = cfg.alphas[0] if args.alpha is None else args.alpha
    L = cfg.n_layers if args.layers is None else args.layers
    K, W = args.steps, args.warmup
    phase("reference arm: generating %d layers of weights" % L, 900)
    layers = oracle_layers(cfg, L)
    phase("reference arm: %d decode steps on the host cores" % K, 1500)
    oracle_decode_steps(cfg, alpha0, C, L, 0, min(W, 1), layers=layers)   # warm-up: page in, thread pool
    secs, done = oracle_decode_steps(cfg, alpha0, C, L, W, K, layers=layers)
    value = cfg.batch * done / secs
    sample = "every one of the %d decode steps through all %d layers on the host cores" % (done, L)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
        "warmup": W, "ms_per_step": 1e3 * secs / max(done, 1), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, alpha0, C, L),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    faulthandler.cancel_dump_traceback_later()
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
