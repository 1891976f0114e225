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

# dram__bytes_read.sum + dram__bytes_write.sum of one ffn_stream_kernel launch divided by the launch's
# algorithmic bytes (8 experts x 12.58 MB), from the ncu capture summarised in
# profiles/ffn_stream_kernel_olmoe_decode.md; traffic grows in proportion to the experts streamed.
DRAM_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.03

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

    def barrier():
        if dist is not None:
            dist.barrier()

    from paper_2602_11192_b200 import build as _build
    if rank == 0:
        _build.build()
    barrier()
    import paper_2602_11192_b200 as M
    from paper_2602_11192_b200.workload import Stack, stats_rows

    cfg = gen.config_by_name(WORKLOAD)
    C = cfg.cache_slots[0]
    alpha0 = cfg.alphas[0] if args.alpha is None else args.alpha
    L = cfg.n_layers if args.layers is None else args.layers
    K, W = args.steps, args.warmup
    d = cfg.d_model
    B_e = cfg.expert_bytes

    phase("building the stack: %d layers x %d experts x %.1f MB in pinned host memory" % (L, cfg.n_experts, B_e / 1e6))
    stack = Stack(cfg, alpha0, C, n_layers=L)
    n_steps = W + K
    # decode inputs for every step, on the device and in pinned host memory
    dec = np.stack([stack.hidden_bits("decode", s) for s in range(n_steps)])          # [S][L][B][d]
    dec_host = torch.from_numpy(dec.view(np.int16)).pin_memory()
    dec_dev = dec_host.cuda()
    pre_dev = None
    if cfg.prefill_tokens:
        pre_dev = torch.from_numpy(stack.hidden_bits("prefill", 0).view(np.int16)).cuda()
        pre_out = torch.empty_like(pre_dev)
    out_dev = torch.empty((L, cfg.batch, d), dtype=torch.int16, device="cuda")
    out_host = torch.empty((L, cfg.batch, d), dtype=torch.int16).pin_memory()
    stats_dev = torch.zeros((n_steps, L, 12), dtype=torch.int32, device="cuda")
    stats_host = torch.zeros((L, 12), dtype=torch.int32).pin_memory()

    def prepare(alpha):
        """Cold start, prompt, then the warm-up decode steps."""
        if alpha != stack.alpha:
            stack.alpha = alpha
            stack.bias = [np.stack([gen.router_bias(cfg.seed, l, s, alpha, cfg.n_experts) for s in range(cfg.batch)])
                          for l in range(L)]
        stack.reset()
        if pre_dev is not None:
            stack.set_phase("prefill")
            stack.forward_all(pre_dev, pre_out, None)
        stack.set_phase("decode")
        torch.cuda.synchronize()

    copy_acc = [0.0, 0.0]   # copy-stream ms and bytes of the most recent run with kernel timing

    def host_link_gbs():
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
        return best

    def timed_device(alpha, with_kernel_timing=False):
        prepare(alpha)
        stats_dev.zero_()
        for s in range(W):
            stack.forward_all(dec_dev[s], out_dev, stats_dev[s])
        torch.cuda.synchronize()
        if with_kernel_timing:
            for ls in stack.layers:
                ls.layer.enable_timing(True)
        barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = M.melinoe_launch_count()
        e0.record()
        for s in range(W, W + K):
            stack.forward_all(dec_dev[s], out_dev, stats_dev[s])
        e1.record()
        torch.cuda.synchronize()
        barrier()
        ms = e0.elapsed_time(e1)
        launches = M.melinoe_launch_count() - n0
        ffn_ms, ffn_n = 0.0, 0
        copy_acc[0] = copy_acc[1] = 0.0
        if with_kernel_timing:
            for ls in stack.layers:
                a, b = ls.layer.ffn_time_ms()
                ffn_ms += a
                ffn_n += b
                cm, cb = ls.layer.transfer_time_ms()
                copy_acc[0] += cm
                copy_acc[1] += cb
                ls.layer.enable_timing(False)
        st = stats_rows(stats_dev[W:W + K])
        if int(st["status"].max()) != 0:
            raise SystemExit("device-side status %d in the timed region" % int(st["status"].max()))
        return ms, launches, st, ffn_ms, ffn_n

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
    phase("timed region: %d warm-up + %d decode steps, device-resident inputs" % (W, K))
    ms, launches, st, _, _ = timed_device(alpha0)
    clocks = sampler.stop() if rank == 0 else None
    ms = max_over_ranks(ms, dist, "cuda")
    tokens = cfg.batch * K * world
    value = job_throughput(cfg.batch * K, world, ms)

    # ---- end to end: host buffers in, host buffers out, one synchronisation per decode step
    phase("end-to-end region: host buffers, %.1f ms/step on the device path" % (ms / K))
    prepare(alpha0)
    s_ptr = torch.cuda.current_stream()
    for s in range(W):
        stack.forward_all_host(dec_host[s], out_host, stats_host)
        s_ptr.synchronize()
    barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(W, W + K):
        stack.forward_all_host(dec_host[s], out_host, stats_host)
        s_ptr.synchronize()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
    e2e = {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": L * cfg.batch * d * 2,
           "d2h_bytes_per_step": L * (cfg.batch * d * 2 + 48),
           "note": "inputs from pinned host memory and outputs + statistics back to it inside the timed region, "
                   "one stream synchronisation per decode step; expert miss traffic (counted in hit_stats) is extra"}

    # ---- roofline of the dominant kernel (streaming expert FFN): same region again with per-launch events
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_src = "measured" if "hbm_gbs" in peaks else "fallback"
    phase("same region with per-launch events around the FFN kernel")
    _, _, st2, ffn_ms, ffn_n = timed_device(alpha0, with_kernel_timing=True)
    ffn_bytes = float((st2["n_distinct"].astype(np.int64) + cfg.n_shared).sum()) * B_e
    achieved = ffn_bytes / (ffn_ms * 1e-3) / 1e9 if ffn_ms > 0 else 0.0
    link_peak = host_link_gbs()
    miss_path = {"achieved_gbs": (copy_acc[1] / (copy_acc[0] * 1e-3) / 1e9) if copy_acc[0] > 0 else None,
                 "peak_gbs": link_peak, "bytes": copy_acc[1], "copy_stream_ms": copy_acc[0],
                 "note": "expert bytes moved by cudaMemcpyAsync from pinned host memory / time between events on the "
                         "copy stream around each wave of transfers; peak = a 512 MiB pinned copy measured in this run"}
    if miss_path["achieved_gbs"]:
        miss_path["frac"] = miss_path["achieved_gbs"] / link_peak
    roofline = {"bound": "hbm", "kernel": "ffn_stream_kernel", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                "frac": achieved / hbm_peak, "peak_source": peak_src,
                "traffic": DRAM_TRAFFIC_PER_ALGORITHMIC_BYTE * ffn_bytes / max(ffn_n, 1),
                "launches": int(ffn_n), "avg_launch_us": 1e3 * ffn_ms / max(ffn_n, 1),
                "bytes_per_launch": ffn_bytes / max(ffn_n, 1),
                "note": "bytes = experts streamed x bytes per expert; launches that found no missed expert to "
                        "compute are included in the time"}

    def hit_summary(s):
        h, m = int(s["hits"].sum()), int(s["misses"].sum())
        return {"hit_rate": h / max(h + m, 1), "misses_per_layer_per_token": m / (K * L * cfg.batch),
                "h2d_expert_bytes_per_step": m * B_e / K}

    extra = {}
    if not args.no_extra and rank == 0 and world == 1:
        for a in cfg.alphas:
            if a == alpha0:
                continue
            phase("alpha=%g" % a)
            ms_a, _, st_a, _, _ = timed_device(a)
            extra["alpha=%g" % a] = dict(value=cfg.batch * K / (ms_a * 1e-3), **hit_summary(st_a))
        # the paper's other eviction policies on the same stream (its Table 13 compares transfers under
        # LRU and LFU): Definition C.1's discounted count, gamma = 1 (LFU) and gamma = 0.9.  These runs
        # plan with the general kernels, so their tokens/s also carries that difference.
        for name, g in (("policy=lfu", 1.0), ("policy=count,gamma=0.9", 0.9)):
            phase(name)
            stack.set_policy("count", g)
            ms_p, _, st_p, _, _ = timed_device(alpha0)
            extra[name] = dict(value=cfg.batch * K / (ms_p * 1e-3), **hit_summary(st_p))
        stack.set_policy("lru")
        # 4-bit host store (the paper keeps its experts in 4-bit form): a miss moves 3.76 times fewer
        # bytes; slots and compute stay bf16, computing with the dequantised weights
        if cfg.d_ff % 64 == 0:
            stack.close()
            stack = Stack(cfg, alpha0, C, n_layers=L, store="q4")
            for a in cfg.alphas[:2]:
                phase("4-bit host store, alpha=%g" % a)
                ms_q, _, st_q, _, _ = timed_device(a)
                extra["store=q4,alpha=%g" % a] = dict(value=cfg.batch * K / (ms_q * 1e-3), **hit_summary(st_q))
                extra["store=q4,alpha=%g" % a]["h2d_expert_bytes_per_step"] = (
                    float(st_q["misses"].sum()) * M.melinoe_moe_expert_bytes_q4(cfg.d_model, cfg.d_ff) / K)
            # the paper's own serving configuration: 4-bit experts and an LFU cache
            phase("4-bit host store with the LFU policy")
            stack.set_policy("count", 1.0)
            ms_q, _, st_q, _, _ = timed_device(alpha0)
            extra["store=q4,policy=lfu"] = dict(value=cfg.batch * K / (ms_q * 1e-3), **hit_summary(st_q))
            extra["store=q4,policy=lfu"]["h2d_expert_bytes_per_step"] = (
                float(st_q["misses"].sum()) * M.melinoe_moe_expert_bytes_q4(cfg.d_model, cfg.d_ff) / K)
            stack.set_policy("lru")
        # everything resident (cache = all experts, warm): the FFN kernel without the miss path
        phase("all experts resident")
        stack.close()
        full = Stack(cfg, alpha0, cfg.n_experts, n_layers=L)
        stack = full
        ms_r, _, _, _, _ = timed_device(alpha0)                    # throughput: no per-launch events
        _, _, st_r, ffn_ms_r, ffn_n_r = timed_device(alpha0, with_kernel_timing=True)
        by_r = float(st_r["n_distinct"].astype(np.int64).sum()) * B_e
        extra["all_resident"] = {"value": cfg.batch * K / (ms_r * 1e-3), "ffn_gbs": by_r / (ffn_ms_r * 1e-3) / 1e9,
                                 "ffn_frac_of_hbm": by_r / (ffn_ms_r * 1e-3) / 1e9 / hbm_peak,
                                 "ffn_launches": int(ffn_n_r), **hit_summary(st_r)}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        phase("CPU oracle on a sample of the same steps")
        cpu_baseline = cpu_oracle_sample(cfg, alpha0, C, L, W, K, budget_s=15.0)

    stack.close()
    faulthandler.cancel_dump_traceback_later()
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": workload_config(cfg, alpha0, C, L),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "miss_path": miss_path, "cpu_baseline": cpu_baseline,
            "hit_stats": hit_summary(st), "other_runs": extra,
        }
        if args.layers is not None:
            line["config"]["reduced_layers"] = True
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
    import oracle
    secs, done = oracle_decode_steps(cfg, alpha, C, L, W, K, max_seconds=budget_s)
    return {"value": cfg.batch * done / secs, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": "the first %d of the %d timed decode steps, all %d layers each (about %.0f s of CPU work)"
                      % (done, K, L, secs)}


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
