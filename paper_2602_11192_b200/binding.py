"""ctypes binding with the same names as include/melinoe_moe.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

__all__ = [
    "MelinoeError", "Stats", "Request", "lib", "library_path", "STATUS_NAMES", "MoELayer",
    "melinoe_moe_expert_bytes", "melinoe_moe_pack_expert", "melinoe_moe_expert_bytes_q4",
    "melinoe_moe_pack_expert_q4", "melinoe_trace_miss_proxies", "ProxyConfig", "melinoe_launch_count",
    "melinoe_last_cuda_error", "melinoe_strerror", "EXPORTED_SYMBOLS",
]

HERE = os.path.dirname(os.path.abspath(__file__))

EXPORTED_SYMBOLS = [
    "melinoe_moe_create", "melinoe_moe_create_q4", "melinoe_moe_destroy", "melinoe_moe_expert_bytes", "melinoe_moe_pack_expert",
    "melinoe_moe_set_router", "melinoe_moe_register_host_experts", "melinoe_moe_register_shared_experts",
    "melinoe_moe_set_router_bias", "melinoe_moe_reserve", "melinoe_moe_forward", "melinoe_moe_forward_host",
    "melinoe_moe_reset_cache", "melinoe_moe_preload", "melinoe_moe_last_routing", "melinoe_moe_last_logits",
    "melinoe_moe_last_requests", "melinoe_moe_last_gather", "melinoe_moe_cache_state",
    "melinoe_moe_enable_timing", "melinoe_moe_ffn_time_ms", "melinoe_moe_set_trace", "melinoe_moe_trace_count",
    "melinoe_moe_trace_record_bytes", "melinoe_moe_set_timeline", "melinoe_moe_timeline_ctas", "melinoe_allocate_slots",
    "melinoe_moe_transfer_time_ms", "melinoe_moe_forward_static", "melinoe_moe_static_scratch_bytes",
    "melinoe_moe_last_call_used_gemm", "melinoe_moe_set_policy", "melinoe_moe_cache_counts", "melinoe_moe_expert_bytes_q4",
    "melinoe_moe_pack_expert_q4", "melinoe_moe_register_host_experts_q4", "melinoe_trace_miss_proxies", "melinoe_launch_count",
    "melinoe_last_cuda_error", "melinoe_strerror", "melinoe_moe_ffn_launch_times_ms", "melinoe_debug_fail_host_copy",
    "melinoe_moe_preload_pooled",
]

STATUS_NAMES = {0: "OK", 1: "INVALID", 2: "STATE", 3: "CUDA", 4: "NOMEM", 5: "TIMEOUT", 6: "UNSUPPORTED"}


class MelinoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s: %s (%d)" % (where, melinoe_strerror(status), status))


class Stats(C.Structure):
    _fields_ = [("status", C.c_int32), ("n_tokens", C.c_int32), ("n_distinct", C.c_int32),
                ("hits", C.c_int32), ("misses", C.c_int32), ("evictions", C.c_int32),
                ("groups", C.c_int32), ("reserved", C.c_int32),
                ("bytes_h2d", C.c_uint64), ("call_no", C.c_uint64)]


class Request(C.Structure):
    _fields_ = [("expert", C.c_int32), ("slot", C.c_int32), ("hit", C.c_int32), ("evicted", C.c_int32)]


def library_path() -> str:
    return os.path.join(HERE, "libmelinoe_moe.so")


_lib = None


def lib():
    """The loaded shared library.  Raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise ImportError("libmelinoe_moe.so is not built: run `python -m paper_2602_11192_b200.build` "
                          "(there is no fallback implementation)")
    L = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
    L.melinoe_moe_create.argtypes = [i32, i32, i32, i32, i32, C.POINTER(vp)]
    L.melinoe_moe_create_q4.argtypes = [i32, i32, i32, i32, i32, C.POINTER(vp)]
    L.melinoe_moe_destroy.argtypes = [vp]
    L.melinoe_moe_expert_bytes.argtypes = [i32, i32]
    L.melinoe_moe_expert_bytes.restype = sz
    L.melinoe_moe_pack_expert.argtypes = [i32, i32, vp, vp, vp, vp]
    L.melinoe_moe_expert_bytes_q4.argtypes = [i32, i32]
    L.melinoe_moe_expert_bytes_q4.restype = sz
    L.melinoe_moe_pack_expert_q4.argtypes = [i32, i32, vp, vp, vp, vp]
    L.melinoe_moe_set_router.argtypes = [vp, vp]
    L.melinoe_moe_register_host_experts.argtypes = [vp, C.POINTER(vp), sz]
    L.melinoe_moe_register_host_experts_q4.argtypes = [vp, C.POINTER(vp), sz]
    L.melinoe_moe_register_shared_experts.argtypes = [vp, i32, C.POINTER(vp)]
    L.melinoe_moe_set_router_bias.argtypes = [vp, vp, vp, i32]
    L.melinoe_moe_reserve.argtypes = [vp, i32]
    L.melinoe_moe_forward.argtypes = [vp, vp, vp, i32, vp, vp]
    L.melinoe_moe_forward_host.argtypes = [vp, vp, vp, i32, vp, vp]
    L.melinoe_moe_forward_static.argtypes = [vp, vp, vp, i32, vp, vp]
    L.melinoe_moe_static_scratch_bytes.restype = sz
    L.melinoe_moe_last_call_used_gemm.argtypes = [vp]
    L.melinoe_moe_reset_cache.argtypes = [vp]
    L.melinoe_trace_miss_proxies.argtypes = [vp, vp, i32, i32, i32, i32, vp, i32, vp, vp]
    L.melinoe_moe_set_policy.argtypes = [vp, i32, C.c_float]
    L.melinoe_moe_cache_counts.argtypes = [vp, vp]
    L.melinoe_moe_preload.argtypes = [vp, vp, i32]
    L.melinoe_moe_preload_pooled.argtypes = [vp, vp, i32, i32]
    L.melinoe_moe_last_routing.argtypes = [vp, vp, vp]
    L.melinoe_moe_last_logits.argtypes = [vp, vp]
    L.melinoe_moe_last_requests.argtypes = [vp, vp, C.POINTER(i32)]
    L.melinoe_moe_last_gather.argtypes = [vp, vp, vp, vp]
    L.melinoe_moe_cache_state.argtypes = [vp, vp, vp]
    L.melinoe_moe_enable_timing.argtypes = [vp, i32]
    L.melinoe_moe_ffn_time_ms.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    L.melinoe_moe_transfer_time_ms.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]
    L.melinoe_moe_ffn_launch_times_ms.argtypes = [vp, vp, i32, C.POINTER(i32)]
    L.melinoe_debug_fail_host_copy.argtypes = [i32]
    L.melinoe_moe_set_trace.argtypes = [vp, vp, sz, i32]
    L.melinoe_moe_trace_count.argtypes = [vp]
    L.melinoe_moe_trace_count.restype = C.c_int64
    L.melinoe_moe_trace_record_bytes.argtypes = [vp, i32]
    L.melinoe_moe_trace_record_bytes.restype = sz
    L.melinoe_moe_set_timeline.argtypes = [vp, vp, sz]
    L.melinoe_moe_timeline_ctas.argtypes = [vp]
    L.melinoe_allocate_slots.argtypes = [vp, i32, i32, i32, C.c_int64, vp]
    L.melinoe_launch_count.restype = C.c_int64
    L.melinoe_last_cuda_error.restype = i32
    L.melinoe_strerror.argtypes = [i32]
    L.melinoe_strerror.restype = C.c_char_p
    _lib = L
    return L


def melinoe_strerror(status: int) -> str:
    try:
        return lib().melinoe_strerror(int(status)).decode()
    except Exception:
        return STATUS_NAMES.get(int(status), "?")


def melinoe_moe_expert_bytes(d_model: int, d_ff: int) -> int:
    return int(lib().melinoe_moe_expert_bytes(d_model, d_ff))


def melinoe_moe_pack_expert(d_model: int, d_ff: int, w_gate_ptr: int, w_up_ptr: int, w_down_ptr: int,
                            blob_ptr: int) -> None:
    rc = lib().melinoe_moe_pack_expert(d_model, d_ff, w_gate_ptr, w_up_ptr, w_down_ptr, blob_ptr)
    if rc:
        raise MelinoeError(rc, "melinoe_moe_pack_expert")


def melinoe_moe_expert_bytes_q4(d_model: int, d_ff: int) -> int:
    return int(lib().melinoe_moe_expert_bytes_q4(d_model, d_ff))


def melinoe_moe_pack_expert_q4(d_model: int, d_ff: int, w_gate_ptr: int, w_up_ptr: int, w_down_ptr: int,
                               blob_ptr: int) -> None:
    rc = lib().melinoe_moe_pack_expert_q4(d_model, d_ff, w_gate_ptr, w_up_ptr, w_down_ptr, blob_ptr)
    if rc:
        raise MelinoeError(rc, "melinoe_moe_pack_expert_q4")


class ProxyConfig(C.Structure):
    _fields_ = [("layer", C.c_int32), ("cache_slots", C.c_int32), ("gamma", C.c_double)]


def melinoe_trace_miss_proxies(stream: int, trace_dev, n_layers: int, n_tokens: int, top_k: int, n_experts: int,
                               configs_dev, n_configs: int, soft_mean_dev, hard_total_dev) -> None:
    rc = lib().melinoe_trace_miss_proxies(stream, _ptr(trace_dev), n_layers, n_tokens, top_k, n_experts,
                                          _ptr(configs_dev), n_configs, _ptr(soft_mean_dev), _ptr(hard_total_dev))
    if rc:
        raise MelinoeError(rc, "melinoe_trace_miss_proxies")


def melinoe_launch_count() -> int:
    return int(lib().melinoe_launch_count())


def melinoe_last_cuda_error() -> int:
    return int(lib().melinoe_last_cuda_error())


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return int(t.data_ptr())
    return int(t.ctypes.data)


class MoELayer:
    """One handle (= one MoE layer).  Methods mirror the C entry points one to one."""

    def __init__(self, d_model: int, d_ff: int, n_experts: int, top_k: int, cache_slots: int, slots: str = "bf16"):
        self.d_model, self.d_ff, self.n_experts, self.top_k, self.cache_slots = (
            int(d_model), int(d_ff), int(n_experts), int(top_k), int(cache_slots))
        self._h = C.c_void_p()
        self._keep = {}
        assert slots in ("bf16", "q4")
        self.slots = slots
        create = lib().melinoe_moe_create if slots == "bf16" else lib().melinoe_moe_create_q4
        rc = create(d_model, d_ff, n_experts, top_k, cache_slots, C.byref(self._h))
        if rc:
            self._h = C.c_void_p()
            raise MelinoeError(rc, "melinoe_moe_create" if slots == "bf16" else "melinoe_moe_create_q4")

    # -- lifetime
    def destroy(self) -> None:
        if getattr(self, "_h", None) and self._h.value:
            lib().melinoe_moe_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def _ck(self, rc: int, where: str) -> None:
        if rc:
            raise MelinoeError(rc, where)

    # -- configuration
    def set_router(self, w_router_dev) -> None:
        self._keep["router"] = w_router_dev
        self._ck(lib().melinoe_moe_set_router(self._h, _ptr(w_router_dev)), "melinoe_moe_set_router")

    def register_host_experts(self, expert_host_ptrs: Sequence[int], bytes_per_expert: int, keep=None) -> None:
        arr = (C.c_void_p * len(expert_host_ptrs))(*[int(p) for p in expert_host_ptrs])
        self._keep["experts"] = keep
        self._ck(lib().melinoe_moe_register_host_experts(self._h, arr, bytes_per_expert),
                 "melinoe_moe_register_host_experts")

    def register_host_experts_q4(self, expert_host_ptrs: Sequence[int], bytes_per_expert: int, keep=None) -> None:
        arr = (C.c_void_p * len(expert_host_ptrs))(*[int(p) for p in expert_host_ptrs])
        self._keep["experts"] = keep
        self._ck(lib().melinoe_moe_register_host_experts_q4(self._h, arr, bytes_per_expert),
                 "melinoe_moe_register_host_experts_q4")

    def register_shared_experts(self, expert_dev_ptrs: Sequence[int], keep=None) -> None:
        n = len(expert_dev_ptrs)
        arr = (C.c_void_p * max(n, 1))(*[int(p) for p in expert_dev_ptrs])
        self._keep["shared"] = keep
        self._ck(lib().melinoe_moe_register_shared_experts(self._h, n, arr), "melinoe_moe_register_shared_experts")

    def set_router_bias(self, seq_bias_dev, token_seq_dev, n_seq: int) -> None:
        self._keep["bias"] = (seq_bias_dev, token_seq_dev)
        self._ck(lib().melinoe_moe_set_router_bias(self._h, _ptr(seq_bias_dev), _ptr(token_seq_dev), n_seq),
                 "melinoe_moe_set_router_bias")

    def reserve(self, max_tokens: int) -> None:
        self._ck(lib().melinoe_moe_reserve(self._h, max_tokens), "melinoe_moe_reserve")

    # -- the hot path
    def forward(self, stream: int, hidden_dev, n_tokens: int, out_dev, stats_dev=None) -> None:
        self._ck(lib().melinoe_moe_forward(self._h, stream, _ptr(hidden_dev), n_tokens, _ptr(out_dev),
                                           _ptr(stats_dev)), "melinoe_moe_forward")

    def forward_static(self, stream: int, hidden_dev, n_tokens: int, out_dev, stats_dev=None) -> None:
        """melinoe_moe_forward_static: the same call on the library's static scratch (allocates nothing)."""
        self._ck(lib().melinoe_moe_forward_static(self._h, stream, _ptr(hidden_dev), n_tokens, _ptr(out_dev),
                                                  _ptr(stats_dev)), "melinoe_moe_forward_static")

    def forward_host(self, stream: int, hidden_host, n_tokens: int, out_host, stats_host=None) -> None:
        self._ck(lib().melinoe_moe_forward_host(self._h, stream, _ptr(hidden_host), n_tokens, _ptr(out_host),
                                                _ptr(stats_host)), "melinoe_moe_forward_host")

    def reset_cache(self) -> None:
        self._ck(lib().melinoe_moe_reset_cache(self._h), "melinoe_moe_reset_cache")

    def set_policy(self, policy: str, gamma: float = 0.0) -> None:
        """Eviction policy: "lru" (default) or "count" (Definition C.1's discounted count; gamma = 1 is LFU)."""
        code = {"lru": 0, "count": 1}[policy]
        self._ck(lib().melinoe_moe_set_policy(self._h, code, C.c_float(gamma)), "melinoe_moe_set_policy")

    def cache_counts(self, n_experts: int):
        import numpy as np
        out = np.empty(n_experts, dtype=np.float32)
        self._ck(lib().melinoe_moe_cache_counts(self._h, out.ctypes.data), "melinoe_moe_cache_counts")
        return out

    def preload(self, expert_ids) -> None:
        import numpy as np
        ids = np.ascontiguousarray(expert_ids, dtype=np.int32)
        self._ck(lib().melinoe_moe_preload(self._h, ids.ctypes.data, ids.size), "melinoe_moe_preload")

    def preload_pooled(self, lists) -> None:
        """lists [n_seq][per_seq]: every sequence's own predicted set; the most-voted experts are preloaded."""
        import numpy as np
        a = np.ascontiguousarray(lists, dtype=np.int32)
        assert a.ndim == 2
        self._ck(lib().melinoe_moe_preload_pooled(self._h, a.ctypes.data, a.shape[0], a.shape[1]),
                 "melinoe_moe_preload_pooled")

    # -- inspection (blocking)
    def last_routing(self, n_tokens: int):
        import numpy as np
        idx = np.empty((n_tokens, self.top_k), np.int32)
        gate = np.empty((n_tokens, self.top_k), np.float32)
        self._ck(lib().melinoe_moe_last_routing(self._h, idx.ctypes.data, gate.ctypes.data), "melinoe_moe_last_routing")
        return idx, gate

    def last_logits(self, n_tokens: int):
        import numpy as np
        lg = np.empty((n_tokens, self.n_experts), np.float32)
        self._ck(lib().melinoe_moe_last_logits(self._h, lg.ctypes.data), "melinoe_moe_last_logits")
        return lg

    def last_requests(self):
        import numpy as np
        buf = np.empty((self.n_experts, 4), np.int32)
        n = C.c_int(0)
        self._ck(lib().melinoe_moe_last_requests(self._h, buf.ctypes.data, C.byref(n)), "melinoe_moe_last_requests")
        return buf[: n.value].copy()

    def last_gather(self, n_tokens: int):
        import numpy as np
        counts = np.empty(self.n_experts, np.int32)
        offsets = np.empty(self.n_experts + 1, np.int32)
        perm = np.empty(n_tokens * self.top_k, np.int32)
        self._ck(lib().melinoe_moe_last_gather(self._h, counts.ctypes.data, offsets.ctypes.data, perm.ctypes.data),
                 "melinoe_moe_last_gather")
        return counts, offsets, perm

    def cache_state(self):
        import numpy as np
        eos = np.empty(self.cache_slots, np.int32)
        tot = np.empty(3, np.uint64)
        self._ck(lib().melinoe_moe_cache_state(self._h, eos.ctypes.data, tot.ctypes.data), "melinoe_moe_cache_state")
        return eos, {"hits": int(tot[0]), "misses": int(tot[1]), "evictions": int(tot[2])}

    def enable_timing(self, enable: bool = True) -> None:
        self._ck(lib().melinoe_moe_enable_timing(self._h, int(enable)), "melinoe_moe_enable_timing")

    def last_call_used_gemm(self) -> bool:
        return bool(lib().melinoe_moe_last_call_used_gemm(self._h))

    def ffn_launch_times_ms(self, capacity: int = 65536):
        """Per-launch times (ms) of the timed FFN launches since the last ffn_time_ms(), in launch order."""
        import numpy as np
        buf = np.empty(capacity, np.float32)
        n = C.c_int(0)
        self._ck(lib().melinoe_moe_ffn_launch_times_ms(self._h, buf.ctypes.data, capacity, C.byref(n)),
                 "melinoe_moe_ffn_launch_times_ms")
        return buf[: min(n.value, capacity)].copy()

    def transfer_time_ms(self):
        ms = C.c_double(0.0)
        nb = C.c_uint64(0)
        self._ck(lib().melinoe_moe_transfer_time_ms(self._h, C.byref(ms), C.byref(nb)), "melinoe_moe_transfer_time_ms")
        return ms.value, nb.value

    def set_timeline(self, trace_dev, n_bytes: int) -> None:
        self._keep["timeline"] = trace_dev
        self._ck(lib().melinoe_moe_set_timeline(self._h, _ptr(trace_dev), n_bytes), "melinoe_moe_set_timeline")

    def timeline_ctas(self) -> int:
        return int(lib().melinoe_moe_timeline_ctas(self._h))

    def trace_record_bytes(self, max_tokens: int) -> int:
        return int(lib().melinoe_moe_trace_record_bytes(self._h, max_tokens))

    def set_trace(self, trace_buf, n_bytes: int, max_tokens: int) -> None:
        """Request trace: one record per forward call into trace_buf (a ring of records), in stream order."""
        self._keep["trace"] = trace_buf
        self._ck(lib().melinoe_moe_set_trace(self._h, _ptr(trace_buf), n_bytes, max_tokens), "melinoe_moe_set_trace")

    def trace_count(self) -> int:
        return int(lib().melinoe_moe_trace_count(self._h))

    def ffn_time_ms(self):
        ms = C.c_double(0.0)
        n = C.c_int64(0)
        self._ck(lib().melinoe_moe_ffn_time_ms(self._h, C.byref(ms), C.byref(n)), "melinoe_moe_ffn_time_ms")
        return ms.value, n.value
