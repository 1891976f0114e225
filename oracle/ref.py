"""ctypes front end of the C oracle (numpy in, numpy out).

bf16 tensors are uint16 bit patterns.  Expert matrices are in the paper's shapes (Eq. 3):
W_g [F][d], W_u [F][d], W_d [d][F].
"""
from __future__ import annotations

import ctypes as C
from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

__all__ = ["pool_prefetch", "threads", "logits", "topk", "route", "gather", "quantize_q4", "dequantize_q4", "miss_proxies", "ExpertCache", "ffn_combine", "layer_forward"]

_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = C.CDLL(_build.build())
        lib.moe_oracle_threads.restype = C.c_int
        lib.moe_oracle_cache_create.restype = C.c_void_p
        lib.moe_oracle_cache_create.argtypes = [C.c_int, C.c_int]
        lib.moe_oracle_cache_destroy.argtypes = [C.c_void_p]
        lib.moe_oracle_cache_reset.argtypes = [C.c_void_p]
        lib.moe_oracle_cache_call.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        lib.moe_oracle_cache_call.restype = C.c_int
        lib.moe_oracle_cache_state.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.moe_oracle_cache_set_policy.argtypes = [C.c_void_p, C.c_int, C.c_float]
        lib.moe_oracle_cache_set_policy.restype = C.c_int
        lib.moe_oracle_cache_preload.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        lib.moe_oracle_cache_preload.restype = C.c_int
        lib.moe_oracle_cache_counts.argtypes = [C.c_void_p, C.c_void_p]
        lib.moe_oracle_pool_prefetch.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p]
        lib.moe_oracle_pool_prefetch.restype = C.c_int
        lib.moe_oracle_logits.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_int, C.c_int, C.c_int, C.c_void_p]
        lib.moe_oracle_topk.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        lib.moe_oracle_gather.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.moe_oracle_ffn_combine.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                               C.c_void_p, C.c_int, C.c_void_p]
        lib.moe_oracle_quantize_q4.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        lib.moe_oracle_dequantize_q4.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 tensors are passed as uint16 bit patterns"
    return a


def pool_prefetch(lists, n_experts: int, cache_slots: int) -> np.ndarray:
    """Pooled prefetch set of a batch (Section 4.3, batch size): lists [n_seq][per_seq] of every
    sequence's predicted experts -> the cache_slots most-voted experts, in load order."""
    a = np.ascontiguousarray(lists, dtype=np.int32)
    assert a.ndim == 2
    out = np.empty(max(cache_slots, 1), dtype=np.int32)
    n = _L().moe_oracle_pool_prefetch(_p(a), a.shape[0], a.shape[1], n_experts, cache_slots, _p(out))
    if n < 0:
        raise ValueError("expert index out of range")
    return out[:n].copy()


def threads() -> int:
    return int(_L().moe_oracle_threads())


def logits(x, w_r, bias=None, token_seq=None) -> np.ndarray:
    """fp32 router logits [T][E] in the oracle's fixed summation order (Eq. 1 argument)."""
    x = _u16(x); w_r = _u16(w_r)
    T, d = x.shape
    E = w_r.shape[0]
    assert w_r.shape[1] == d
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32).reshape(-1, E)
    ts = None if token_seq is None else np.ascontiguousarray(token_seq, dtype=np.int32)
    out = np.empty((T, E), dtype=np.float32)
    rc = _L().moe_oracle_logits(_p(x), _p(w_r), _p(b), _p(ts), T, d, E, _p(out))
    if rc:
        raise ValueError("moe_oracle_logits rc=%d" % rc)
    return out


def topk(lg: np.ndarray, k: int, raw_softmax: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    lg = np.ascontiguousarray(lg, dtype=np.float32)
    T, E = lg.shape
    idx = np.empty((T, k), dtype=np.int32)
    gate = np.empty((T, k), dtype=np.float64)
    rc = _L().moe_oracle_topk(_p(lg), T, E, k, int(raw_softmax), _p(idx), _p(gate))
    if rc:
        raise ValueError("moe_oracle_topk rc=%d" % rc)
    return idx, gate


def route(x, w_r, k, bias=None, token_seq=None):
    """(idx [T][k] int32, gate [T][k] fp64, logits [T][E] fp32)."""
    lg = logits(x, w_r, bias, token_seq)
    idx, gate = topk(lg, k)
    return idx, gate, lg


def gather(idx: np.ndarray, n_experts: int):
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    T, k = idx.shape
    counts = np.empty(n_experts, dtype=np.int32)
    offsets = np.empty(n_experts + 1, dtype=np.int32)
    perm = np.empty(T * k, dtype=np.int32)
    rc = _L().moe_oracle_gather(_p(idx), T, k, n_experts, _p(counts), _p(offsets), _p(perm))
    if rc:
        raise ValueError("moe_oracle_gather rc=%d" % rc)
    return counts, offsets, perm


def quantize_q4(w) -> Tuple[np.ndarray, np.ndarray]:
    """w [rows][cols] bf16 bits -> (codes [rows][cols/2] uint8, scales [rows][cols/64] bf16 bits)."""
    w = _u16(w)
    rows, cols = w.shape
    codes = np.zeros((rows, cols // 2), dtype=np.uint8)
    scales = np.zeros((rows, max(cols // 64, 1)), dtype=np.uint16)
    if _L().moe_oracle_quantize_q4(_p(w), rows, cols, _p(codes), _p(scales)):
        raise ValueError("cols must be a positive multiple of 64")
    return codes, scales


def dequantize_q4(codes, scales) -> np.ndarray:
    """The bf16 weights (bit patterns) the layer computes with for a 4-bit matrix."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = _u16(scales)
    rows, cols = codes.shape[0], codes.shape[1] * 2
    out = np.empty((rows, cols), dtype=np.uint16)
    if _L().moe_oracle_dequantize_q4(_p(codes), _p(scales), rows, cols, _p(out)):
        raise ValueError("cols must be a positive multiple of 64")
    return out


def miss_proxies(idx, n_experts: int, cache_slots: int, gamma: float):
    """Cache-miss proxies of one layer's routing trace (Section 3.1's cache simulation and
    Definition C.1), forward only.  idx [T][K]: the experts each token selected.

    Returns (soft, hard):
      soft  [T] fp64: sum_i r_i (1 - c_i) per token with the soft cache state c of Section 3.1
            (c starts at 0 and follows c <- gamma c + r while its L1 norm is below C; the first
            update that reaches C is rescaled to norm C and starts the normaliser Z = 1; from
            then on c <- (gamma Z c + r) / Z', Z' = gamma Z + K / C, which keeps the norm at C);
            their mean is the loss L_cs of that layer;
      hard  [T] int: requested experts outside the hard cache Top-C(count) of Definition C.1
            (count starts at 0, count <- gamma count + r; the cache holds the up to C experts of
            largest non-zero count, lower index first among equals): the misses of a
            gamma-discounted cache, whose sum is the number of transfers of Appendix C.1.
    """
    idx = np.asarray(idx, dtype=np.int64)
    T, K = idx.shape
    E, C = int(n_experts), int(cache_slots)
    c = np.zeros(E)
    Z, filled = 1.0, False
    count = np.zeros(E)
    soft = np.zeros(T)
    hard = np.zeros(T, dtype=np.int64)
    for t in range(T):
        r = np.zeros(E)
        r[idx[t]] = 1.0
        soft[t] = float((r * (1.0 - c)).sum())
        order = [i for i in np.argsort(-count, kind="stable") if count[i] > 0][:C]
        resident = np.zeros(E)
        resident[order] = 1.0
        hard[t] = int((r * (1.0 - resident)).sum())
        if not filled:
            nxt = gamma * c + r
            if nxt.sum() >= C:
                nxt *= C / nxt.sum()
                filled, Z = True, 1.0
            c = nxt
        else:
            Zn = gamma * Z + r.sum() / C
            c = (gamma * Z * c + r) / Zn
            Z = Zn
        count = gamma * count + r
    return soft, hard


class ExpertCache:
    """Expert cache of one layer; `call` takes one forward call's routing indices.

    policy "lru" (default) or "count": the gamma-discounted count of Definition C.1
    (gamma = 1 is LFU).
    """

    def __init__(self, cache_slots: int, n_experts: int, policy: str = "lru", gamma: float = 0.0):
        self.C, self.E = int(cache_slots), int(n_experts)
        self._h = _L().moe_oracle_cache_create(self.C, self.E)
        if not self._h:
            raise ValueError("bad cache shape")
        if policy != "lru":
            self.set_policy(policy, gamma)

    def set_policy(self, policy: str, gamma: float = 0.0) -> None:
        code = {"lru": 0, "count": 1}[policy]
        if _L().moe_oracle_cache_set_policy(self._h, code, C.c_float(gamma)):
            raise ValueError("bad policy or gamma")

    def preload(self, expert_ids) -> np.ndarray:
        """One request per id, in order, before the first token; returns the request records."""
        ids = np.ascontiguousarray(expert_ids, dtype=np.int32).reshape(-1)
        out = np.empty((max(ids.size, 1), 4), dtype=np.int32)
        n = _L().moe_oracle_cache_preload(self._h, _p(ids), ids.size, _p(out))
        if n < 0:
            raise ValueError("expert index out of range")
        return out[:n].copy()

    def counts(self) -> np.ndarray:
        c = np.empty(self.E, dtype=np.float32)
        _L().moe_oracle_cache_counts(self._h, _p(c))
        return c

    def __del__(self):
        if getattr(self, "_h", None):
            _L().moe_oracle_cache_destroy(self._h)
            self._h = None

    def reset(self):
        _L().moe_oracle_cache_reset(self._h)

    def call(self, idx) -> np.ndarray:
        """Returns the call's request records [n][4] = (expert, slot, hit, evicted) in order."""
        idx = np.ascontiguousarray(idx, dtype=np.int32).reshape(-1)
        out = np.empty((self.E, 4), dtype=np.int32)
        n = _L().moe_oracle_cache_call(self._h, _p(idx), idx.size, _p(out))
        if n < 0:
            raise ValueError("expert index out of range")
        return out[:n].copy()

    def state(self):
        eos = np.empty(self.C, dtype=np.int32)
        st = np.empty(self.C, dtype=np.uint64)
        tot = np.empty(3, dtype=np.uint64)
        _L().moe_oracle_cache_state(self._h, _p(eos), _p(st), _p(tot))
        return eos, st, {"hits": int(tot[0]), "misses": int(tot[1]), "evictions": int(tot[2])}


def ffn_combine(x, idx, gate, experts: Sequence, d_ff: int, n_shared: int = 0,
                tokens: Optional[Sequence[int]] = None) -> np.ndarray:
    """y [n_sel][d] fp64 (Eq. 2-3).  experts[e] = (W_g, W_u, W_d) bf16 bits or None; the
    n_shared shared experts follow the E routed ones in the list."""
    x = _u16(x)
    T, d = x.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    gate = np.ascontiguousarray(gate, dtype=np.float64)
    k = idx.shape[1]
    E = len(experts) - n_shared
    keep: List[np.ndarray] = []
    arrs = [(C.c_void_p * len(experts))() for _ in range(3)]
    for e, w in enumerate(experts):
        if w is None:
            continue
        shapes = ((d_ff, d), (d_ff, d), (d, d_ff))
        for m in range(3):
            a = _u16(w[m])
            assert a.shape == shapes[m], (a.shape, shapes[m])
            keep.append(a)
            arrs[m][e] = a.ctypes.data
    tok = None if tokens is None else np.ascontiguousarray(tokens, dtype=np.int32)
    n_sel = T if tok is None else tok.size
    y = np.empty((n_sel, d), dtype=np.float64)
    rc = _L().moe_oracle_ffn_combine(_p(x), _p(idx), _p(gate), arrs[0], arrs[1], arrs[2], d, d_ff, E, k,
                                     n_shared, _p(tok), n_sel, _p(y))
    if rc:
        raise ValueError("moe_oracle_ffn_combine rc=%d" % rc)
    return y


def layer_forward(x, w_r, experts, k, d_ff, cache: Optional[ExpertCache] = None, bias=None,
                  token_seq=None, n_shared: int = 0, tokens=None):
    """One forward call of the layer: routing, cache trace, outputs.  Returns a dict."""
    idx, gate, lg = route(x, w_r, k, bias, token_seq)
    E = np.asarray(w_r).shape[0]
    counts, offsets, perm = gather(idx, E)
    req = cache.call(idx) if cache is not None else None
    y = ffn_combine(x, idx, gate, experts, d_ff, n_shared, tokens)
    return {"idx": idx, "gate": gate, "logits": lg, "counts": counts, "offsets": offsets,
            "perm": perm, "requests": req, "y": y}
