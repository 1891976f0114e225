"""Set-up helpers shared by the tests, the smoke check and the benchmark: build the pinned
expert store of a layer from paper-layout matrices, create the handle, move inputs.

Nothing here computes any step of the layer; torch is used for device / pinned memory and
streams only.
"""
from __future__ import annotations

import concurrent.futures as cf
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

from . import binding as B

__all__ = ["LayerSetup", "to_dev_bf16", "current_stream_ptr"]


def current_stream_ptr() -> int:
    return int(torch.cuda.current_stream().cuda_stream)


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> device tensor (kept as int16 storage; only its address is used)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()


class LayerSetup:
    """One layer: pinned host store of packed experts, device router, the library handle."""

    def __init__(self, d_model: int, d_ff: int, n_experts: int, top_k: int, cache_slots: int, n_shared: int = 0,
                 slots: str = "bf16"):
        """slots = "q4": the cache slots (and therefore the store and the shared experts) hold 4-bit blobs."""
        self.d, self.F, self.E, self.k, self.C, self.n_shared = d_model, d_ff, n_experts, top_k, cache_slots, n_shared
        self.slots = slots
        if slots == "q4":
            self.expert_bytes = B.melinoe_moe_expert_bytes_q4(d_model, d_ff)
            self.store = None
        else:
            self.expert_bytes = B.melinoe_moe_expert_bytes(d_model, d_ff)
            self.store = torch.empty((n_experts, self.expert_bytes), dtype=torch.uint8, pin_memory=True)
        self.shared_store: Optional[torch.Tensor] = None
        self.layer = B.MoELayer(d_model, d_ff, n_experts, top_k, cache_slots, slots=slots)
        self.router_dev: Optional[torch.Tensor] = None
        self.bias_dev = None
        self.seq_dev = None

    # -- weights
    def pack_expert_into(self, dst_ptr: int, wg, wu, wd) -> None:
        """wg/wu [F][d], wd [d][F]: numpy uint16 or torch bf16 CPU tensors, contiguous."""
        def ptr(a):
            if isinstance(a, torch.Tensor):
                assert a.is_contiguous() and a.device.type == "cpu"
                return a.data_ptr()
            a = np.ascontiguousarray(a)
            self._tmp.append(a)
            return a.ctypes.data
        self._tmp: List = []
        B.melinoe_moe_pack_expert(self.d, self.F, ptr(wg), ptr(wu), ptr(wd), dst_ptr)
        self._tmp = []

    def set_experts(self, experts: Sequence[Tuple], shared: Sequence[Tuple] = ()) -> None:
        """experts[e] = (W_g, W_u, W_d) in the paper's shapes; packs them into the pinned store."""
        assert len(experts) == self.E and len(shared) == self.n_shared
        base = self.store.data_ptr()
        for e, (wg, wu, wd) in enumerate(experts):
            self.pack_expert_into(base + e * self.expert_bytes, wg, wu, wd)
        self.layer.register_host_experts([base + e * self.expert_bytes for e in range(self.E)],
                                         self.expert_bytes, keep=self.store)
        if self.n_shared:
            tmp = torch.empty((self.n_shared, self.expert_bytes), dtype=torch.uint8)
            for s, (wg, wu, wd) in enumerate(shared):
                self.pack_expert_into(tmp.data_ptr() + s * self.expert_bytes, wg, wu, wd)
            self.shared_store = tmp.cuda()
            sb = self.shared_store.data_ptr()
            self.layer.register_shared_experts([sb + s * self.expert_bytes for s in range(self.n_shared)],
                                               keep=self.shared_store)

    def set_experts_q4(self, experts: Sequence[Tuple], shared: Sequence[Tuple] = ()) -> None:
        """experts[e] = (W_g, W_u, W_d) numpy uint16 (bf16 bits): quantised into a 4-bit pinned store."""
        assert len(experts) == self.E
        if self.n_shared and self.slots == "q4":
            assert len(shared) == self.n_shared
            tmp = torch.empty((self.n_shared, self.expert_bytes), dtype=torch.uint8)
            for s_, w in enumerate(shared):
                a = [np.ascontiguousarray(m) for m in w]
                B.melinoe_moe_pack_expert_q4(self.d, self.F, a[0].ctypes.data, a[1].ctypes.data, a[2].ctypes.data,
                                             tmp.data_ptr() + s_ * self.expert_bytes)
            self.shared_store = tmp.cuda()
            sb = self.shared_store.data_ptr()
            self.layer.register_shared_experts([sb + s_ * self.expert_bytes for s_ in range(self.n_shared)],
                                               keep=self.shared_store)
        qb = B.melinoe_moe_expert_bytes_q4(self.d, self.F)
        assert qb > 0, "the 4-bit store needs d_ff % 64 == 0"
        self.store_q4 = torch.empty((self.E, qb), dtype=torch.uint8, pin_memory=True)
        base = self.store_q4.data_ptr()
        for e, (wg, wu, wd) in enumerate(experts):
            a = [np.ascontiguousarray(m) for m in (wg, wu, wd)]
            B.melinoe_moe_pack_expert_q4(self.d, self.F, a[0].ctypes.data, a[1].ctypes.data, a[2].ctypes.data,
                                         base + e * qb)
        self.layer.register_host_experts_q4([base + e * qb for e in range(self.E)], qb, keep=self.store_q4)

    def set_experts_stacked(self, wg: torch.Tensor, wu: torch.Tensor, wd: torch.Tensor, threads: int = 16) -> None:
        """Whole layer at once: wg/wu [E][F][d], wd [E][d][F] bf16 CPU tensors."""
        base = self.store.data_ptr()
        eb = self.expert_bytes

        def one(e):
            B.melinoe_moe_pack_expert(self.d, self.F, wg[e].data_ptr(), wu[e].data_ptr(), wd[e].data_ptr(),
                                      base + e * eb)
        with cf.ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(one, range(self.E)))
        self.layer.register_host_experts([base + e * eb for e in range(self.E)], eb, keep=self.store)

    def set_experts_stacked_q4(self, wg: torch.Tensor, wu: torch.Tensor, wd: torch.Tensor, threads: int = 16) -> None:
        """Whole layer at once into a 4-bit pinned store: wg/wu [E][F][d], wd [E][d][F] bf16 CPU tensors."""
        qb = B.melinoe_moe_expert_bytes_q4(self.d, self.F)
        assert qb > 0, "the 4-bit store needs d_ff % 64 == 0"
        self.store_q4 = torch.empty((self.E, qb), dtype=torch.uint8, pin_memory=True)
        base = self.store_q4.data_ptr()

        def one(e):
            B.melinoe_moe_pack_expert_q4(self.d, self.F, wg[e].data_ptr(), wu[e].data_ptr(), wd[e].data_ptr(),
                                         base + e * qb)
        with cf.ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(one, range(self.E)))
        self.layer.register_host_experts_q4([base + e * qb for e in range(self.E)], qb, keep=self.store_q4)

    def set_shared_stacked(self, wg: torch.Tensor, wu: torch.Tensor, wd: torch.Tensor) -> None:
        """Shared experts of the layer: wg/wu [n_shared][F][d], wd [n_shared][d][F] bf16 CPU tensors."""
        assert wg.shape[0] == self.n_shared
        tmp = torch.empty((self.n_shared, self.expert_bytes), dtype=torch.uint8)
        pack = B.melinoe_moe_pack_expert_q4 if self.slots == "q4" else B.melinoe_moe_pack_expert
        for s in range(self.n_shared):
            pack(self.d, self.F, wg[s].data_ptr(), wu[s].data_ptr(), wd[s].data_ptr(), tmp.data_ptr() + s * self.expert_bytes)
        self.shared_store = tmp.cuda()
        sb = self.shared_store.data_ptr()
        self.layer.register_shared_experts([sb + s * self.expert_bytes for s in range(self.n_shared)],
                                           keep=self.shared_store)

    def set_router(self, w_r_bits: np.ndarray) -> None:
        self.router_dev = to_dev_bf16(w_r_bits)
        self.layer.set_router(self.router_dev)

    def set_bias(self, bias: Optional[np.ndarray], token_seq: Optional[np.ndarray]) -> None:
        if bias is None:
            self.bias_dev = self.seq_dev = None
            self.layer.set_router_bias(None, None, 0)
            return
        bias = np.ascontiguousarray(bias, dtype=np.float32).reshape(-1, self.E)
        self.bias_dev = torch.from_numpy(bias).cuda()
        self.seq_dev = None if token_seq is None else torch.from_numpy(
            np.ascontiguousarray(token_seq, dtype=np.int32)).cuda()
        self.layer.set_router_bias(self.bias_dev, self.seq_dev, bias.shape[0])

    # -- one call with numpy in / numpy out (blocking; for tests)
    def forward_np(self, hidden_bits: np.ndarray, want_stats: bool = True, entry: str = "forward"):
        T = hidden_bits.shape[0]
        x = to_dev_bf16(hidden_bits)
        out = torch.full((T, self.d), 0x7FC0, dtype=torch.int16, device="cuda")   # NaN pattern: must be overwritten
        stats = torch.zeros(12, dtype=torch.int32, device="cuda") if want_stats else None
        call = self.layer.forward_static if entry == "static" else self.layer.forward
        call(current_stream_ptr(), x, T, out, stats)
        torch.cuda.synchronize()
        res = {"out_bits": out.cpu().numpy().view(np.uint16)}
        if want_stats:
            s = stats.cpu().numpy()
            res["stats"] = {"status": int(s[0]), "n_tokens": int(s[1]), "n_distinct": int(s[2]), "hits": int(s[3]),
                            "misses": int(s[4]), "evictions": int(s[5]), "groups": int(s[6]),
                            "bytes_h2d": int(s[8:10].view(np.uint64)[0]), "call_no": int(s[10:12].view(np.uint64)[0])}
        return res

    def close(self) -> None:
        self.layer.destroy()
