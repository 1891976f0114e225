"""CPU-side checks of the CUDA library: it loads, exports what the header declares, and its
pure-host helpers work.  No kernel is launched here."""
import os
import re

import numpy as np
import pytest

import gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def m():
    from paper_2602_11192_b200 import build
    build.build()
    import paper_2602_11192_b200 as mod
    return mod


def test_library_exports_every_declared_symbol(m):
    hdr = open(os.path.join(ROOT, "include", "melinoe_moe.h")).read()
    declared = set(re.findall(r"^(?:int|size_t|int64_t|const char \*)\s*(melinoe_[a-z0-9_]+)\s*\(", hdr, re.M))
    assert declared, "no declarations found"
    L = m.lib()
    for name in sorted(declared):
        assert hasattr(L, name), "library does not export %s" % name
    assert declared == set(m.EXPORTED_SYMBOLS), declared ^ set(m.EXPORTED_SYMBOLS)


def test_status_strings_and_sizes(m):
    assert m.melinoe_strerror(0) == "ok" and "argument" in m.melinoe_strerror(1)
    assert m.melinoe_moe_expert_bytes(4096, 14336) == 352321536
    assert m.melinoe_moe_expert_bytes(2048, 1024) == 12 * 2 ** 20
    assert m.melinoe_moe_expert_bytes(0, 5) == 0


def test_pack_expert_layout(m):
    """Per hidden unit f the blob holds W_g[f] | W_u[f] | W_d[:, f]; inside every 64-element group the
    eight 8-element pieces sit at (piece xor (f mod 8)).  Undoing that permutation with index
    arithmetic written here gives the three matrices back."""
    d, F = 256, 24
    wg, wu, wd = gen.expert_weights(1, 0, 0, d, F)
    blob = np.zeros(3 * d * F, np.uint16)
    m.melinoe_moe_pack_expert(d, F, wg.ctypes.data, wu.ctypes.data, wd.ctypes.data, blob.ctypes.data)
    rows = blob.reshape(F, 3, d // 64, 8, 8)                     # f, vector, group, stored piece, element
    plain = np.empty_like(rows)
    for f in range(F):
        for piece in range(8):
            plain[f, :, :, piece, :] = rows[f, :, :, piece ^ (f & 7), :]
    plain = plain.reshape(F, 3, d)
    assert np.array_equal(plain[:, 0, :], wg) and np.array_equal(plain[:, 1, :], wu)
    assert np.array_equal(plain[:, 2, :], wd.T)
    # rows 0 and 8 are stored unpermuted, row 1 swaps neighbouring pieces
    assert np.array_equal(blob[:8], wg[0, :8]) and np.array_equal(blob[3 * d:3 * d + 8], wg[1, 8:16])
    with pytest.raises(m.MelinoeError):
        m.melinoe_moe_pack_expert(d, F, 0, wu.ctypes.data, wd.ctypes.data, blob.ctypes.data)


def test_pack_expert_q4_matches_the_oracle_bit_for_bit(m):
    """The library's host-side quantiser against the oracle's (independent code, same definition).  The
    blob is per hidden unit f: codes of W_g[f], W_u[f], W_d[:, f] (the quantisation groups of W_d run down
    its columns), then the three scale vectors; 16-byte code pieces at (piece xor (f mod 8)) within every
    eight; the codes of W_d[:, f] are interleaved within every group of 64 (position p = element 8 (p mod 8) + p // 8)."""
    import oracle
    for d, F in ((256, 24), (512, 64)):
        rs = np.random.default_rng(3)
        w = [gen.f32_to_bf16_bits(rs.normal(0.0, 0.02, shp).astype(np.float32)) for shp in ((F, d), (F, d), (d, F))]
        w[0][0, :64] = 0                                            # an all-zero group
        w[1][1, :8] = gen.f32_to_bf16_bits(np.array([0.875, -0.875, 0.0625, 0.1875, -0.0625, -0.1875, 0.125, 0.0], np.float32))
        w[1][1, 8:64] = 0                                           # ties exactly between two codes
        unit = (3 * (d // 2) + 3 * (d // 64) * 2 + 15) // 16 * 16
        qb = m.melinoe_moe_expert_bytes_q4(d, F)
        assert qb == F * unit
        blob = np.full(qb, 0xAB, np.uint8)
        m.melinoe_moe_pack_expert_q4(d, F, w[0].ctypes.data, w[1].ctypes.data, w[2].ctypes.data, blob.ctypes.data)
        units = blob.reshape(F, unit)
        want = [oracle.quantize_q4(w[0]), oracle.quantize_q4(w[1]), oracle.quantize_q4(np.ascontiguousarray(w[2].T))]
        for f in range(F):
            for i, (codes, scales) in enumerate(want):
                stored = units[f, i * (d // 2):(i + 1) * (d // 2)].reshape(-1, 16)
                plain = np.empty_like(stored)
                for piece in range(stored.shape[0]):
                    plain[piece] = stored[(piece & ~7) | ((piece ^ f) & 7)]
                got = plain.reshape(-1)
                if i == 2:
                    # W_d[:, f]: within a group of 64, code position p holds element 8 (p mod 8) + p // 8
                    nib = np.stack([got & 15, got >> 4], axis=1).reshape(-1, 8, 8)       # group, element mod 8, element // 8
                    nib = nib.transpose(0, 2, 1).reshape(-1, 2)
                    got = (nib[:, 0] | (nib[:, 1] << 4)).astype(np.uint8)
                assert np.array_equal(got, codes[f]), (d, f, i)
                sc = units[f, 3 * (d // 2) + i * (d // 32):3 * (d // 2) + (i + 1) * (d // 32)].view(np.uint16)
                assert np.array_equal(sc, scales[f]), (d, f, i)
            assert not units[f, 3 * (d // 2) + 3 * (d // 32):].any()      # padding is zeroed
    assert m.melinoe_moe_expert_bytes_q4(256, 40) == 40 * 416 and m.melinoe_moe_expert_bytes_q4(256, 36) == 0
    assert m.melinoe_moe_expert_bytes_q4(320, 64) == 0
    with pytest.raises(m.MelinoeError):
        m.melinoe_moe_pack_expert_q4(256, 36, w[0].ctypes.data, w[1].ctypes.data, w[2].ctypes.data, blob.ctypes.data)


def test_budget_allocation_spends_slots_where_they_save_transfers(m):
    """Host logic of the per-layer budget (melinoe_allocate_slots): greedy on the marginal transfers saved.
    Pure host code: needs the library, no device."""
    def alloc(hard, sizes, budget):
        hard = np.ascontiguousarray(hard, dtype=np.int64)
        out = np.zeros(hard.shape[0], np.int32)
        rc = m.lib().melinoe_allocate_slots(hard.ctypes.data, hard.shape[0], hard.shape[1], sizes[0], budget, out.ctypes.data)
        if rc:
            raise ValueError("status %d" % rc)
        return out.tolist()
    sizes = [2, 3, 4, 5, 6]
    hard = np.array([[100, 60, 50, 49, 49],      # layer 0: the third slot is worth 40, then little
                     [100, 95, 90, 85, 80],      # layer 1: every slot is worth 5
                     [30, 30, 30, 30, 30]])      # layer 2: nothing to gain
    assert alloc(hard, sizes, 6) == [2, 2, 2]
    assert alloc(hard, sizes, 7) == [3, 2, 2]
    assert alloc(hard, sizes, 8) == [4, 2, 2]                 # 10 saved on layer 0 beats 5 on layer 1
    assert alloc(hard, sizes, 10) == [4, 4, 2]
    assert alloc(hard, sizes, 30) == [6, 6, 6]                # more budget than sizes: everything at the largest
    with pytest.raises(ValueError):
        alloc(hard, sizes, 5)


def test_create_fails_loudly_without_a_device(m):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(m.MelinoeError) as ei:
        m.MoELayer(256, 64, 8, 2, 4)
    assert ei.value.status == 3          # CUDA error, never a CPU fallback
