"""Mirrors a host Scenario on the GPU: same arenas, same free orders, same allocation calls, made
through the C ABI of the CUDA library."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_27040_b200 import binding as B
from tests.helpers import Scenario


def to_dev(a: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns -> int16 CUDA tensor with the same bytes."""
    return torch.from_numpy(a.view(np.int16)).cuda()


def to_host(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint16)


def kv_to_dev(a: np.ndarray) -> torch.Tensor:
    """KV blocks [..., 2, 16, Hkv, 128] in canonical order (as the oracle reads them) -> device tensor
    in the library's block format."""
    return to_dev(B.kv_block_swizzle(a))


def kv_to_host(t: torch.Tensor) -> np.ndarray:
    """Device KV blocks in the library's block format -> canonical order on the host."""
    return B.kv_block_swizzle(to_host(t))


def layout_positions(layout: int, L: int, n_blocks: int, slab: int, group: int) -> np.ndarray:
    """[L][n_blocks] block position of every (layer, id) in an arena of the given layout, from the
    oracle's address map (tests place and read bytes through it; the library has its own)."""
    import oracle
    bb = 64
    return np.array([[oracle.layout_offset(layout, L, n_blocks, slab, max(group, 1), bb, l, b) // bb
                      for b in range(n_blocks)] for l in range(L)], np.int64)


class GpuScenario:
    def __init__(self, sc: Scenario, host_lent: bool = False, layout: int = 0, layer_group: int = 0, **kw):
        self.sc = sc
        self.layout = layout
        if sc.slab:
            kw["slab_blocks"] = sc.slab
        if layer_group:
            kw["layer_group"] = layer_group
        if layout:
            kw["layout"] = layout
            self.pos_local = layout_positions(layout, sc.L, sc.pl.local_blocks, sc.slab, layer_group)
            self.pos_lent = layout_positions(layout, sc.L, sc.lent_phys, sc.slab, layer_group)
        local_h, lent_h = self.to_layout(sc.local, True), self.to_layout(sc.lent, False)
        self.local = kv_to_dev(local_h)
        if host_lent:       # the lent arena behind a real link: mapped pinned host memory
            self.lent = torch.from_numpy(B.kv_block_swizzle(lent_h).view(np.int16)).pin_memory()
            kw["lent_kind"] = 1
        else:
            self.lent = kv_to_dev(lent_h)
        self.staging = kv_to_dev(sc.staging)
        self.q = to_dev(sc.q)
        self.out = torch.zeros_like(self.q)
        self.lse = torch.zeros((sc.L, sc.nseq, sc.Hq), dtype=torch.float32, device="cuda")
        self.main = torch.cuda.Stream()
        self.side = torch.cuda.Stream(priority=-1)
        torch.cuda.synchronize()
        ring = sc.wl.ring_slots // max(layer_group, 1)      # sc.wl.ring_slots counts layer slots
        assert ring * max(layer_group, 1) == sc.wl.ring_slots
        self.s = B.Slice(sc.L, sc.Hkv, sc.pl.local_blocks, sc.pl.lent_blocks, sc.staging_cap,
                         local=self.local, lent=self.lent, staging=self.staging,
                         lent_blocks_physical=sc.lent_phys, ring_slots=ring,
                         max_seqs=sc.nseq + 4, max_blocks_per_seq=sc.max_blocks,
                         local_free_order=sc.local_order, lent_free_order=sc.lent_order, **kw)
        for i, hints in zip(sc.seq_ids, sc.pl.hints):
            for h in hints:
                rc, _ = self.s.slice_alloc_blocks(i, 1, int(h))
                assert rc == B.OK
            assert self.s.slice_set_seq_len(i, int(sc.pl.lengths[i])) == B.OK

    def to_layout(self, canon: np.ndarray, local: bool) -> np.ndarray:
        """Canonical [L][N][block] host arena -> the same blocks in the device arena's order."""
        if not self.layout:
            return canon
        pos = self.pos_local if local else self.pos_lent
        flat = np.empty_like(canon).reshape((-1,) + canon.shape[2:])
        flat[pos.ravel()] = canon.reshape((-1,) + canon.shape[2:])
        return flat.reshape(canon.shape)

    def from_layout(self, dev: torch.Tensor, local: bool) -> np.ndarray:
        """Device arena -> canonical [L][N][block] host array (canonical token rows)."""
        h = kv_to_host(dev)
        if not self.layout:
            return h
        pos = self.pos_local if local else self.pos_lent
        return h.reshape((-1,) + h.shape[2:])[pos]

    def tables_equal_oracle(self):
        for i in self.sc.seq_ids:
            rc, t, ln = self.s.slice_get_block_table(i)
            rc2, t2, ln2 = self.sc.orc.block_table(i)
            assert rc == rc2 == 0 and ln == ln2 and t.tolist() == t2.tolist()
        order = sorted if self.sc.slab else list      # the slab rule, not a stack, orders the free ids
        assert order(self.s.slice_get_free_stack(B.TIER_LOCAL).tolist()) == order(self.sc.orc.free_stack(1).tolist())
        assert order(self.s.slice_get_free_stack(B.TIER_LENT).tolist()) == order(self.sc.orc.free_stack(2).tolist())

    def device_ok(self):
        st = self.s.slice_stats()
        assert st["device_status"] == 0 and st["last_cuda_error"] == 0
        return st
