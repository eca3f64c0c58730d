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


class GpuScenario:
    def __init__(self, sc: Scenario, host_lent: bool = False, **kw):
        self.sc = sc
        self.local = kv_to_dev(sc.local)
        if host_lent:       # the lent arena behind a real link: mapped pinned host memory
            self.lent = torch.from_numpy(B.kv_block_swizzle(sc.lent).view(np.int16)).pin_memory()
            kw["lent_kind"] = 1
        else:
            self.lent = kv_to_dev(sc.lent)
        self.staging = kv_to_dev(sc.staging)
        self.q = to_dev(sc.q)
        self.out = torch.zeros_like(self.q)
        self.lse = torch.zeros((sc.L, sc.nseq, sc.Hq), dtype=torch.float32, device="cuda")
        self.main = torch.cuda.Stream()
        self.side = torch.cuda.Stream(priority=-1)
        torch.cuda.synchronize()
        self.s = B.Slice(sc.L, sc.Hkv, sc.pl.local_blocks, sc.pl.lent_blocks, sc.staging_cap,
                         local=self.local, lent=self.lent, staging=self.staging,
                         lent_blocks_physical=sc.lent_phys, ring_slots=sc.wl.ring_slots,
                         max_seqs=sc.nseq + 4, max_blocks_per_seq=sc.max_blocks,
                         local_free_order=sc.local_order, lent_free_order=sc.lent_order, **kw)
        for i, hints in zip(sc.seq_ids, sc.pl.hints):
            for h in hints:
                rc, _ = self.s.slice_alloc_blocks(i, 1, int(h))
                assert rc == B.OK
            assert self.s.slice_set_seq_len(i, int(sc.pl.lengths[i])) == B.OK

    def tables_equal_oracle(self):
        for i in self.sc.seq_ids:
            rc, t, ln = self.s.slice_get_block_table(i)
            rc2, t2, ln2 = self.sc.orc.block_table(i)
            assert rc == rc2 == 0 and ln == ln2 and t.tolist() == t2.tolist()
        assert self.s.slice_get_free_stack(B.TIER_LOCAL).tolist() == self.sc.orc.free_stack(1).tolist()
        assert self.s.slice_get_free_stack(B.TIER_LENT).tolist() == self.sc.orc.free_stack(2).tolist()

    def device_ok(self):
        st = self.s.slice_stats()
        assert st["device_status"] == 0 and st["last_cuda_error"] == 0
        return st
