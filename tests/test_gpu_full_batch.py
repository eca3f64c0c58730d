"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The Llama-3-8B- and 70B-shaped batches are decoded with the default knobs (one persistent launch
per pass, one CTA per SM, work stealing). At these sizes a CTA's range is longer than 48 blocks, so
finished sequences are queued to the CTA's merge warp instead of being merged in line, and with 9
(6, 5) layers every buffer of split-KV partials is reused, some twice, behind the cross-CTA wait on
the merges of the layer that used it last: the combination that nearly every timed layer of the
benchmark runs. Everything is compared with the CPU oracle: resolved tables and staged bytes in
full, attention for every sequence and every head of the first, a middle and the last layer.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_27040_b200 import binding as B
from paper_2609_27040_b200 import build as build_mod
from paper_2609_27040_b200 import synth
from tests.helpers import attention_close

pytestmark = pytest.mark.gpu

ATOL = RTOL = 1e-2   # bf16 attention tolerance of the benchmark definition


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class FullBatch:
    """Arenas, slice and oracle state of one full-size workload restricted to L layers (block ids
    and tables do not depend on the layer, so a one-layer oracle serves every layer's bytes)."""

    def __init__(self, name: str, L: int, seed: int = 0, **kw):
        self.wl = wl = synth.WORKLOADS[name]
        self.L = L
        self.pl = pl = synth.make_placement(wl, seed, slack_blocks=64)
        gen = torch.Generator(device="cuda").manual_seed(seed)
        shape = (2, wl.block_tokens, wl.num_kv_heads, wl.head_dim)
        bf = torch.bfloat16
        self.local = torch.empty((L, pl.local_blocks) + shape, device="cuda", dtype=bf).normal_(generator=gen)
        self.lent = torch.empty((L, pl.lent_blocks) + shape, device="cuda", dtype=bf).normal_(generator=gen)
        self.staging = torch.zeros((2, pl.staging_blocks) + shape, device="cuda", dtype=bf)
        self.q = torch.empty((L, wl.batch, wl.num_q_heads, wl.head_dim), device="cuda", dtype=bf).normal_(generator=gen)
        self.out = torch.zeros_like(self.q)
        self.max_blocks = 520
        self.s = B.Slice(L, wl.num_kv_heads, pl.local_blocks, pl.lent_blocks, pl.staging_blocks, local=self.local,
                         lent=self.lent, staging=self.staging, max_seqs=wl.batch, max_blocks_per_seq=self.max_blocks,
                         local_free_order=pl.local_free_order, lent_free_order=pl.lent_free_order, **kw)
        self.orc = oracle.OracleSlice(1, wl.block_tokens, wl.block_bytes, pl.local_blocks, pl.lent_blocks, pl.lent_blocks,
                                      1, pl.staging_blocks, max_seqs=wl.batch, max_blocks_per_seq=self.max_blocks,
                                      local_free_order=pl.local_free_order, lent_free_order=pl.lent_free_order)
        for i, hints in enumerate(pl.hints):
            for h in hints:
                assert self.s.slice_alloc_blocks(i, 1, int(h))[0] == 0 and self.orc.alloc_blocks(i, 1, int(h))[0] == 0
            assert self.s.slice_set_seq_len(i, int(pl.lengths[i])) == 0 and self.orc.set_seq_len(i, int(pl.lengths[i])) == 0
        self.seqs = np.arange(wl.batch, dtype=np.int32)
        self.lens = np.asarray(pl.lengths, np.uint32)
        self.main, self.side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
        self.scale = 1.0 / np.sqrt(wl.head_dim)

    def decode_passes(self, n: int):
        for _ in range(n):
            assert self.s.slice_decode_step(self.seqs, self.q, self.wl.num_q_heads, self.scale, self.out, False, True,
                                            self.main, self.side) == B.OK
        torch.cuda.synchronize()
        st = self.s.slice_stats()
        assert st["device_status"] == 0 and st["last_cuda_error"] == 0
        return st

    def check_tables(self):
        rc, resolved, k = self.orc.gather(0, self.seqs, None, None)
        rc2, res_gpu, k_gpu = self.s.slice_get_resolved(self.seqs)
        assert rc == rc2 == 0 and k == k_gpu == self.pl.staging_blocks
        assert (resolved == res_gpu).all()
        for i in range(self.wl.batch):
            assert self.s.slice_get_block_table(i)[1].tolist() == self.orc.block_table(i)[1].tolist()
        return resolved, k

    def check_staged_bytes(self, k: int):
        """The two ring slots, in full, against the lent arena read through the oracle's tables (on the
        device), and slot 0 once more against the oracle's own gather (on the host)."""
        L = self.L
        ids = torch.tensor([~int(e) for i in range(self.wl.batch)
                            for e in self.orc.block_table(i)[1][: synth.blocks_for(self.pl.lengths[i])] if e < 0], device="cuda")
        last_odd = L - 1 if (L - 1) % 2 else L - 2
        for layer, slot in ((0, 0), (last_odd, 1)):        # slot 0 was refilled with layer 0 for the next pass
            assert torch.equal(self.staging[slot, :k], self.lent[layer].index_select(0, ids)), (layer, slot)
        lent0 = _bits(B.kv_block_swizzle(self.lent[0]))
        staged = np.zeros((1, k) + lent0.shape[1:], np.uint16)
        rc, _, k2 = self.orc.gather(0, self.seqs, lent0[None], staged)
        assert rc == 0 and k2 == k
        assert (_bits(B.kv_block_swizzle(self.staging[0, :k])) == staged[0]).all()

    def check_attention_in_full(self, layer: int, resolved: np.ndarray, k: int, q_layer=None, out_layer=None):
        """Every sequence and every query head of `layer`: the oracle gathers the layer's lent blocks
        into a host staging slot and attends in fp64 through the resolved table. q_layer / out_layer
        (device tensors) replace self.q[layer] / self.out[layer] where the pass used other buffers."""
        wl = self.wl
        q_layer = self.q[layer] if q_layer is None else q_layer
        out_layer = self.out[layer] if out_layer is None else out_layer
        local = _bits(B.kv_block_swizzle(self.local[layer]))       # block format -> canonical token rows
        lent = _bits(B.kv_block_swizzle(self.lent[layer]))
        staged = np.zeros((1, max(k, 1)) + lent.shape[1:], np.uint16)
        assert self.orc.gather(0, self.seqs, lent[None], staged)[0] == 0
        rc, ref, _ = oracle.paged_attention(_bits(q_layer), local, staged[0], resolved, self.lens, wl.num_q_heads,
                                            wl.num_kv_heads, wl.head_dim, wl.block_tokens, self.scale, want_lse=False)
        assert rc == 0
        got = out_layer.double().cpu().numpy()
        assert np.isfinite(got).all()
        ok, max_abs, max_rel = attention_close(got, ref, ATOL, RTOL)
        assert ok, (layer, max_abs, max_rel)
        return max_abs


@pytest.mark.parametrize("name,L,kw", [
    ("llama3_8b_decode", 9, {}),                              # four partial buffers, each reused at least once
    ("llama3_70b_decode", 6, {}),
    ("llama3_8b_decode", 5, {"prefetch_priority": 1}),        # two partial buffers, reused twice
    ("llama3_8b_decode", 9, {"pipeline_mode": 3}),            # the same pass as a chain of one launch per layer
])
def test_timed_launch_configuration_matches_oracle_in_full(name, L, kw):
    fb = FullBatch(name, L, **kw)
    per = -(-fb.pl.total_blocks // 148)
    assert per > 48                                            # merges are queued, not done in line
    st = fb.decode_passes(2)
    per_pass = L if kw.get("pipeline_mode") == 3 else 1
    assert st["kernel_launches"] <= 2 * per_pass + 3           # one launch per pass (per layer in a chain), plus the
                                                               # gathers of layer 0 (priming; refill of a slot the
                                                               # last layer shares)
    resolved, k = fb.check_tables()
    fb.check_staged_bytes(k)
    mid = max(4, L // 2) if L > 5 else 3
    for layer in sorted({0, mid, L - 1}):
        fb.check_attention_in_full(layer, resolved, k)
    fb.s.close()


@pytest.mark.parametrize("swap", [1, 2])
def test_swap_out_pass_at_full_batch_writes_the_ring_back_inside_its_one_launch(swap):
    """swap_out at the benchmark's size: the write-back of every staged layer (1), or of its staged
    tail blocks only (2), is done by the copy threads of the one launch that is the pass. A block of
    layer 0 is changed in its STAGED copy only (as an appended row would: a tail block); after the
    next pass the lent arena must hold the change, the pass must have attended to it, and every
    other byte of the lent arena must be as it was."""
    L = 6
    fb = FullBatch("llama3_8b_decode", L, swap_out=swap)
    fb.decode_passes(1)                                        # leaves layer 0 staged in slot 0 for the next pass
    before = fb.lent.clone()
    rc, resolved, k = fb.orc.gather(0, fb.seqs, None, None)
    assert rc == 0 and k == fb.pl.staging_blocks
    # the first sequence whose tail block is lent: its staging position and its lent id
    pos, lent_id, at = None, None, 0
    for i in range(fb.wl.batch):
        entries = fb.orc.block_table(i)[1][: synth.blocks_for(fb.pl.lengths[i])]
        staged = [int(e) for e in entries if e < 0]
        if pos is None and entries[-1] < 0:
            pos, lent_id = at + len(staged) - 1, ~int(entries[-1])
        at += len(staged)
    assert pos is not None
    assert torch.equal(fb.staging[0, pos], fb.lent[0, lent_id])
    fb.staging[0, pos].mul_(-1.0)                              # the change exists in the ring only
    changed = fb.staging[0, pos].clone()
    assert not torch.equal(changed, fb.lent[0, lent_id])
    k0 = fb.s.slice_stats()["kernel_launches"]
    st = fb.decode_passes(1)
    assert st["kernel_launches"] - k0 <= 3                     # one launch for the pass (+ at most the gathers of layer 0)
    assert torch.equal(fb.lent[0, lent_id], changed)           # written back
    before[0, lent_id] = changed
    assert torch.equal(fb.lent, before)                        # and nothing else moved
    resolved, k = fb.check_tables()
    for layer in (0, 3, L - 1):                                # layer 0 was attended to with the change in place
        fb.check_attention_in_full(layer, resolved, k)
    fb.s.close()
