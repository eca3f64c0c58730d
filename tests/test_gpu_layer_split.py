"""Layer-split placement (Section 4.1: a request keeps part of its LAYERS in its own memory and the
rest in the peer's; with half of them there the expansion ratio is the paper's 2). Every block has
one id that names its place in both arenas; layers below the split are attended to in place, layers
from the split on are prefetched whole, layer by layer, ahead of their attention.

The oracle side is two of the oracle's slices fed the same allocation calls: one whose blocks are
all local (the layers below the split), one whose blocks are all lent (the layers from the split
on); with the plain ascending id order both hand out the same ids."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_27040_b200 import binding as B
from paper_2609_27040_b200 import build as build_mod
from paper_2609_27040_b200 import synth
from tests.helpers import Scenario, attention_close

pytestmark = pytest.mark.gpu

ATOL = RTOL = 1e-2


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


class SplitScenario:
    def __init__(self, L, split, seed, hq=16, hkv=4, nseq=5, group=0, **kw):
        from tests.gpu_helpers import kv_to_dev, to_dev
        self.L, self.split, self.group = L, split, max(group, 1)
        ring = 2 * self.group
        wl_a = synth.Workload("split_local", split, hq, hkv, nseq, 40, 900, 0.0, ring_slots=ring)
        wl_b = synth.Workload("split_lent", L - split, hq, hkv, nseq, 40, 900, 1.0, ring_slots=ring)
        self.a = Scenario(wl_a, seed, permute=False, slack=24)      # layers 0 .. split-1: every block local
        self.b = Scenario(wl_b, seed, permute=False, slack=24)      # layers split .. L-1: every block lent
        a, b = self.a, self.b
        assert (a.pl.lengths == b.pl.lengths).all() and a.pl.local_blocks == b.lent_phys
        for i in a.seq_ids:                                          # the same ids on both sides
            assert a.orc.block_table(i)[1].tolist() == (~b.orc.block_table(i)[1]).tolist()
        self.seq_ids, self.nseq, self.Hq, self.Hkv = a.seq_ids, a.nseq, hq, hkv
        self.local, self.lent = kv_to_dev(a.local), kv_to_dev(b.lent)
        self.staging = kv_to_dev(b.staging)                          # [ring layer slots][all blocks of the batch]
        self.q = torch.cat([to_dev(a.q), to_dev(b.q)])
        self.out = torch.zeros_like(self.q)
        self.main, self.side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
        torch.cuda.synchronize()
        self.s = B.Slice(L, hkv, a.pl.local_blocks, b.lent_phys, b.staging_cap, local=self.local, lent=self.lent,
                         staging=self.staging, ring_slots=2, max_seqs=nseq + 2, max_blocks_per_seq=a.max_blocks,
                         split_layer=split, layer_group=group, **kw)
        for i, hints in zip(a.seq_ids, a.pl.hints):
            for _ in hints:
                assert self.s.slice_alloc_blocks(i, 1, B.TIER_AUTO)[0] == B.OK
            assert self.s.slice_set_seq_len(i, int(a.pl.lengths[i])) == B.OK
            assert self.s.slice_get_block_table(i)[1].tolist() == a.orc.block_table(i)[1].tolist()

    def part(self, layer):
        """(scenario, layer index inside it) that holds `layer`."""
        return (self.a, layer) if layer < self.split else (self.b, layer - self.split)

    def reference(self, layer):
        sc, l = self.part(layer)
        rc, resolved, k = sc.orc.gather(l, sc.seq_ids, sc.lent, sc.staging)
        assert rc == oracle.OK
        q = self.q[layer].cpu().numpy().view(np.uint16)
        # the oracle's own slice has L - split layers and stages layer l in slot l mod ring; the
        # library stages global layer `layer` in slot layer mod ring: compare bytes through `k`
        rc, ref, _ = oracle.paged_attention(q, sc.local[l], sc.staging[l % sc.wl.ring_slots], resolved, sc.lengths(),
                                            sc.Hq, sc.Hkv, sc.D, sc.T, sc.sm_scale)
        assert rc == oracle.OK
        return ref, k, sc.staging[l % sc.wl.ring_slots]

    def check_pass(self):
        from tests.gpu_helpers import kv_to_host
        seqs = np.asarray(self.seq_ids, np.int32)
        self.out.zero_()
        assert self.s.slice_decode_step(seqs, self.q, self.Hq, float(self.a.sm_scale), self.out, False, True, self.main,
                                        self.side) == B.OK
        torch.cuda.synchronize()
        st = self.s.slice_stats()
        assert st["device_status"] == 0 and st["last_cuda_error"] == 0
        got = self.out.view(torch.bfloat16).double().cpu().numpy()
        ring = 2 * self.group
        last_in_slot = {}
        for layer in range(self.L):
            ref, k, staged = self.reference(layer)
            ok, max_abs, _ = attention_close(got[layer], ref, ATOL, RTOL)
            assert ok, (layer, max_abs)
            if layer >= self.split:
                last_in_slot[layer % ring] = (k, staged.copy())
        for slot, (k, staged) in last_in_slot.items():               # what the lent half left in the ring
            assert (kv_to_host(self.staging[slot, :k]) == staged[:k]).all(), slot


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
@pytest.mark.parametrize("L,split,group", [(6, 3, 0), (8, 4, 2), (5, 1, 0), (5, 4, 0)])
def test_layer_split_matches_oracle_in_every_pipeline(mode, L, split, group):
    sp = SplitScenario(L, split, 11, group=group, pipeline_mode=mode, decode_ctas=12)
    n_blocks = sum(len(h) for h in sp.a.pl.hints)
    ring = 2 * max(group, 1)
    for rep in range(2):
        before = sp.s.slice_stats()["prefetched_blocks"]
        sp.check_pass()
        fetched = sp.s.slice_stats()["prefetched_blocks"] - before
        # every block of every lent layer in the first pass; later passes find the layers still
        # staged that no other lent layer has displaced from its slot (the local half uses no slot)
        displaced = sum(1 for l in range(split, L) if any(j != l and j % ring == l % ring for j in range(split, L)))
        assert fetched == ((L - split) if rep == 0 else displaced) * n_blocks, (rep, fetched // n_blocks)


def test_layer_split_calls_that_do_not_apply_and_append():
    from tests.gpu_helpers import kv_to_host, to_dev
    sp = SplitScenario(6, 3, 5)
    assert sp.s.slice_alloc_blocks(40, 1, B.TIER_LENT)[0] == B.EINVAL     # ids are not lent one by one
    assert sp.s.slice_reclaim(4, sp.main)[0] == B.EINVAL                  # nothing can migrate: preempt instead
    assert sp.s.prefetch_layer(1, sp.seq_ids, sp.side) == B.OK            # local half: nothing to do
    assert sp.s.slice_writeback_layer(1, sp.seq_ids, sp.main) == B.EINVAL
    sp.check_pass()
    # one more token for every sequence, all layers in one launch: the home of a layer's row is the
    # local arena below the split and the lent arena from it on (plus the staged copy where staged)
    rng = np.random.default_rng(2)
    for sc in (sp.a, sp.b):
        for i in sc.seq_ids:
            _, tab, ln = sc.orc.block_table(i)
            if ln % sc.T == 0:
                assert sc.orc.alloc_blocks(i, 1, oracle.LOCAL if sc is sp.a else oracle.LENT)[0] == 0
            assert sc.orc.set_seq_len(i, ln + 1) == 0
            sc.pl.lengths[i] = ln + 1
    for i in sp.seq_ids:
        n_have = len(sp.s.slice_get_block_table(i)[1])
        if n_have < len(sp.a.orc.block_table(i)[1]):
            assert sp.s.slice_alloc_blocks(i, 1, B.TIER_AUTO)[0] == B.OK
        assert sp.s.slice_set_seq_len(i, int(sp.a.pl.lengths[i])) == B.OK
        assert sp.s.slice_get_block_table(i)[1].tolist() == sp.a.orc.block_table(i)[1].tolist()
    k_all = synth.normal_bf16_bits(rng, (sp.L, sp.nseq, sp.Hkv, 128))
    v_all = synth.normal_bf16_bits(rng, (sp.L, sp.nseq, sp.Hkv, 128))
    for layer in range(sp.L):
        sc, l = sp.part(layer)
        assert sc.orc.append_kv(l, sc.seq_ids, k_all[layer], v_all[layer], sp.Hkv, 128, sc.local, sc.lent, None) == 0
    assert sp.s.slice_append_kv(B.ALL_LAYERS, sp.seq_ids, to_dev(k_all), to_dev(v_all), sp.main) == B.OK
    torch.cuda.synchronize()
    assert (kv_to_host(sp.local) == sp.a.local).all() and (kv_to_host(sp.lent) == sp.b.lent).all()
    sp.check_pass()
    # a request leaves by preemption; the others are unaffected
    gone = sp.seq_ids[1]
    assert sp.s.slice_preempt_seq(gone, B.PREEMPT_RECLAIM) == B.OK
    assert sp.s.slice_get_block_table(gone)[0] == B.ESTATE
