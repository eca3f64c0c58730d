"""Swap-out beside swap-in (Section 2.3: layers are swapped in and out cyclically, and what comes in
is matched by what goes out). With swap_out = 1 the ring is a write-back cache: a new token's row
goes to the staged copy only, and every pass writes each staged layer back to the lent arena while
that layer is attended to and the next one comes in. After a pass the lent arena must hold exactly
what the oracle's write-through append put there, and attention must be the oracle's throughout."""
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


@pytest.mark.parametrize("mode,swap,dependent", [(0, 1, False), (0, 2, False), (1, 1, False), (2, 1, False), (3, 1, False),
                                                 (1, 2, False), (2, 2, False), (3, 2, False), (0, 1, True), (0, 2, True)])
@pytest.mark.parametrize("ring", [2, 3])
def test_appended_rows_reach_the_lent_arena_through_the_ring(mode, swap, dependent, ring):
    """swap = 1: every staged block of a layer is written back; swap = 2: only the blocks that can have
    changed, the tail blocks."""
    from tests.gpu_helpers import GpuScenario, kv_to_host, to_dev
    wl = synth.Workload("swap", 5, 32, 8, 5, 17, 300, 0.5, ring_slots=ring)
    sc = Scenario(wl, 9, slack=16)
    g = GpuScenario(sc, pipeline_mode=mode, swap_out=swap, decode_ctas=12)
    seqs = np.asarray(sc.seq_ids, np.int32)
    rng = np.random.default_rng(3)

    def check_pass():
        g.out.zero_()
        k0 = g.s.slice_stats()["kernel_launches"]
        if dependent:      # the layer-dependent form of the pass: its queries released by the caller's stream
            caller = torch.cuda.Stream()
            assert g.s.slice_step_begin(seqs, g.q, sc.Hq, float(sc.sm_scale), g.out, True, g.main) == B.OK
            for layer in range(sc.L):
                assert g.s.slice_step_submit_q(layer, caller) == B.OK
        else:
            assert g.s.slice_decode_step(seqs, g.q, sc.Hq, float(sc.sm_scale), g.out, False, True, g.main, g.side) == B.OK
        torch.cuda.synchronize()
        g.device_ok()
        if mode == 0:      # the write-backs are part of the pass's one launch (plus, at most, gathers of the first layers)
            assert g.s.slice_stats()["kernel_launches"] - k0 <= 1 + ring
        got = g.out.view(torch.bfloat16).double().cpu().numpy()
        for layer in range(sc.L):
            rc, resolved, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
            _, ref, _ = oracle.paged_attention(sc.q[layer], sc.local[layer], sc.staging[layer % ring], resolved, sc.lengths(),
                                               sc.Hq, sc.Hkv, sc.D, sc.T, sc.sm_scale)
            assert attention_close(got[layer], ref, ATOL, RTOL)[0], layer

    check_pass()
    for step in range(3):
        for i in sc.seq_ids:                                 # every sequence grows by a token
            _, tab, ln = sc.orc.block_table(i)
            if ln % sc.T == 0:
                assert sc.orc.alloc_blocks(i, 1, oracle.AUTO)[0] == 0 and g.s.slice_alloc_blocks(i, 1, B.TIER_AUTO)[0] == 0
            assert sc.orc.set_seq_len(i, ln + 1) == 0 and g.s.slice_set_seq_len(i, ln + 1) == 0
            sc.pl.lengths[i] = ln + 1
        # the first layers are in the ring when the rows arrive: they land in the staged copies only
        staged_layers = list(range(min(ring, sc.L)))
        for layer in staged_layers:
            assert g.s.prefetch_layer(layer, sc.seq_ids, g.side) == B.OK
            assert sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)[0] == 0
        k_all = synth.normal_bf16_bits(rng, (sc.L, sc.nseq, sc.Hkv, sc.D))
        v_all = synth.normal_bf16_bits(rng, (sc.L, sc.nseq, sc.Hkv, sc.D))
        lent_before = kv_to_host(g.lent)
        for layer in range(sc.L):
            slot = sc.staging[layer % ring] if layer in staged_layers else None
            assert sc.orc.append_kv(layer, sc.seq_ids, k_all[layer], v_all[layer], sc.Hkv, sc.D, sc.local, sc.lent, slot) == 0
        assert g.s.slice_append_kv(B.ALL_LAYERS, sc.seq_ids, to_dev(k_all), to_dev(v_all), g.main) == B.OK
        torch.cuda.synchronize()
        lent_now = kv_to_host(g.lent)
        for layer in staged_layers:                          # write-back cache: the homes of staged blocks are untouched
            assert (lent_now[layer] == lent_before[layer]).all()
        assert (kv_to_host(g.local) == sc.local).all()
        check_pass()                                         # the pass reads the rows from the ring and writes them back
        assert (kv_to_host(g.lent) == sc.lent).all(), step
        assert (kv_to_host(g.local) == sc.local).all()
    check_pass()


def test_swap_out_with_the_layer_split():
    """The paper's own arrangement: half the layers remote, each of them brought in whole before its
    attention and written back whole while it is attended to."""
    from tests.gpu_helpers import kv_to_host, to_dev
    from tests.test_gpu_layer_split import SplitScenario
    sp = SplitScenario(6, 3, 4, pipeline_mode=2, swap_out=1, decode_ctas=12)
    sp.check_pass()
    before = sp.s.slice_stats()["kernel_launches"]
    sp.check_pass()
    # per pass: 6 layer launches, and for each of the 3 lent layers a write-back (gathers ride in the layer launches)
    assert sp.s.slice_stats()["kernel_launches"] - before >= 6 + 3
    assert (kv_to_host(sp.lent) == sp.b.lent).all()          # written back unchanged
