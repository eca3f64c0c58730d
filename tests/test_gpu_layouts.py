"""GPU parity with the slab allocator, layer groups and the three memory layouts of Section 4.2:
whatever order the arenas keep their blocks in, and whether a ring slot holds one layer or a group,
the staged bytes, the attention results, appended rows and migrated blocks are those of the oracle
(which works on canonical arenas; the tests carry bytes between the two orders through the oracle's
address map)."""
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


def _f64(t):
    return t.view(torch.bfloat16).double().cpu().numpy()


def _make(layout, slab, group, ring_groups=2, layers=8, seed=3, hq=16, hkv=4, **kw):
    from tests.gpu_helpers import GpuScenario
    wl = synth.Workload("lay", layers, hq, hkv, 6, 40, 900, 0.4, ring_slots=ring_groups * max(group, 1))
    sc = Scenario(wl, seed, slab_blocks=slab, slack=24)
    return sc, GpuScenario(sc, layout=layout, layer_group=group, **kw)


def _oracle_layer(sc, layer):
    rc, resolved, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
    assert rc == oracle.OK
    rc, ref, lse = oracle.paged_attention(sc.q[layer], sc.local[layer], sc.staging[layer % sc.wl.ring_slots], resolved,
                                          sc.lengths(), sc.Hq, sc.Hkv, sc.D, sc.T, sc.sm_scale)
    assert rc == oracle.OK
    return resolved, k, ref, lse


@pytest.mark.parametrize("layout,slab,group", [(0, 10, 1), (0, 10, 4), (1, 10, 4), (2, 10, 4), (1, 3, 2), (2, 3, 2), (2, 5, 1),
                                               (1, 1, 8), (2, 1, 8)])
def test_per_layer_calls_in_every_layout(layout, slab, group):
    """prefetch_layer + paged_decode layer by layer: staged bytes bit for bit, resolved tables,
    attention within tolerance, for slab sizes 1..10 and groups 1..8."""
    from tests.gpu_helpers import kv_to_host
    sc, g = _make(layout, slab, group)
    g.tables_equal_oracle()
    for layer in range(sc.L):
        resolved, k, ref, ref_lse = _oracle_layer(sc, layer)
        assert g.s.prefetch_layer(layer, sc.seq_ids, g.side) == B.OK
        out = torch.zeros_like(g.q[layer])
        lse = torch.zeros((sc.nseq, sc.Hq), dtype=torch.float32, device="cuda")
        assert g.s.paged_decode(layer, sc.seq_ids, g.q[layer], sc.Hq, float(sc.sm_scale), out, lse, g.main) == B.OK
        torch.cuda.synchronize()
        g.device_ok()
        rc, res_gpu, k_gpu = g.s.slice_get_resolved(sc.seq_ids)
        assert rc == B.OK and k_gpu == k and (res_gpu == resolved).all()
        slot = layer % sc.wl.ring_slots
        assert (kv_to_host(g.staging[slot, :k]) == sc.staging[slot, :k]).all()
        ok, max_abs, _ = attention_close(_f64(out), ref, ATOL, RTOL)
        assert ok, (layer, max_abs)
        assert np.abs(lse.double().cpu().numpy() - ref_lse).max() <= 1e-3


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
@pytest.mark.parametrize("layout,slab,group,layers,ring", [(2, 10, 4, 8, 2), (1, 10, 2, 8, 2), (0, 4, 3, 7, 2), (2, 4, 2, 6, 3),
                                                           (2, 10, 4, 12, 2), (1, 5, 4, 8, 1)])
def test_pipelines_fetch_one_group_ahead(mode, layout, slab, group, layers, ring):
    """slice_decode_step in all three pipelines: a ring slot holds a layer group, the pass fetches
    layer l + k while layer l is attended to and the first group of the next pass at its end. Three
    passes, every layer against the oracle; the bytes left in the ring are the oracle's."""
    from tests.gpu_helpers import kv_to_host
    sc, g = _make(layout, slab, group, ring_groups=ring, layers=layers, decode_ctas=12, pipeline_mode=mode)
    seqs = np.asarray(sc.seq_ids, np.int32)
    for rep in range(3):
        g.out.zero_()
        assert g.s.slice_decode_step(seqs, g.q, sc.Hq, float(sc.sm_scale), g.out, False, True, g.main, g.side) == B.OK
        torch.cuda.synchronize()
        g.device_ok()
        got = _f64(g.out)
        for layer in range(sc.L):
            _, _, ref, _ = _oracle_layer(sc, layer)
            ok, max_abs, _ = attention_close(got[layer], ref, ATOL, RTOL)
            assert ok, (rep, layer, max_abs)
    # what every layer slot holds now: the last layer that was fetched into it
    LS = sc.wl.ring_slots
    holder = {}
    for l in list(range(sc.L)) + list(range(min(group, sc.L))):          # pass order, then the next pass's first group
        holder[l % LS] = l
    for slot, layer in holder.items():
        rc, _, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
        assert (kv_to_host(g.staging[slot, :k]) == sc.staging[slot, :k]).all(), (slot, layer)


@pytest.mark.parametrize("layout,slab,group", [(1, 5, 2), (2, 5, 4), (0, 5, 2)])
def test_append_and_reclaim_move_the_right_bytes_in_every_layout(layout, slab, group):
    """A token is appended to every sequence in all layers at once (home block and staged copy), then
    the lender takes a third of the lent ids: the arenas, read back through the address map, and the
    tables equal the oracle's; attention afterwards is right."""
    from tests.gpu_helpers import to_dev
    sc, g = _make(layout, slab, group, layers=4, seed=8)
    seqs = np.asarray(sc.seq_ids, np.int32)
    assert g.s.slice_decode_step(seqs, g.q, sc.Hq, float(sc.sm_scale), g.out, False, True, g.main, g.side) == B.OK
    rng = np.random.default_rng(4)
    for i in sc.seq_ids:
        _, tab, ln = sc.orc.block_table(i)
        if ln % sc.T == 0:
            assert sc.orc.alloc_blocks(i, 1, oracle.AUTO)[0] == 0 and g.s.slice_alloc_blocks(i, 1, B.TIER_AUTO)[0] == 0
        assert sc.orc.set_seq_len(i, ln + 1) == 0 and g.s.slice_set_seq_len(i, ln + 1) == 0
        sc.pl.lengths[i] = ln + 1
    g.tables_equal_oracle()
    k_all = synth.normal_bf16_bits(rng, (sc.L, sc.nseq, sc.Hkv, sc.D))
    v_all = synth.normal_bf16_bits(rng, (sc.L, sc.nseq, sc.Hkv, sc.D))
    for layer in range(sc.L):
        assert sc.orc.append_kv(layer, sc.seq_ids, k_all[layer], v_all[layer], sc.Hkv, sc.D, sc.local, sc.lent, None) == 0
    assert g.s.slice_append_kv(B.ALL_LAYERS, sc.seq_ids, to_dev(k_all), to_dev(v_all), g.main) == B.OK
    torch.cuda.synchronize()
    assert (g.from_layout(g.local, True) == sc.local).all() and (g.from_layout(g.lent, False) == sc.lent).all()
    take = sc.orc.lent_capacity // 3
    rc, mig = sc.orc.reclaim(take, sc.local, sc.lent)
    rc2, mig2 = g.s.slice_reclaim(take, g.main)
    assert rc == rc2 == 0 and mig == mig2 and mig > 0
    torch.cuda.synchronize()
    g.device_ok()
    g.tables_equal_oracle()
    local_gpu, lent_gpu = g.from_layout(g.local, True), g.from_layout(g.lent, False)
    for i in sc.seq_ids:
        _, tab, _ = sc.orc.block_table(i)
        for l in range(sc.L):
            for e in tab.tolist():
                a = local_gpu[l, e] if e >= 0 else lent_gpu[l, ~e]
                b = sc.local[l, e] if e >= 0 else sc.lent[l, ~e]
                assert (a == b).all()
    g.out.zero_()
    assert g.s.slice_decode_step(seqs, g.q, sc.Hq, float(sc.sm_scale), g.out, False, True, g.main, g.side) == B.OK
    torch.cuda.synchronize()
    g.device_ok()
    got = _f64(g.out)
    for layer in range(sc.L):
        _, _, ref, _ = _oracle_layer(sc, layer)
        assert attention_close(got[layer], ref, ATOL, RTOL)[0], layer


@pytest.mark.parametrize("hq,hkv", [(4, 1), (8, 2), (2, 2)])
@pytest.mark.parametrize("layout,slab,group", [(0, 10, 1), (2, 10, 4), (0, 0, 1)])
def test_small_blocks_are_gathered_in_runs(hq, hkv, layout, slab, group):
    """With 1 or 2 KV heads a block is 8 or 16 KB; where the slab allocator has kept a sequence's lent
    blocks together, the fused gather moves up to 64 KB of neighbouring blocks per copy unit. The
    staged bytes and the attention must not depend on how the units were cut (slab 0: seeded free
    order, hardly any neighbours; slabs: long runs)."""
    from tests.gpu_helpers import kv_to_host
    sc, g = _make(layout, slab, group, layers=8, hq=hq, hkv=hkv, decode_ctas=10)
    seqs = np.asarray(sc.seq_ids, np.int32)
    for rep in range(2):
        g.out.zero_()
        assert g.s.slice_decode_step(seqs, g.q, sc.Hq, float(sc.sm_scale), g.out, False, True, g.main, g.side) == B.OK
        torch.cuda.synchronize()
        g.device_ok()
        got = _f64(g.out)
        for layer in range(sc.L):
            _, _, ref, _ = _oracle_layer(sc, layer)
            ok, max_abs, _ = attention_close(got[layer], ref, ATOL, RTOL)
            assert ok, (rep, layer, max_abs)
    LS = sc.wl.ring_slots
    holder = {}
    for l in list(range(sc.L)) + list(range(min(max(group, 1), sc.L))):
        holder[l % LS] = l
    for slot, layer in holder.items():
        rc, _, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
        assert (kv_to_host(g.staging[slot, :k]) == sc.staging[slot, :k]).all(), (slot, layer)
