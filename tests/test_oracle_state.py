"""Pins of the oracle's integer state machine, gather and reclaim migration: hand-worked cases
(tests/golden), tag round trips, byte/logical-order preservation and invariants under random
operation sequences. CPU only."""
import json
import os

import numpy as np
import pytest

import oracle
from oracle import AUTO, LENT, LOCAL
from paper_2609_27040_b200 import synth
from tests.helpers import Scenario

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
WL1 = synth.WORKLOADS["single_layer_mha"]
SMALL3 = synth.Workload("small3", 3, 8, 8, 6, 20, 200, 0.5, ring_slots=2)


def _tiny(local=4, lent=4, phys=None, **kw):
    return oracle.OracleSlice(2, 16, 64, local, lent, phys, 2, 8, max_seqs=8, max_blocks_per_seq=8, **kw)


def test_hand_worked_allocation_order():
    """Golden: allocation takes free local memory first and only then the lent part
    (Section 4.1); a freed sequence's blocks come back in ascending logical order."""
    with open(os.path.join(GOLDEN, "alloc_reclaim_worked_example.json")) as f:
        gold = json.load(f)
    o = _tiny()
    trace = []
    for op in gold["ops"]:
        if op[0] == "alloc":
            rc, ent = o.alloc_blocks(op[1], op[2], op[3])
            trace.append([rc, ent.tolist() if rc == oracle.OK else []])
        elif op[0] == "free":
            trace.append([o.free_seq(op[1]), []])
        elif op[0] == "reclaim":
            rc, mig = o.reclaim(op[1], None, None)
            trace.append([rc, [mig]])
        elif op[0] == "lend":
            trace.append([o.lend(op[1]), []])
    assert trace == gold["expected"]
    for seq, tab in gold["final_tables"].items():
        assert o.block_table(int(seq))[1].tolist() == tab
    assert o.free_stack(LOCAL).tolist() == gold["final_free_local"]
    assert o.free_stack(LENT).tolist() == gold["final_free_lent"]
    assert o.lent_capacity == gold["final_lent_capacity"]


def test_enospc_and_bad_calls_leave_state_untouched():
    o = _tiny()
    assert o.alloc_blocks(0, 3, AUTO)[0] == oracle.OK
    before = (o.block_table(0)[1].tolist(), o.free_stack(LOCAL).tolist(), o.free_stack(LENT).tolist())
    assert o.alloc_blocks(1, 6, AUTO)[0] == oracle.E_NOSPC      # 5 free in total
    assert o.alloc_blocks(0, 6, AUTO)[0] == oracle.E_INVAL      # 3 + 6 > 8 blocks per sequence
    assert o.alloc_blocks(1, 2, LOCAL)[0] == oracle.E_NOSPC     # 1 free local
    assert o.alloc_blocks(1, 5, LENT)[0] == oracle.E_NOSPC
    assert o.num_seqs == 1                                       # failed calls create no sequence
    assert o.free_seq(5) == oracle.E_STATE
    assert o.set_seq_len(0, 49) == oracle.E_INVAL               # 3 blocks hold 48 tokens
    assert o.set_seq_len(0, 48) == oracle.OK
    after = (o.block_table(0)[1].tolist(), o.free_stack(LOCAL).tolist(), o.free_stack(LENT).tolist())
    assert before == after


def test_seeded_free_orders_are_followed():
    lo = np.array([2, 0, 3, 1], np.uint32)
    ro = np.array([5, 1, 0, 4, 3, 2], np.uint32)        # physical 6, capacity 4: ids 4,5 are not lent yet
    o = _tiny(4, 4, 6, local_free_order=lo, lent_free_order=ro)
    assert o.alloc_blocks(0, 4, LOCAL)[1].tolist() == [2, 0, 3, 1]
    assert o.alloc_blocks(1, 4, LENT)[1].tolist() == [~1, ~0, ~3, ~2]
    assert o.lend(2) == oracle.OK
    assert o.alloc_blocks(2, 2, AUTO)[1].tolist() == [~4, ~5]


# ------------------------------------------------------------------------------------------------
def _tag_arena(arr, tier):
    """Unique 64-bit tag per (tier, layer, block, plane): every block's content names its origin."""
    L, nb = arr.shape[:2]
    v = arr.reshape(L, nb, 2, -1).view(np.uint64)
    l, b, p = np.meshgrid(np.arange(L), np.arange(nb), np.arange(2), indexing="ij")
    v[...] = ((tier << 60) | (l.astype(np.uint64) << 40) | (b.astype(np.uint64) << 8) | p.astype(np.uint64))[..., None]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_gather_tags_positions_and_resolved(seed):
    """P6: through the resolved table every (seq, block) yields the bytes of its home block; staged
    positions are a bijection onto [0, k); the resolved table does not depend on the layer."""
    sc = Scenario(SMALL3, seed)
    _tag_arena(sc.local, 1)
    _tag_arena(sc.lent, 2)
    sc.staging[...] = 0
    first = None
    for layer in range(sc.L):
        rc, resolved, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
        assert rc == oracle.OK
        slot = layer % sc.wl.ring_slots
        seen = []
        n_lent = 0
        for pos, i in enumerate(sc.seq_ids):
            _, table, ln = sc.orc.block_table(i)
            nb = synth.blocks_for(ln, sc.T)
            for b in range(nb):
                e, r = int(table[b]), int(resolved[pos, b])
                if e >= 0:
                    assert r == e
                else:
                    n_lent += 1
                    assert r < 0
                    seen.append(~r)
                    assert (sc.staging[slot, ~r] == sc.lent[layer, ~e]).all()
        assert k == n_lent and sorted(seen) == list(range(k))
        assert seen == list(range(k))          # canonical order: batch position, then logical index
        if first is None:
            first = resolved.copy()
        assert (resolved == first).all()


def test_gather_skips_blocks_past_length_and_checks_capacity():
    o = oracle.OracleSlice(1, 16, 64, 4, 8, 8, 2, 2, max_seqs=4, max_blocks_per_seq=8)
    assert o.alloc_blocks(0, 4, LENT)[0] == oracle.OK
    o.set_seq_len(0, 17)                        # two blocks in use, two allocated ahead
    lent = np.arange(8 * 64, dtype=np.uint8).reshape(1, 8, 64)
    stg = np.zeros((2, 2, 64), np.uint8)
    rc, res, k = o.gather(0, [0], lent, stg)
    assert rc == oracle.OK and k == 2 and res[0, :2].tolist() == [~0, ~1]
    assert (stg[0, 0] == lent[0, 0]).all() and (stg[0, 1] == lent[0, 1]).all()
    o.set_seq_len(0, 33)                        # three lent blocks > slot capacity 2
    before = stg.copy()
    rc, _, _ = o.gather(0, [0], lent, stg)
    assert rc == oracle.E_STAGING and (stg == before).all()
    assert o.gather(0, [0, 0], lent, stg)[0] == oracle.E_INVAL      # duplicate sequence
    assert o.gather(0, [3], lent, stg)[0] == oracle.E_STATE


def test_gather_identity_is_memcpy_and_scatter_round_trips():
    """P10: with identity free order and an all-lent sequence the gather is a plain copy; writing
    the staged blocks back to their homes leaves the lent arena unchanged."""
    rng = np.random.default_rng(3)
    nb, bb = 12, 256
    o = oracle.OracleSlice(2, 16, bb, 2, nb, nb, 2, nb, max_seqs=4, max_blocks_per_seq=16)
    o.alloc_blocks(0, nb, LENT)
    o.set_seq_len(0, nb * 16)
    lent = rng.integers(0, 256, size=(2, nb, bb), dtype=np.uint8)
    stg = np.zeros((2, nb, bb), np.uint8)
    for layer in range(2):
        assert o.gather(layer, [0], lent, stg)[0] == oracle.OK
        assert stg[layer % 2].tobytes() == lent[layer].tobytes()
    keep = lent.copy()
    lent[...] = 0
    for layer in range(2):
        assert o.scatter(layer, [0], stg, lent) == oracle.OK
    assert (lent == keep).all()


# ------------------------------------------------------------------------------------------------
def _check_invariants(o: oracle.OracleSlice, seqs, local_blocks):
    used_local, used_lent = [], []
    for s in seqs:
        rc, tab, _ = o.block_table(s)
        assert rc == oracle.OK
        for e in tab.tolist():
            (used_local if e >= 0 else used_lent).append(e if e >= 0 else ~e)
    fl, fr = o.free_stack(LOCAL).tolist(), o.free_stack(LENT).tolist()
    assert len(set(used_local)) == len(used_local) and len(set(used_lent)) == len(used_lent)
    assert sorted(used_local + fl) == list(range(local_blocks))            # conservation, disjoint
    assert sorted(used_lent + fr) == list(range(o.lent_capacity))


@pytest.mark.parametrize("seed", [0, 1])
def test_migration_preserves_bytes_and_logical_order(seed):
    """P7: reclaim moves every byte of the victims, keeps table lengths and logical order, leaves
    no entry at or above the cut, and reclaim(all) leaves nothing lent."""
    sc = Scenario(SMALL3, seed, slack=64, lent_extra_physical=5)
    before = {(i, l): sc.logical_view(i, l).copy() for i in sc.seq_ids for l in range(sc.L)}
    lens_before = {i: len(sc.orc.block_table(i)[1]) for i in sc.seq_ids}
    cap = sc.orc.lent_capacity
    take = cap // 3
    rc, mig = sc.orc.reclaim(take, sc.local, sc.lent)
    assert rc == oracle.OK and mig > 0
    cut = cap - take
    assert sc.orc.lent_capacity == cut
    for i in sc.seq_ids:
        tab = sc.orc.block_table(i)[1]
        assert len(tab) == lens_before[i]
        assert all((e >= 0) or (~e < cut) for e in tab.tolist())
        for l in range(sc.L):
            assert (sc.logical_view(i, l) == before[(i, l)]).all()
    _check_invariants(sc.orc, sc.seq_ids, sc.pl.local_blocks)
    rc, mig2 = sc.orc.reclaim(0xFFFFFFFF, sc.local, sc.lent)
    assert rc == oracle.OK
    assert sc.orc.lent_capacity == 0 and sc.orc.free_stack(LENT).size == 0
    for i in sc.seq_ids:
        assert (sc.orc.block_table(i)[1] >= 0).all()
        for l in range(sc.L):
            assert (sc.logical_view(i, l) == before[(i, l)]).all()
    rc, _, k = sc.orc.gather(0, sc.seq_ids, sc.lent, sc.staging)
    assert rc == oracle.OK and k == 0


def test_reclaim_compacts_into_lower_lent_ids_when_local_is_full():
    o = _tiny(2, 6)
    assert o.alloc_blocks(0, 2, LOCAL)[0] == oracle.OK
    assert o.alloc_blocks(1, 6, LENT)[1].tolist() == [~0, ~1, ~2, ~3, ~4, ~5]
    assert o.free_seq(1) == oracle.OK
    assert o.alloc_blocks(2, 2, LENT)[1].tolist() == [~0, ~1]
    assert o.alloc_blocks(3, 2, LENT)[1].tolist() == [~2, ~3]
    assert o.alloc_blocks(4, 2, LENT)[1].tolist() == [~4, ~5]
    assert o.free_seq(2) == oracle.OK                       # ids 0,1 free; local full
    lent = np.arange(2 * 6 * 64, dtype=np.uint16).reshape(2, 6, 64).astype(np.uint8)
    lent[...] = (np.arange(2 * 6)[:, None] + 1).reshape(2, 6, 1)
    local = np.zeros((2, 2, 64), np.uint8)
    rc, mig = o.reclaim(2, local, lent)                     # cut = 4: victims 4,5 -> smallest free 0,1
    assert rc == oracle.OK and mig == 2
    assert o.block_table(4)[1].tolist() == [~0, ~1]
    assert (lent[:, 0] == lent[:, 4]).all() and (lent[:, 1] == lent[:, 5]).all()
    assert o.free_stack(LENT).size == 0 and o.lent_capacity == 4
    # no room left: reclaim of two more ids must fail and change nothing
    tabs = [o.block_table(s)[1].tolist() for s in (0, 3, 4)]
    rc, _ = o.reclaim(2, local, lent)
    assert rc == oracle.E_NOSPC
    assert tabs == [o.block_table(s)[1].tolist() for s in (0, 3, 4)] and o.lent_capacity == 4


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_allocator_invariants_under_random_ops(seed):
    """P8: conservation, injectivity, failed calls change nothing, AUTO never uses the lent part
    while local memory is free."""
    rng = np.random.default_rng(seed)
    LB, RB, PH = 12, 10, 14
    o = oracle.OracleSlice(1, 16, 64, LB, RB, PH, 2, 8, max_seqs=6, max_blocks_per_seq=9,
                           local_free_order=synth.free_order(rng, LB), lent_free_order=synth.free_order(rng, PH))
    live = set()

    def snapshot():
        return ({s: o.block_table(s)[1].tolist() for s in live}, o.free_stack(LOCAL).tolist(),
                o.free_stack(LENT).tolist(), o.lent_capacity)

    for _ in range(4000):
        op = rng.integers(0, 10)
        snap = snapshot()
        if op < 5:
            s, n, hint = int(rng.integers(0, 8)), int(rng.integers(0, 5)), int(rng.integers(0, 3))
            n_free_local = len(snap[1])
            rc, ent = o.alloc_blocks(s, n, hint)
            if rc == oracle.OK:
                live.add(s)
                if hint == AUTO:
                    n_loc = int((ent >= 0).sum())
                    assert n_loc == min(n, n_free_local) and (ent[:n_loc] >= 0).all()
            else:
                assert snapshot() == snap
        elif op < 7 and live:
            s = int(rng.choice(sorted(live)))
            assert o.free_seq(s) == oracle.OK
            live.discard(s)
        elif op == 7:
            rc, _ = o.reclaim(int(rng.integers(0, 5)), None, None)
            if rc != oracle.OK:
                assert rc == oracle.E_NOSPC and snapshot() == snap
        elif op == 8:
            rc = o.lend(int(rng.integers(0, 4)))
            if rc != oracle.OK:
                assert snapshot() == snap
        else:
            assert o.free_seq(99) == oracle.E_STATE and snapshot() == snap
        _check_invariants(o, sorted(live), LB)
        assert o.num_seqs == len(live)


def test_append_writes_home_and_staged_copy():
    wl = synth.Workload("app", 2, 8, 8, 3, 17, 60, 0.5)
    sc = Scenario(wl, 5, slack=8)
    rng = np.random.default_rng(9)
    layer = 1
    # grow every sequence by one token (allocate a block when the last one is full)
    for i in sc.seq_ids:
        _, tab, ln = sc.orc.block_table(i)
        if ln % sc.T == 0:
            assert sc.orc.alloc_blocks(i, 1, AUTO)[0] == oracle.OK
        assert sc.orc.set_seq_len(i, ln + 1) == oracle.OK
    rc, resolved, k = sc.orc.gather(layer, sc.seq_ids, sc.lent, sc.staging)
    assert rc == oracle.OK
    k_new = synth.normal_bf16_bits(rng, (sc.nseq, sc.Hkv, sc.D))
    v_new = synth.normal_bf16_bits(rng, (sc.nseq, sc.Hkv, sc.D))
    local0, lent0, stg0 = sc.local.copy(), sc.lent.copy(), sc.staging.copy()
    slot = layer % wl.ring_slots
    assert sc.orc.append_kv(layer, sc.seq_ids, k_new, v_new, sc.Hkv, sc.D, sc.local, sc.lent,
                            sc.staging[slot]) == oracle.OK
    changed = 0
    for pos, i in enumerate(sc.seq_ids):
        _, tab, ln = sc.orc.block_table(i)
        t = ln - 1
        b, r = t // sc.T, t % sc.T
        e = int(tab[b])
        home = sc.local[layer, e] if e >= 0 else sc.lent[layer, ~e]
        assert (home[0, r] == k_new[pos]).all() and (home[1, r] == v_new[pos]).all()
        changed += 2 * sc.Hkv * sc.D
        if e < 0:
            st = sc.staging[slot, ~int(resolved[pos, b])]
            assert (st[0, r] == k_new[pos]).all() and (st[1, r] == v_new[pos]).all()
            assert (st == home).all()
    # nothing else moved
    assert ((sc.local != local0).sum() + (sc.lent != lent0).sum()) <= changed
    assert (sc.staging[1 - slot] == stg0[1 - slot]).all()
