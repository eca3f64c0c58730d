"""Pins of the oracle's reclaim by preemption (Section 4.1), its victim rule (Section 4.2.1: the
slab with the fewest active requests), the cap that follows a preemption (Section 5.3) and the
counters by cause (Section 6.6): hand-worked cases, properties checked against twin states that
take the plain reclaim instead, a brute-force count of the requests per slab, and the paper's
back-and-forth scenario with and without the cap. CPU only."""
import numpy as np
import pytest

import oracle
from oracle import AUTO, LENT, LOCAL


def _slice(local=4, lent=12, **kw):
    return oracle.OracleSlice(2, 16, 64, local, lent, None, 2, 16, max_seqs=16, max_blocks_per_seq=16, **kw)


def _fill_worked_example(o):
    """Local part full (request 0); lent ids 0..11 in three slabs of four:
    slab 0 = request 1 alone; slab 1 = requests 2, 3, 4; slab 2 = requests 4, 5."""
    assert o.alloc_blocks(0, 4, LOCAL)[0] == oracle.OK
    assert o.alloc_blocks(1, 4, LENT)[1].tolist() == [~0, ~1, ~2, ~3]
    assert o.alloc_blocks(2, 2, LENT)[1].tolist() == [~4, ~5]
    assert o.alloc_blocks(3, 1, LENT)[1].tolist() == [~6]
    assert o.alloc_blocks(4, 2, LENT)[1].tolist() == [~7, ~8]
    assert o.alloc_blocks(5, 3, LENT)[1].tolist() == [~9, ~10, ~11]


def test_hand_worked_victim_is_the_slab_with_the_fewest_requests():
    """The lender takes ids 8..11 back (four blocks in use there, no free place anywhere). Evicting
    from the reclaimed slab would cost two requests (4 and 5); slab 0 holds one request whose four
    blocks are exactly the room needed, so request 1 alone is preempted and the rest compacts."""
    o = _slice()
    _fill_worked_example(o)
    assert o.reclaim(4, None, None)[0] == oracle.E_NOSPC            # the migration alone has no room
    lent = np.zeros((2, 12, 64), np.uint8)
    lent[...] = (np.arange(24).reshape(2, 12, 1) + 1)
    local = np.zeros((2, 4, 64), np.uint8)
    before = lent.copy()
    rc, victims, mig = o.reclaim_preempt(4, 4, local, lent)
    assert rc == oracle.OK and victims == [1] and mig == 4
    assert o.lent_capacity == 8 and o.num_seqs == 5
    assert o.block_table(4)[1].tolist() == [~7, ~0]                  # id 8 -> smallest free id 0
    assert o.block_table(5)[1].tolist() == [~1, ~2, ~3]              # ids 9, 10, 11 -> 1, 2, 3
    assert o.block_table(2)[1].tolist() == [~4, ~5] and o.block_table(3)[1].tolist() == [~6]
    for layer in range(2):
        assert (lent[layer, 0] == before[layer, 8]).all()
        for k in range(3):
            assert (lent[layer, 1 + k] == before[layer, 9 + k]).all()
    assert o.block_table(1)[0] == oracle.E_STATE
    st = o.preempt_state()
    assert st["preempt_reclaim"] == 1 and st["preempt_oom"] == 0


def test_ties_go_to_the_highest_slab_and_rounds_repeat_until_there_is_room():
    """Slabs of two ids; every slab holds one request, so each round takes the highest slab that
    still holds one: request 6 (ids 10, 11), then request 5 (ids 8, 9), then request 4 (ids 6, 7):
    all of them lie in the reclaimed range 6..11, so nothing is left to move."""
    o = _slice(local=2, lent=12)
    assert o.alloc_blocks(0, 2, LOCAL)[0] == oracle.OK
    for q in range(1, 7):
        assert o.alloc_blocks(q, 2, LENT)[1].tolist() == [~(2 * q - 2), ~(2 * q - 1)]
    rc, victims, mig = o.reclaim_preempt(6, 2, None, None)
    assert rc == oracle.OK and victims == [6, 5, 4] and mig == 0
    assert o.lent_capacity == 6 and sorted(o.free_stack(LENT).tolist()) == []
    # With room for some of the range, fewer rounds are needed: same start, two ids free below.
    o = _slice(local=2, lent=12)
    assert o.alloc_blocks(0, 2, LOCAL)[0] == oracle.OK
    for q in range(1, 7):
        assert o.alloc_blocks(q, 2, LENT)[0] == oracle.OK
    assert o.free_seq(1) == oracle.OK                                 # ids 0, 1 free
    rc, victims, mig = o.reclaim_preempt(6, 2, None, None)
    assert rc == oracle.OK and victims == [6, 5] and mig == 2        # request 4 moves to ids 0, 1
    assert sorted(~e for e in o.block_table(4)[1].tolist()) == [0, 1]


def test_bad_arguments_change_nothing():
    o = _slice()
    _fill_worked_example(o)
    tabs = {q: o.block_table(q)[1].tolist() for q in range(6)}
    assert o.reclaim_preempt(4, 0, None, None)[0] == oracle.E_INVAL   # slab of no blocks
    assert o.reclaim_preempt(4, 4, None, None, max_victims=0)[0] == oracle.E_INVAL
    assert tabs == {q: o.block_table(q)[1].tolist() for q in range(6)} and o.lent_capacity == 12
    assert o.preempt_seq(0, 3) == oracle.E_INVAL and o.preempt_seq(77, 1) == oracle.E_STATE
    assert o.preempt_state()["preempt_reclaim"] == 0


def _slab_counts(tables, slab, lent_cap):
    """Brute force: distinct requests with a block in each slab of the lent range."""
    n = (lent_cap + slab - 1) // slab
    sets = [set() for _ in range(n)]
    for q, tab in tables.items():
        for e in tab:
            if e < 0:
                sets[(~e) // slab].add(q)
    return [len(x) for x in sets], sets


def _rounds(victims, sets):
    """Splits the eviction order into rounds: each round is every not yet evicted request of one
    slab, in ascending id order. Returns [(slab, [requests])]; where several slabs fit, the highest."""
    out, evicted, k = [], set(), 0
    while k < len(victims):
        fit = [sl for sl, st in enumerate(sets)
               if st - evicted and sorted(st - evicted) == victims[k:k + len(st - evicted)]]
        assert fit, (victims, sets)
        sl = max(fit)
        grp = sorted(sets[sl] - evicted)
        out.append((sl, grp))
        evicted |= set(grp)
        k += len(grp)
    return out


@pytest.mark.parametrize("seed", range(6))
def test_properties_against_twins_that_reclaim_without_preemption(seed):
    """Three states take the same random calls. Where the plain reclaim succeeds the preempting one
    evicts nobody. Where it fails for lack of room, the preempting one succeeds; every round of its
    evictions empties a slab whose count of requests (brute force over the tables) is the smallest
    at that moment, the highest such slab; before each round the plain reclaim still had no room
    (replayed on the third state); evicting the same requests by hand and reclaiming plainly ends
    in the same tables and free lists; survivors keep their bytes, in logical order, below the cut."""
    rng = np.random.default_rng(seed)
    LB, RB, L, BB = 10, 24, 2, 64
    slab = int(rng.integers(1, 7))

    def fresh():
        return oracle.OracleSlice(L, 16, BB, LB, RB, None, 2, RB, max_seqs=12, max_blocks_per_seq=10)

    a, b, c = fresh(), fresh(), fresh()
    local = rng.integers(0, 255, (L, LB, BB), dtype=np.uint8)
    lent = rng.integers(0, 255, (L, RB, BB), dtype=np.uint8)
    live, preempted, no_room = set(), 0, 0

    def view(o, q):
        return [(local[:, e] if e >= 0 else lent[:, ~e]).copy() for e in o.block_table(q)[1].tolist()]

    def same_state(x, y):
        return (all(x.block_table(q)[1].tolist() == y.block_table(q)[1].tolist() for q in live)
                and x.free_stack(LOCAL).tolist() == y.free_stack(LOCAL).tolist()
                and x.free_stack(LENT).tolist() == y.free_stack(LENT).tolist()
                and x.lent_capacity == y.lent_capacity and x.num_seqs == y.num_seqs == len(live))

    for _ in range(400):
        op = rng.integers(0, 10)
        if op < 6:
            q, n = int(rng.integers(0, 12)), int(rng.integers(1, 5))
            rcs = [o.alloc_blocks(q, n, AUTO)[0] for o in (a, b, c)]
            assert rcs[0] == rcs[1] == rcs[2]
            if rcs[0] == oracle.OK:
                live.add(q)
        elif op < 7 and live:
            q = int(rng.choice(sorted(live)))
            assert [o.free_seq(q) for o in (a, b, c)] == [oracle.OK] * 3
            live.discard(q)
        elif op < 8:
            n = int(rng.integers(0, 5))
            assert a.lend(n) == b.lend(n) == c.lend(n)
        else:
            take = int(rng.integers(1, 9))
            cap0 = a.lent_capacity
            cut = cap0 - min(take, cap0)
            tables = {q: a.block_table(q)[1].tolist() for q in live}
            views = {q: view(a, q) for q in live}
            rc_b, _ = b.reclaim(take, None, None)
            rc, victims, mig = a.reclaim_preempt(take, slab, local, lent)
            assert rc == oracle.OK and a.lent_capacity == cut
            assert (rc_b == oracle.OK) == (victims == [])
            assert len(set(victims)) == len(victims) and set(victims) <= live
            if victims:
                assert rc_b == oracle.E_NOSPC
                no_room += 1
                _, sets = _slab_counts(tables, slab, cap0)
                evicted = set()
                for sl, grp in _rounds(victims, sets):
                    left = [len(st - evicted) for st in sets]
                    least = min(x for x in left if x > 0)
                    assert left[sl] == least and sl == max(k for k, x in enumerate(left) if x == least)
                    assert c.reclaim(take, None, None)[0] == oracle.E_NOSPC      # not yet enough
                    for q in grp:
                        assert c.free_seq(q) == oracle.OK and b.free_seq(q) == oracle.OK
                    evicted |= set(grp)
                assert b.reclaim(take, None, None) == (oracle.OK, mig)
                live -= set(victims)
                preempted += len(victims)
            assert c.reclaim(take, None, None)[0] == oracle.OK
            for q in live:
                tab = a.block_table(q)[1].tolist()
                assert len(tab) == len(tables[q]) and all(e >= 0 or ~e < cut for e in tab)
                for x, y in zip(view(a, q), views[q]):
                    assert (x == y).all()
            assert a.preempt_state()["preempt_reclaim"] == preempted
        assert same_state(a, b) and same_state(a, c)
    assert no_room >= 3


# ------------------------------------------------------------------------------------------------
# The cap after a preemption (Section 5.3)
# ------------------------------------------------------------------------------------------------
def _borrower_at_ten_blocks(window):
    """Static share 4 blocks (the local part), 8 lent; the user holds 10: requests 0 (4 local),
    1 (lent 0..2), 2 (lent 3, 4), 3 (lent 5)."""
    o = _slice(local=4, lent=8)
    assert o.set_preempt_window(window) == oracle.OK
    assert o.alloc_blocks(0, 4, LOCAL)[0] == oracle.OK
    assert o.alloc_blocks(1, 3, LENT)[0] == oracle.OK
    assert o.alloc_blocks(2, 2, LENT)[0] == oracle.OK
    assert o.alloc_blocks(3, 1, LENT)[0] == oracle.OK
    return o


def test_cap_time_line():
    """k0, a lower k1 inside the window, and the lift after T, on a hand-worked time line."""
    o = _borrower_at_ten_blocks(window=100)
    assert o.set_time(5) == oracle.OK
    # The lender takes 4 ids (4..7): ids 4 and 5 are in use, ids 6, 7 free but in the range: no
    # room. Slabs of 4: slab 0 = {1, 2}, slab 1 = {2, 3}; tie -> slab 1: requests 2 and 3 go.
    rc, victims, mig = o.reclaim_preempt(4, 4, None, None)
    assert rc == oracle.OK and victims == [2, 3] and mig == 0
    st = o.preempt_state()
    assert st["cap_level"] == 7 and st["cap_until"] == 105 and st["preempt_reclaim"] == 2   # 10 -> 7 blocks
    assert o.alloc_blocks(4, 1, AUTO)[0] == oracle.E_CAPPED          # 7 + 1 > 7, though id 3 is free
    assert o.num_seqs == 2                                           # a refused call creates nothing
    assert o.alloc_blocks(4, 0, AUTO)[0] == oracle.OK               # an empty request is not growth
    assert o.free_seq(4) == oracle.OK
    assert o.free_seq(1) == oracle.OK                                # completion: 4 blocks held
    assert o.alloc_blocks(5, 3, AUTO)[0] == oracle.OK               # back to 7: allowed
    assert o.alloc_blocks(5, 1, AUTO)[0] == oracle.E_CAPPED
    # t = 50: the engine preempts request 5 for the lender at 7 > 4 blocks: k1 = 4 < k0 = 7.
    assert o.set_time(50) == oracle.OK
    assert o.preempt_seq(5, oracle.PREEMPT_RECLAIM) == oracle.OK
    st = o.preempt_state()
    assert st["cap_level"] == 4 and st["cap_until"] == 150 and st["preempt_reclaim"] == 3
    assert o.set_time(120) == oracle.OK                              # past the first window, inside the second
    assert o.alloc_blocks(6, 1, AUTO)[0] == oracle.E_CAPPED
    assert o.set_time(149) == oracle.OK and o.alloc_blocks(6, 1, AUTO)[0] == oracle.E_CAPPED
    assert o.set_time(150) == oracle.OK                              # T expired: lifted
    assert o.preempt_state()["cap_level"] == 0 and o.preempt_state()["cap_until"] == 0
    assert o.alloc_blocks(6, 4, AUTO)[0] == oracle.OK
    assert o.set_time(149) == oracle.E_INVAL and o.preempt_state()["now"] == 150


def test_what_sets_no_cap():
    # window 0: never
    o = _borrower_at_ten_blocks(window=0)
    assert o.reclaim_preempt(4, 4, None, None)[1] == [2, 3]
    assert o.preempt_state()["cap_level"] == 0 and o.alloc_blocks(4, 1, AUTO)[0] == oracle.OK
    # a preemption for lack of memory counts, and caps nothing
    o = _borrower_at_ten_blocks(window=100)
    assert o.preempt_seq(3, oracle.PREEMPT_OOM) == oracle.OK
    st = o.preempt_state()
    assert st["preempt_oom"] == 1 and st["preempt_reclaim"] == 0 and st["cap_level"] == 0
    assert o.alloc_blocks(3, 1, AUTO)[0] == oracle.OK
    # a reclaim that needs no eviction caps nothing
    o = _borrower_at_ten_blocks(window=100)
    assert o.reclaim_preempt(2, 4, None, None)[1] == []               # ids 6, 7 are free
    assert o.preempt_state()["cap_level"] == 0
    # a preemption at or below the static share caps nothing: 3 lent blocks held, local part empty
    o = _slice(local=4, lent=8)
    o.set_preempt_window(100)
    assert o.alloc_blocks(1, 3, LENT)[0] == oracle.OK
    assert o.preempt_seq(1, oracle.PREEMPT_RECLAIM) == oracle.OK
    assert o.preempt_state()["preempt_reclaim"] == 1 and o.preempt_state()["cap_level"] == 0
    # a later preemption at a higher level does not raise the cap
    o = _borrower_at_ten_blocks(window=100)
    assert o.preempt_seq(1, oracle.PREEMPT_RECLAIM) == oracle.OK      # 10 -> 7
    assert o.preempt_seq(2, oracle.PREEMPT_RECLAIM) == oracle.OK      # 7 -> 5
    assert o.preempt_state()["cap_level"] == 5
    assert o.free_seq(3) == oracle.OK and o.alloc_blocks(7, 1, AUTO)[0] == oracle.OK   # 4 -> 5
    assert o.alloc_blocks(7, 1, AUTO)[0] == oracle.E_CAPPED


def _back_and_forth(window, rounds=12):
    """Section 5.3's cycle: user A grows past its share whenever there is room; the lender B takes
    4 ids back, releases them a little later, and so on. Returns A's preemptions by reclamation."""
    o = _slice(local=4, lent=8)
    o.set_preempt_window(window)
    next_id, t = 0, 0
    for _ in range(rounds):
        for _ in range(6):                                   # A admits requests of 2 blocks while it may
            t += 1
            o.set_time(t)
            if o.alloc_blocks(next_id, 2, AUTO)[0] == oracle.OK:
                next_id += 1
        t += 1
        o.set_time(t)
        assert o.reclaim_preempt(4, 2, None, None)[0] == oracle.OK     # B's demand rises
        t += 1
        o.set_time(t)
        assert o.lend(4) == oracle.OK                                   # and falls again
    return o.preempt_state()["preempt_reclaim"]


def test_the_cap_ends_the_back_and_forth():
    without, with_cap = _back_and_forth(0), _back_and_forth(1000)
    assert without == 2 * 12            # every round evicts two requests of two blocks again
    assert with_cap == 2                # once: afterwards A stays at the level it was preempted to
    assert _back_and_forth(3) == without    # a window shorter than the cycle changes nothing
