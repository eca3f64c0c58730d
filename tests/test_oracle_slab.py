"""Pins of the oracle's slab allocator and memory layouts (Sections 4.2.1 - 4.2.3, defaults of
Section 6.7): a hand-worked allocation sequence, the rule checked by brute force over random
operation sequences, the layouts as nested arrays, the paper's layer-group index example, and the
sizes of the contiguous pieces one swap moves in each layout. CPU only."""
import json
import os

import numpy as np
import pytest

import oracle
from oracle import AUTO, LENT, LOCAL, LAYER_MAJOR, SLAB_MAJOR, LAYER_GROUP_MAJOR

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _slice(local, lent, slab, phys=None):
    o = oracle.OracleSlice(2, 16, 64, local, lent, phys, 2, 64, max_seqs=64, max_blocks_per_seq=64)
    assert o.set_slab_blocks(slab) == oracle.OK
    return o


def test_hand_worked_slab_allocation():
    with open(os.path.join(GOLDEN, "slab_alloc_worked_example.json")) as f:
        gold = json.load(f)
    o = _slice(gold["local_blocks"], gold["lent_blocks"], gold["slab_blocks"])
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
    assert trace == gold["expected"]
    for seq, tab in gold["final_tables"].items():
        assert o.block_table(int(seq))[1].tolist() == tab
    assert sorted(o.free_stack(LOCAL).tolist()) == gold["final_free_local"]
    assert sorted(o.free_stack(LENT).tolist()) == gold["final_free_lent"]
    assert o.lent_capacity == gold["final_lent_capacity"]


def test_slab_mode_must_be_chosen_before_the_first_allocation():
    o = oracle.OracleSlice(1, 16, 64, 8, 8, None, 2, 8, max_seqs=4, max_blocks_per_seq=8)
    assert o.alloc_blocks(0, 1, LOCAL)[0] == oracle.OK
    assert o.set_slab_blocks(4) == oracle.E_STATE


@pytest.mark.parametrize("seed,slab", [(0, 4), (1, 3), (2, 10), (3, 1)])
def test_every_allocation_obeys_the_slab_rule(seed, slab):
    """Brute force beside the oracle: before every single-block allocation the test works out, from
    the tables alone, which ids are in use, which slabs therefore belong to the user, and what the
    rule allows: a free id in a slab in use if there is one (the lowest), else the lowest free id.
    Also: no id is handed out twice, freed ids come back, ENOSPC exactly when nothing is free."""
    rng = np.random.default_rng(seed)
    LB, RB = 23, 17                                     # not multiples of the slab: last slabs are short
    o = _slice(LB, RB, slab)
    tables = {}

    def in_use(tier):
        return {(e if tier == LOCAL else ~e) for t in tables.values() for e in t if (e >= 0) == (tier == LOCAL)}

    def expected(tier):
        cap = LB if tier == LOCAL else o.lent_capacity
        used = in_use(tier)
        free = [i for i in range(cap) if i not in used]
        if not free:
            return None
        owned = {i // slab for i in used}
        in_owned = [i for i in free if i // slab in owned]
        return in_owned[0] if in_owned else free[0]

    for step in range(1500):
        op = int(rng.integers(0, 10))
        if op < 6:
            q, tier = int(rng.integers(0, 12)), int(rng.integers(1, 3))
            if len(tables.get(q, [])) >= 60:
                continue
            want = expected(tier)
            rc, ent = o.alloc_blocks(q, 1, tier)
            if want is None:
                assert rc == oracle.E_NOSPC
            else:
                assert rc == oracle.OK and int(ent[0]) == (want if tier == LOCAL else ~want)
                tables.setdefault(q, []).append(int(ent[0]))
        elif op == 6 and tables:
            q = int(rng.choice(sorted(tables)))
            assert o.free_seq(q) == oracle.OK
            del tables[q]
        elif op == 7:                                   # AUTO: the local part first, by the same rule
            q = int(rng.integers(0, 12))
            if len(tables.get(q, [])) >= 60:
                continue
            wl, wr = expected(LOCAL), expected(LENT)
            rc, ent = o.alloc_blocks(q, 1, AUTO)
            if wl is None and wr is None:
                assert rc == oracle.E_NOSPC
            else:
                assert rc == oracle.OK and int(ent[0]) == (wl if wl is not None else ~wr)
                tables.setdefault(q, []).append(int(ent[0]))
        elif op == 8:
            take = int(rng.integers(0, 5))
            before = {q: list(t) for q, t in tables.items()}
            rc, mig = o.reclaim(take, None, None)
            if rc == oracle.OK:
                for q in tables:
                    tables[q] = o.block_table(q)[1].tolist()
                # logical order and lengths unchanged; moved entries were at or above the cut
                cut = o.lent_capacity
                for q, t in tables.items():
                    assert len(t) == len(before[q])
                    for a, b in zip(before[q], t):
                        assert a == b or (a < 0 and ~a >= cut)
                assert all(~e < cut for t in tables.values() for e in t if e < 0)
            else:
                assert rc == oracle.E_NOSPC
        else:
            o.lend(int(rng.integers(0, 4)))
        for q, t in tables.items():
            assert o.block_table(q)[1].tolist() == t
        ids = [e for t in tables.values() for e in t]
        assert len(ids) == len(set(ids))
        assert sorted(o.free_stack(LOCAL).tolist()) == sorted(set(range(LB)) - in_use(LOCAL))
        assert sorted(o.free_stack(LENT).tolist()) == sorted(set(range(o.lent_capacity)) - in_use(LENT))


def test_slabs_keep_more_whole_slabs_free_than_the_block_stack():
    """What the slab is for (Section 4.2.1): memory returns to the slice a whole slab at a time, and
    only whole free slabs can go to the other user. Requests of mixed lifetimes come and go; under
    the slab rule the survivors end up packed into few slabs, under the plain free stack (ids handed
    out in the order they were freed) they are scattered."""
    def run(slab_mode):
        rng = np.random.default_rng(5)
        o = oracle.OracleSlice(1, 16, 64, 200, 0, None, 2, 8, max_seqs=256, max_blocks_per_seq=16)
        if slab_mode:
            assert o.set_slab_blocks(10) == oracle.OK
        live, nxt = [], 0
        for step in range(3000):
            if live and (len(live) > 40 or rng.random() < 0.45):
                q = live.pop(int(rng.integers(0, len(live))))
                o.free_seq(q)
            else:
                n = int(rng.integers(1, 5))
                if o.alloc_blocks(nxt, n, LOCAL)[0] == oracle.OK:
                    live.append(nxt)
                nxt += 1
        used = {int(e) for q in live for e in o.block_table(q)[1]}
        return sum(1 for s in range(20) if not any(i // 10 == s for i in used)), len(used)
    free_slab, used_slab = run(True)
    free_stack, used_stack = run(False)
    assert used_slab == used_stack                       # same requests alive either way
    assert free_slab > free_stack


# ---------------------------------------------------------------------------------------------
# layouts
# ---------------------------------------------------------------------------------------------
BB = 64
L, NB, S, K = 8, 40, 10, 2          # 8 layers, 4 slabs of 10 blocks, groups of 2 layers


def _arena(layout, k=K):
    """Where every (layer, id) sits, as an array over block positions; checks that the map is a
    bijection onto the arena."""
    pos = np.array([[oracle.layout_offset(layout, L, NB, S, k, BB, l, b) for b in range(NB)] for l in range(L)])
    assert (pos % BB == 0).all()
    assert sorted((pos // BB).ravel().tolist()) == list(range(L * NB))
    return pos // BB


def test_layouts_are_the_nested_arrays_of_the_figures():
    """The maps against numpy's own C-order indexing of the arrays the three figures draw."""
    lm, sm, gm = _arena(LAYER_MAJOR), _arena(SLAB_MAJOR), _arena(LAYER_GROUP_MAJOR)
    a = np.arange(L * NB)
    for l in range(L):
        for b in range(NB):
            assert lm[l, b] == a.reshape(L, NB)[l, b]
            assert sm[l, b] == a.reshape(NB // S, L, S)[b // S, l, b % S]
            assert gm[l, b] == a.reshape(L // K, NB // S, K, S)[l // K, b // S, l % K, b % S]


def test_contiguity_each_layout_guarantees():
    lm, sm, gm = _arena(LAYER_MAJOR), _arena(SLAB_MAJOR), _arena(LAYER_GROUP_MAJOR)
    for l in range(L):
        for b in range(NB - 1):
            assert lm[l, b + 1] == lm[l, b] + 1                      # layer-major: a layer is one piece
            if (b + 1) % S:
                assert sm[l, b + 1] == sm[l, b] + 1 and gm[l, b + 1] == gm[l, b] + 1   # a slab of a layer is one piece
    for l in range(L - 1):
        for s in range(NB // S):
            first_next, last_this = s * S, s * S + S - 1
            # slab-major: consecutive layers of one slab follow each other (a layer group is contiguous)
            assert sm[l + 1, first_next] == sm[l, last_this] + 1
            # layer-group-major: only inside a group; the next group of the slab is elsewhere
            assert (gm[l + 1, first_next] == gm[l, last_this] + 1) == ((l + 1) % K != 0)
    for g in range(L // K):
        for s in range(NB // S - 1):
            # layer-group-major: slab s+1 of a group follows slab s of the same group
            assert gm[g * K, (s + 1) * S] == gm[g * K + K - 1, s * S + S - 1] + 1
            # slab-major: it does not (all the other groups of slab s lie in between)
            assert sm[g * K, (s + 1) * S] != sm[g * K + K - 1, s * S + S - 1] + 1


def test_layer_group_index_example_of_section_4_2_2():
    """With a layer group size of 2, layer groups 0-2 are layers 0-5 and layer group 2 is layers 4
    and 5: the example the paper gives for operating on group indices instead of layer indices."""
    assert [l for g in range(0, 3) for l in oracle.group_layers(2, g)] == [0, 1, 2, 3, 4, 5]
    assert list(oracle.group_layers(2, 2)) == [4, 5]
    # and a group of slab-major memory is one piece holding exactly those layers
    sm = _arena(SLAB_MAJOR)
    piece = sorted(sm[l, b] for l in oracle.group_layers(2, 2) for b in range(S))        # slab 0
    assert piece == list(range(piece[0], piece[0] + 2 * S))


@pytest.mark.parametrize("slabs", [[1], [1, 2], [0, 1, 2], [0, 2], [1, 2, 3, 5, 6, 8]])
def test_swap_piece_sizes_per_layout(slabs):
    """Section 4.2.3: with S the bytes of one slab of one layer, k the group size and runs of up to
    m adjacent slabs, one swap of a layer group moves pieces of S..mS (layer-major), exactly kS
    (slab-major) and kS..mkS (layer-group-major)."""
    nb, k, Lx = 100, 4, 8                                   # 10 slabs of 10; the user never holds both end slabs
    Sb = S * BB
    runs, cur = [], [slabs[0]]
    for a, b in zip(slabs, slabs[1:]):
        if b == a + 1:
            cur.append(b)
        else:
            runs.append(len(cur))
            cur = [b]
    runs.append(len(cur))
    for g in range(Lx // k):
        lm = oracle.swap_pieces(LAYER_MAJOR, Lx, nb, S, k, BB, g, slabs)
        sm = oracle.swap_pieces(SLAB_MAJOR, Lx, nb, S, k, BB, g, slabs)
        gm = oracle.swap_pieces(LAYER_GROUP_MAJOR, Lx, nb, S, k, BB, g, slabs)
        assert sum(lm) == sum(sm) == sum(gm) == k * len(slabs) * Sb       # the same bytes move in every layout
        assert lm == [r * Sb for r in runs] * k                          # per layer: runs of adjacent slabs
        assert sm == [k * Sb] * len(slabs)                               # fixed: one slab's group
        assert gm == [r * k * Sb for r in runs]                          # runs of adjacent slabs, k layers each
        m = max(runs)
        assert min(lm) >= Sb and max(lm) == m * Sb and min(gm) >= k * Sb and max(gm) == m * k * Sb


def test_whole_arena_and_single_layer_group_edge_cases():
    Sb = S * BB
    # a user that holds every slab: layer-major and layer-group-major move one piece per group
    assert oracle.swap_pieces(LAYER_MAJOR, L, NB, S, K, BB, 1, [0, 1, 2, 3]) == [K * 4 * Sb]
    assert oracle.swap_pieces(LAYER_GROUP_MAJOR, L, NB, S, K, BB, 1, [0, 1, 2, 3]) == [K * 4 * Sb]
    assert oracle.swap_pieces(SLAB_MAJOR, L, NB, S, K, BB, 1, [0, 1, 2, 3]) == [K * Sb] * 4
    # group size 1: slab-major and layer-group-major differ only in what lies next to a piece
    assert oracle.swap_pieces(SLAB_MAJOR, L, NB, S, 1, BB, 3, [1, 2]) == [Sb, Sb]
    assert oracle.swap_pieces(LAYER_GROUP_MAJOR, L, NB, S, 1, BB, 3, [1, 2]) == [2 * Sb]
    # one group spanning all layers: a slab is one piece in slab-major, and adjacent slabs join
    assert oracle.swap_pieces(SLAB_MAJOR, L, NB, S, L, BB, 0, [1, 2]) == [2 * L * Sb]
