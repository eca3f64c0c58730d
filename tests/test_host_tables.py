"""Host logic of the CUDA library, run without a GPU in its tables-only mode: the library's
allocator, resolved tables, staging order and reclaim planning must agree bit for bit with the
oracle's integer state machine; the shared object must export every entry point the header
declares."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2609_27040_b200 import binding as B
from paper_2609_27040_b200 import build as build_mod
from paper_2609_27040_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def _null_slice(L, Hkv, local, lent, phys, cap, max_seqs, max_blocks, lo=None, ro=None, ring=2):
    return B.Slice(L, Hkv, local, lent, cap, lent_blocks_physical=phys, ring_slots=ring, max_seqs=max_seqs,
                   max_blocks_per_seq=max_blocks, flags=B.FLAG_NULL_DEVICE, local_free_order=lo,
                   lent_free_order=ro)


def test_library_exports_every_declared_entry_point():
    with open(os.path.join(ROOT, "include", "emaslice.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    declared = set(re.findall(r"\b(?:int|const char\*)\s+(\w+)\s*\(", text))
    assert declared == set(B.EXPORTS)
    lib = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_config_struct_matches_header_size():
    # 14 uint32, 3 pointers, 4 uint64, 2 pointers, 13 uint32 (+ 4 bytes of tail padding)
    assert C.sizeof(B.SliceConfig) == 14 * 4 + 3 * 8 + 4 * 8 + 2 * 8 + 13 * 4 + 4


def test_create_rejects_bad_configs():
    with pytest.raises(B.SliceError):
        _null_slice(1, 9, 4, 4, 4, 4, 4, 4)                       # more than 8 KV heads
    with pytest.raises(B.SliceError):
        _null_slice(1, 8, 4, 5, 4, 4, 4, 4)                       # lent capacity beyond the arena
    with pytest.raises(B.SliceError):
        _null_slice(1, 8, 4, 4, 4, 4, 4, 4, ring=0)
    with pytest.raises(B.SliceError):
        _null_slice(1, 8, 4, 4, 4, 4, 4, 4, lo=np.array([0, 0, 1, 2], np.uint32))   # not a permutation
    with pytest.raises(B.SliceError):
        B.Slice(1, 8, 4, 4, 4)                                     # device mode needs arenas
    for kw in ({"pipeline_mode": 4}, {"copy_kind": 4}, {"prefetch_priority": 2}, {"swap_out": 3}):
        with pytest.raises(B.SliceError):
            B.Slice(2, 8, 4, 4, 4, max_seqs=4, max_blocks_per_seq=4, flags=B.FLAG_NULL_DEVICE, **kw)
    for kw in ({"pipeline_mode": 3}, {"copy_kind": 3}):                # the chain of launches; the SM-sharing gather
        B.Slice(2, 8, 4, 4, 4, max_seqs=4, max_blocks_per_seq=4, flags=B.FLAG_NULL_DEVICE, **kw).close()


def _same_state(s: B.Slice, o: oracle.OracleSlice, live):
    for q in live:
        rc1, t1, l1 = s.slice_get_block_table(q)
        rc2, t2, l2 = o.block_table(q)
        assert rc1 == rc2 == 0 and l1 == l2 and t1.tolist() == t2.tolist()
    assert s.slice_get_free_stack(B.TIER_LOCAL).tolist() == o.free_stack(oracle.LOCAL).tolist()
    assert s.slice_get_free_stack(B.TIER_LENT).tolist() == o.free_stack(oracle.LENT).tolist()
    st = s.slice_stats()
    assert st["lent_capacity"] == o.lent_capacity and st["num_seqs"] == o.num_seqs


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_random_ops_match_oracle_state_machine(seed):
    rng = np.random.default_rng(seed)
    LB, RB, PH, CAP = 24, 14, 20, 12
    lo, ro = synth.free_order(rng, LB), synth.free_order(rng, PH)
    s = _null_slice(2, 8, LB, RB, PH, CAP, 6, 9, lo, ro)
    o = oracle.OracleSlice(2, 16, 65536, LB, RB, PH, 2, CAP, max_seqs=6, max_blocks_per_seq=9,
                           local_free_order=lo, lent_free_order=ro)
    live = set()
    for step in range(3000):
        op = int(rng.integers(0, 12))
        if op < 5:
            q, n, hint = int(rng.integers(0, 8)), int(rng.integers(0, 5)), int(rng.integers(0, 3))
            rc1, e1 = s.slice_alloc_blocks(q, n, hint)
            rc2, e2 = o.alloc_blocks(q, n, hint)
            assert rc1 == rc2
            if rc1 == 0:
                assert e1.tolist() == e2.tolist()
                live.add(q)
        elif op == 5 and live:
            q = int(rng.choice(sorted(live)))
            nb = len(o.block_table(q)[1])
            ln = int(rng.integers(0, nb * 16 + 3))
            assert s.slice_set_seq_len(q, ln) == o.set_seq_len(q, ln)
        elif op == 6:
            q = int(rng.integers(0, 8))
            rc1, rc2 = s.slice_free_seq(q), o.free_seq(q)
            assert rc1 == rc2
            live.discard(q)
        elif op == 7:
            take = int(rng.integers(0, 6))
            rc1, m1 = s.slice_reclaim(take)
            rc2, m2 = o.reclaim(take, None, None)
            assert rc1 == rc2 and (rc1 != 0 or m1 == m2)
        elif op == 8:
            n = int(rng.integers(0, 4))
            assert s.slice_lend(n) == o.lend(n)
        elif live:
            # resolved tables and staging order of a random batch
            batch = [int(x) for x in rng.permutation(sorted(live))[: int(rng.integers(1, len(live) + 1))]]
            rc2, r2, k2 = o.gather(int(rng.integers(0, 2)), batch, None, None)
            rc1, r1, k1 = s.slice_get_resolved(batch)
            assert rc1 == rc2
            if rc1 == 0:
                assert k1 == k2 and (r1 == r2).all()
        _same_state(s, o, live)
    s.close()


def test_error_codes_and_unchanged_state():
    s = _null_slice(2, 8, 4, 4, 4, 2, 4, 8)
    assert s.slice_alloc_blocks(0, 3, B.TIER_LENT)[0] == B.OK
    assert s.slice_set_seq_len(0, 48) == B.OK
    assert s.prefetch_layer(0, [0]) == B.ESTAGING                  # three lent blocks, slot holds two
    assert s.slice_set_seq_len(0, 20) == B.OK
    assert s.paged_decode(0, [0], None, 8, 1.0, None) == B.ESTALE   # nothing staged yet
    assert s.prefetch_layer(0, [0]) == B.OK
    assert s.paged_decode(0, [0], None, 8, 1.0, None) == B.OK       # tables-only mode: no launch
    assert s.paged_decode(1, [0], None, 8, 1.0, None) == B.ESTALE   # other layer not staged
    assert s.prefetch_layer(2, [0]) == B.EINVAL
    assert s.prefetch_layer(0, [0, 0]) == B.EINVAL
    assert s.prefetch_layer(0, [7]) == B.ESTATE
    assert s.paged_decode(0, [0], None, 12, 1.0, None) == B.EINVAL  # 12 query heads over 8 KV heads
    assert s.slice_set_seq_len(0, 21) == B.OK                       # tables changed: staged copy is stale
    assert s.paged_decode(0, [0], None, 8, 1.0, None) == B.ESTALE
    assert s.prefetch_layer(0, [0]) == B.OK
    rc, mig = s.slice_reclaim(B.TAKE_ALL)
    assert rc == B.OK and mig == 3
    assert s.paged_decode(0, [0], None, 8, 1.0, None) == B.OK       # all local now: nothing to stage
    assert s.slice_get_block_table(0)[1].tolist() == [0, 1, 2]
    assert s.slice_free_seq(0) == B.OK and s.slice_free_seq(0) == B.ESTATE
    assert B.slice_strerror(B.ENOSPC) == "not enough free blocks"
    s.close()


def test_decode_step_drives_the_layer_pipeline_in_tables_only_mode():
    s = _null_slice(4, 8, 8, 8, 8, 4, 4, 8)
    s.slice_alloc_blocks(0, 2, B.TIER_LENT)
    s.slice_alloc_blocks(0, 1, B.TIER_LOCAL)
    s.slice_set_seq_len(0, 40)
    assert s.slice_decode_step([0], None, 8, 1.0, None) == B.OK
    st = s.slice_stats()
    # four layers prefetched, plus layer 0 again for the next pass (cyclic order)
    assert st["prefetch_calls"] == 5 and st["decode_calls"] == 4 and st["plans_built"] == 1
    assert s.slice_decode_step([0], None, 8, 1.0, None, wrap_prefetch=False) == B.OK
    st = s.slice_stats()
    assert st["prefetch_calls"] == 8 and st["decode_calls"] == 8   # layer 0 was already staged
    s.close()


def test_layer_dependent_pass_bookkeeping_in_tables_only_mode():
    """slice_step_begin does the same bookkeeping as slice_decode_step; the calls that feed and follow
    the running pass need a pass begun by it, and only the one-launch pipeline has one."""
    s = _null_slice(4, 8, 8, 8, 8, 4, 4, 8)
    s.slice_alloc_blocks(0, 2, B.TIER_LENT)
    s.slice_alloc_blocks(0, 1, B.TIER_LOCAL)
    s.slice_set_seq_len(0, 40)
    assert s.slice_step_submit_q(0, None) == B.EINVAL and s.slice_step_wait_out(0, None) == B.EINVAL
    assert s.slice_step_flags()[0] == B.EINVAL
    assert s.slice_step_begin([0], None, 8, 1.0, None) == B.OK
    st = s.slice_stats()
    assert st["prefetch_calls"] == 5 and st["decode_calls"] == 4
    for layer in range(4):
        assert s.slice_step_submit_q(layer, None) == B.OK and s.slice_step_wait_out(layer, None) == B.OK
    assert s.slice_step_submit_q(4, None) == B.EINVAL and s.slice_step_relay(None) == B.OK
    rc, _, _, epoch = s.slice_step_flags()
    assert rc == B.OK and epoch == 1
    assert s.slice_decode_step([0], None, 8, 1.0, None) == B.OK       # a free-running pass ends the dependent one
    assert s.slice_step_submit_q(0, None) == B.EINVAL
    assert s.slice_step_begin([0], None, 12, 1.0, None) == B.EINVAL   # bad head count
    assert s.slice_set_seq_len(0, 0) == B.OK
    assert s.slice_step_begin([0], None, 8, 1.0, None) == B.EINVAL    # empty sequence
    s.close()
    for kw in ({"pipeline_mode": 1}, {"pipeline_mode": 2}, {"pipeline_mode": 3}, {"ring_slots": 1}):
        s = B.Slice(4, 8, 8, 8, 4, lent_blocks_physical=8, max_seqs=4, max_blocks_per_seq=8, flags=B.FLAG_NULL_DEVICE, **kw)
        s.slice_alloc_blocks(0, 2, B.TIER_LENT)
        s.slice_set_seq_len(0, 20)
        assert s.slice_step_begin([0], None, 8, 1.0, None) == B.EINVAL
        s.close()


def test_decode_step_with_a_shared_ring_slot_for_first_and_last_layer():
    """Five layers on a ring of two: the last layer and layer 0 share slot 0, so the prefetch of
    layer 0 for the next pass may only follow the last attention."""
    s = _null_slice(5, 8, 8, 8, 8, 4, 4, 8)
    s.slice_alloc_blocks(0, 2, B.TIER_LENT)
    s.slice_set_seq_len(0, 20)
    for _ in range(3):
        assert s.slice_decode_step([0], None, 8, 1.0, None) == B.OK
    st = s.slice_stats()
    assert st["decode_calls"] == 15 and st["prefetch_calls"] == 16
    s.close()


def test_kv_block_swizzle_is_the_documented_self_inverse_permutation():
    """Block format of include/emaslice.h: within every 128 bytes of token row r, 16-byte unit u is
    stored at unit u ^ (r & 7); applying it twice gives the rows back."""
    rng = np.random.default_rng(3)
    x = rng.integers(0, 65536, size=(3, 2, 16, 4, 128), dtype=np.uint16)
    y = B.kv_block_swizzle(x)
    assert y.shape == x.shape and (B.kv_block_swizzle(y) == x).all()
    rows_x = x.reshape(3, 2, 16, -1)       # 4 heads * 128 bf16 = 1024 B per row = 8 windows of 128 B
    rows_y = y.reshape(3, 2, 16, -1)
    for r in range(16):
        for w in range(8):
            for u in range(8):
                src = rows_x[..., r, w * 64 + u * 8: w * 64 + u * 8 + 8]
                dst = rows_y[..., r, w * 64 + (u ^ (r & 7)) * 8: w * 64 + (u ^ (r & 7)) * 8 + 8]
                assert (src == dst).all()
    with pytest.raises(ValueError):
        B.kv_block_swizzle(np.zeros((15, 4, 128), np.uint16))


@pytest.mark.parametrize("ring,calls", [(1, 11), (2, 11), (3, 10), (4, 8)])
def test_decode_step_plans_prefetches_for_any_ring_depth(ring, calls):
    """Tables-only mode: two passes over 5 layers succeed for every pipeline and ring depth (a ring
    of one slot prefetches after the attention that reads the slot), and the number of prefetches
    follows from which layers are still staged when the second pass starts."""
    for mode in (0, 1, 2, 3):
        s = B.Slice(5, 4, 64, 64, 64, lent_blocks_physical=64, ring_slots=ring, max_seqs=8, max_blocks_per_seq=64,
                    flags=B.FLAG_NULL_DEVICE, pipeline_mode=mode)
        for i in range(3):
            for b in range(10):
                assert s.slice_alloc_blocks(i, 1, B.TIER_LENT if b % 2 else B.TIER_LOCAL)[0] == B.OK
            assert s.slice_set_seq_len(i, 150) == B.OK
        seqs = np.arange(3, dtype=np.int32)
        for _ in range(2):
            assert s.slice_decode_step(seqs, None, 16, 0.1, None, False, True, None, None) == B.OK
        assert s.slice_stats()["prefetch_calls"] == calls
        s.slice_destroy()


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_preemption_calls_match_oracle_state_machine(seed):
    """Reclaim by preemption, engine-chosen preemptions, the clock and the cap: return codes, the
    victims and their order, tables, free lists and the counters agree with the oracle over random
    call sequences in which the lender's demand comes and goes."""
    rng = np.random.default_rng(100 + seed)
    LB, RB, PH, CAP = 10, 18, 24, 24
    lo, ro = synth.free_order(rng, LB), synth.free_order(rng, PH)
    s = _null_slice(2, 8, LB, RB, PH, CAP, 10, 9, lo, ro)
    o = oracle.OracleSlice(2, 16, 65536, LB, RB, PH, 2, CAP, max_seqs=10, max_blocks_per_seq=9,
                           local_free_order=lo, lent_free_order=ro)
    window = int(rng.choice([0, 5, 40]))
    assert s.slice_set_preempt_window(window) == o.set_preempt_window(window) == 0
    live, now, evictions, capped = set(), 0, 0, 0
    for step in range(3000):
        op = int(rng.integers(0, 14))
        if op < 6:
            q, n, hint = int(rng.integers(0, 12)), int(rng.integers(0, 5)), int(rng.integers(0, 3))
            rc1, e1 = s.slice_alloc_blocks(q, n, hint)
            rc2, e2 = o.alloc_blocks(q, n, hint)
            assert rc1 == rc2
            capped += rc1 == B.ECAPPED
            if rc1 == 0:
                assert e1.tolist() == e2.tolist()
                live.add(q)
        elif op == 6:
            q = int(rng.integers(0, 12))
            assert s.slice_free_seq(q) == o.free_seq(q)
            live.discard(q)
        elif op == 7:
            q, cause = int(rng.integers(0, 12)), int(rng.integers(0, 4))
            rc1, rc2 = s.slice_preempt_seq(q, cause), o.preempt_seq(q, cause)
            assert rc1 == rc2
            if rc1 == 0:
                live.discard(q)
        elif op in (8, 9):
            take, slab = int(rng.integers(0, 9)), int(rng.integers(0, 6))
            cap = None if rng.random() < 0.8 else int(rng.integers(0, 3))
            rc1, v1, m1 = s.slice_reclaim_preempt(take, slab, max_victims=cap)
            rc2, v2, m2 = o.reclaim_preempt(take, slab, None, None, max_victims=cap)
            assert rc1 == rc2 and v1 == v2 and (rc1 != 0 or m1 == m2), (rc1, rc2, v1, v2)
            if rc1 == 0:
                live -= set(v1)
                evictions += len(v1)
        elif op == 10:
            take = int(rng.integers(0, 6))
            rc1, m1 = s.slice_reclaim(take)
            rc2, m2 = o.reclaim(take, None, None)
            assert rc1 == rc2 and (rc1 != 0 or m1 == m2)
        elif op == 11:
            n = int(rng.integers(0, 6))
            assert s.slice_lend(n) == o.lend(n)
        elif op == 12:
            now += int(rng.integers(0, 8))
            assert s.slice_set_time(now) == o.set_time(now) == 0
        else:
            back = max(now - 1, 0)
            assert s.slice_set_time(back) == o.set_time(back)          # refused unless equal
        _same_state(s, o, live)
        assert s.slice_preempt_stats() == o.preempt_state()
    assert evictions > 0 and (window == 0 or capped > 0)
    s.close()


def _snapshot(s: B.Slice, seqs):
    return ([(q,) + tuple(x.tolist() if hasattr(x, "tolist") else x for x in s.slice_get_block_table(q)) for q in seqs],
            s.slice_get_free_stack(B.TIER_LOCAL).tolist(), s.slice_get_free_stack(B.TIER_LENT).tolist(),
            s.slice_preempt_stats(), {k: v for k, v in s.slice_stats().items() if k != "last_cuda_error"})


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_failed_migration_leaves_reclaim_and_preemption_uncommitted(seed):
    """Injected on the host (a test hook makes the step that enqueues the migration report failure,
    as a failed CUDA call would): slice_reclaim and slice_reclaim_preempt return ECUDA and tables,
    free lists, the evicted requests, counters and the cap are exactly as before; a twin slice
    without the hook, fed the same calls, shows what the same request does when the copy goes
    through (when nothing has to migrate there is no copy to fail, and both succeed alike)."""
    rng = np.random.default_rng(40 + seed)
    LB, RB, PH = 6, 16, 16
    lo, ro = synth.free_order(rng, LB), synth.free_order(rng, PH)
    mk = lambda flags: B.Slice(2, 8, LB, RB, 16, lent_blocks_physical=PH, max_seqs=8, max_blocks_per_seq=8,
                               flags=B.FLAG_NULL_DEVICE | flags, local_free_order=lo, lent_free_order=ro)
    seqs = list(range(6))
    lens = [16 * (4 if q < 4 else 3) - int(rng.integers(0, 16)) for q in seqs]
    failed_with_victims = 0
    for take in range(3, 12):
        bad, good = mk(B.FLAG_TEST_FAIL_COPY), mk(0)
        for s in (bad, good):
            assert s.slice_set_preempt_window(50) == B.OK and s.slice_set_time(3) == B.OK
            for q in seqs:                                  # fill both parts completely
                assert s.slice_alloc_blocks(q, 4 if q < 4 else 3, B.TIER_AUTO)[0] == B.OK
                assert s.slice_set_seq_len(q, lens[q]) == B.OK
        before = _snapshot(bad, seqs)
        assert before == _snapshot(good, seqs)
        assert good.slice_reclaim(take)[0] == B.ENOSPC and bad.slice_reclaim(take)[0] == B.ENOSPC   # no room
        assert _snapshot(bad, seqs) == before
        rc_g, victims_g, mig_g = good.slice_reclaim_preempt(take, 4)
        assert rc_g == B.OK and len(victims_g) > 0
        rc, victims, mig = bad.slice_reclaim_preempt(take, 4)
        if mig_g > 0:                                       # something had to be copied: the copy "fails"
            assert rc == B.ECUDA and victims == [] and mig == 0
            assert _snapshot(bad, seqs) == before           # nobody evicted, nothing counted, no cap
            assert bad.slice_stats()["last_cuda_error"] != 0
            assert bad.slice_get_resolved(seqs)[0] == B.OK  # and the state is still usable
            failed_with_victims += 1
        else:
            assert rc == B.OK and victims == victims_g
            live = [q for q in seqs if q not in victims]
            assert _snapshot(bad, live) == _snapshot(good, live)
        bad.close()
        good.close()
    assert failed_with_victims >= 2
    # a plain migration that has room fails the same way and commits nothing
    bad = mk(B.FLAG_TEST_FAIL_COPY)
    for q in seqs[:4]:
        assert bad.slice_alloc_blocks(q, 1, B.TIER_LENT)[0] == B.OK and bad.slice_set_seq_len(q, 14) == B.OK
    before = _snapshot(bad, seqs[:4])
    assert bad.slice_reclaim(B.TAKE_ALL)[0] == B.ECUDA
    assert _snapshot(bad, seqs[:4]) == before
    bad.close()


def test_preemption_bad_arguments():
    s = _null_slice(2, 8, 4, 4, 4, 4, 4, 8)
    assert s.slice_reclaim_preempt(2, 0)[0] == B.EINVAL
    assert s.slice_preempt_seq(0, B.PREEMPT_OOM) == B.ESTATE
    assert s.slice_alloc_blocks(0, 1, B.TIER_LENT)[0] == B.OK
    assert s.slice_preempt_seq(0, 0) == B.EINVAL and s.slice_preempt_seq(0, 3) == B.EINVAL
    assert s.slice_set_time(5) == B.OK and s.slice_set_time(4) == B.EINVAL
    assert B.slice_strerror(B.ECAPPED).startswith("a cap")
    s.close()


@pytest.mark.parametrize("seed", [0, 1])
def test_slice_choice_matches_oracle(seed):
    """Greedy-Least-Loaded over several slices of different sizes, with requests coming and going
    and the peers' own use changing: the library picks the slice the oracle picks, ties included."""
    rng = np.random.default_rng(seed)
    shapes = [(8, 8), (8, 8), (6, 10), (16, 16)]                    # (local, lent): equal and unequal capacities
    slices = [_null_slice(1, 8, lb, rb, rb, rb, 64, 8) for lb, rb in shapes]
    cap = [lb + rb for lb, rb in shapes]
    own, peer, homes, next_id, ties = [0] * 4, [0] * 4, {}, 0, 0
    for step in range(1500):
        op = int(rng.integers(0, 4))
        if op < 2:
            k = B.slice_schedule_gll(slices)
            assert k == oracle.gll_choose(own, peer, cap)
            from fractions import Fraction
            u = [Fraction(own[i] + peer[i], cap[i]) for i in range(4)]
            ties += sum(x == min(u) for x in u) > 1
            n = int(rng.integers(1, 3))
            if slices[k].slice_alloc_blocks(next_id, n, B.TIER_AUTO)[0] == B.OK:
                own[k] += n
                homes[next_id] = (k, n)
                next_id += 1
        elif op == 2 and homes:
            q = int(rng.choice(sorted(homes)))
            k, n = homes.pop(q)
            assert slices[k].slice_free_seq(q) == B.OK
            own[k] -= n
        else:
            k = int(rng.integers(0, 4))
            used = int(rng.integers(0, shapes[k][1] + 2))
            rc = slices[k].slice_set_peer_used(used)
            assert rc == (B.OK if used <= shapes[k][1] else B.EINVAL)
            if rc == B.OK:
                peer[k] = used
    assert ties > 20
    with pytest.raises(B.SliceError):
        B.slice_schedule_gll([])
    for sl in slices:
        sl.close()


@pytest.mark.parametrize("seed,slab", [(0, 4), (1, 3), (2, 10), (3, 1)])
def test_slab_allocator_matches_oracle_state_machine(seed, slab):
    """Slab allocator (Section 4.2.1) in the library and in the oracle over random allocations,
    frees, reclaims (plain and by preemption) and lends: the same ids in the same order, the same
    migration destinations, the same free ids (as sets: in slab mode the rule, not a stack, orders
    them), capacities not multiples of the slab."""
    rng = np.random.default_rng(300 + seed)
    LB, RB, PH, CAP = 23, 17, 26, 26
    s = B.Slice(2, 8, LB, RB, CAP, lent_blocks_physical=PH, max_seqs=10, max_blocks_per_seq=9,
                flags=B.FLAG_NULL_DEVICE, slab_blocks=slab)
    o = oracle.OracleSlice(2, 16, 65536, LB, RB, PH, 2, CAP, max_seqs=10, max_blocks_per_seq=9)
    assert o.set_slab_blocks(slab) == 0
    live = set()
    moved = evicted = 0
    for step in range(2500):
        op = int(rng.integers(0, 12))
        if op < 6:
            q, n, hint = int(rng.integers(0, 12)), int(rng.integers(0, 5)), int(rng.integers(0, 3))
            rc1, e1 = s.slice_alloc_blocks(q, n, hint)
            rc2, e2 = o.alloc_blocks(q, n, hint)
            assert rc1 == rc2
            if rc1 == 0:
                assert e1.tolist() == e2.tolist()
                live.add(q)
        elif op == 6:
            q = int(rng.integers(0, 12))
            assert s.slice_free_seq(q) == o.free_seq(q)
            live.discard(q)
        elif op == 7:
            take = int(rng.integers(0, 7))
            rc1, m1 = s.slice_reclaim(take)
            rc2, m2 = o.reclaim(take, None, None)
            assert rc1 == rc2 and (rc1 != 0 or m1 == m2)
            moved += m1 if rc1 == 0 else 0
        elif op == 8:
            take, sb = int(rng.integers(0, 9)), int(rng.integers(1, 6))
            rc1, v1, m1 = s.slice_reclaim_preempt(take, sb)
            rc2, v2, m2 = o.reclaim_preempt(take, sb, None, None)
            assert rc1 == rc2 and v1 == v2 and (rc1 != 0 or m1 == m2)
            if rc1 == 0:
                live -= set(v1)
                evicted += len(v1)
        elif op == 9:
            n = int(rng.integers(0, 6))
            assert s.slice_lend(n) == o.lend(n)
        elif live:
            batch = [int(x) for x in rng.permutation(sorted(live))[: int(rng.integers(1, len(live) + 1))]]
            rc2, r2, k2 = o.gather(0, batch, None, None)
            rc1, r1, k1 = s.slice_get_resolved(batch)
            assert rc1 == rc2 and (rc1 != 0 or (k1 == k2 and (r1 == r2).all()))
        for q in live:
            assert s.slice_get_block_table(q)[1].tolist() == o.block_table(q)[1].tolist()
        assert sorted(s.slice_get_free_stack(B.TIER_LOCAL).tolist()) == sorted(o.free_stack(oracle.LOCAL).tolist())
        assert sorted(s.slice_get_free_stack(B.TIER_LENT).tolist()) == sorted(o.free_stack(oracle.LENT).tolist())
        assert s.slice_stats()["lent_capacity"] == o.lent_capacity
    assert moved > 0 and evicted > 0
    s.close()


def test_layout_and_group_configurations_are_validated():
    ok = dict(lent_blocks_physical=20, max_seqs=4, max_blocks_per_seq=8, flags=B.FLAG_NULL_DEVICE)
    B.Slice(8, 8, 20, 20, 8, slab_blocks=10, layer_group=4, layout=B.LAYOUT_LAYER_GROUP_MAJOR, **ok).close()
    B.Slice(8, 8, 20, 20, 8, slab_blocks=5, layer_group=2, layout=B.LAYOUT_SLAB_MAJOR, **ok).close()
    B.Slice(8, 8, 23, 20, 8, slab_blocks=10, layer_group=3, **ok).close()       # layer-major: no divisibility needed
    for bad in (dict(layout=3), dict(layout=1), dict(layout=2, slab_blocks=10, layer_group=3),
                dict(layout=1, slab_blocks=7), dict(layer_group=9), dict(layout=1, slab_blocks=10, lent_block_stride=65536),
                dict(slab_blocks=4, local_free_order=np.arange(20, dtype=np.uint32))):
        with pytest.raises(B.SliceError):
            B.Slice(8, 8, 20, 20, 8, **{**ok, **bad})


@pytest.mark.parametrize("group,ring,layers,first,second", [(1, 2, 8, 9, 8), (4, 2, 8, 8, 0), (2, 2, 8, 10, 8), (2, 3, 7, 8, 2),
                                                            (4, 1, 8, 12, 8), (3, 2, 5, 5, 0)])
def test_decode_step_prefetches_one_layer_group_ahead(group, ring, layers, first, second):
    """Layer groups (Section 4.2.2): a ring slot holds one group, the pass fetches layer l + k while
    layer l runs and the first group of the next pass at its end. Tables-only mode, every pipeline:
    the counts are worked out by hand. (1,2,8): layer 0, then 1..7 inside the pass, then layer 0 again
    = 9, later passes 8. (4,2,8) and (3,2,5): the ring holds the whole model, every layer is fetched
    once and stays. (2,2,8): 0,1 then 2..7 then 0,1 = 10, later 8. (2,3,7): six layer slots for
    seven layers: 0,1 then 2..6, layer 6 displacing layer 0, which is fetched again once layer 6 has
    been attended to = 8; later passes fetch only those two.
    (4,1,8): a ring of one group: every fetch follows the attention that frees its slot: 12, later 8."""
    for mode in (0, 1, 2, 3):
        s = B.Slice(layers, 4, 64, 64, 64, lent_blocks_physical=64, ring_slots=ring, max_seqs=8, max_blocks_per_seq=64,
                    flags=B.FLAG_NULL_DEVICE, pipeline_mode=mode, layer_group=group)
        for i in range(3):
            for b in range(10):
                assert s.slice_alloc_blocks(i, 1, B.TIER_LENT if b % 2 else B.TIER_LOCAL)[0] == B.OK
            assert s.slice_set_seq_len(i, 150) == B.OK
        seqs = np.arange(3, dtype=np.int32)
        assert s.slice_decode_step(seqs, None, 16, 0.1, None, False, True, None, None) == B.OK
        st1 = s.slice_stats()
        assert st1["prefetch_calls"] == first and st1["decode_calls"] == layers, (mode, st1["prefetch_calls"])
        assert s.slice_decode_step(seqs, None, 16, 0.1, None, False, True, None, None) == B.OK
        st2 = s.slice_stats()
        assert st2["prefetch_calls"] - first == second and st2["decode_calls"] == 2 * layers, (mode, st2["prefetch_calls"])
        s.slice_destroy()
