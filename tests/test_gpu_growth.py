"""Tiny replica of the bursty-growth workload: sequences arrive, grow by one token per decode step
(allocating a block whenever a block fills up), finish and are freed, while the lender takes blocks
back and lends them again. Every step the CUDA library and the oracle go through the same calls;
tables and free stacks are compared after every change, attention of every layer after every decode
step, and the arenas byte by byte at the end. Exercises allocator, append, prefetch + attention in
one launch per pass, reclaim migration and lend together, on state that neither side starts from."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from paper_2609_27040_b200 import binding as B
from paper_2609_27040_b200 import synth
from tests.helpers import attention_close

pytestmark = pytest.mark.gpu

ATOL = RTOL = 1e-2
L, HQ, HKV, D, T = 2, 16, 4, 128, 16
LOCAL, LENT, MAXSEQ, MAXBLK, STEPS = 36, 36, 8, 16, 60


def _tables_equal(s, orc, ids):
    for i in ids:
        rc, t, ln = s.slice_get_block_table(i)
        rc2, t2, ln2 = orc.block_table(i)
        assert rc == rc2 == 0 and ln == ln2 and t.tolist() == t2.tolist()
    assert s.slice_get_free_stack(B.TIER_LOCAL).tolist() == orc.free_stack(1).tolist()
    assert s.slice_get_free_stack(B.TIER_LENT).tolist() == orc.free_stack(2).tolist()
    assert s.slice_stats()["lent_capacity"] == orc.lent_capacity


@pytest.mark.parametrize("pipeline_mode,static_split", [(0, 0), (0, 1), (1, 0)])
def test_bursty_growth_replica_matches_oracle(pipeline_mode, static_split):
    import torch
    from tests.gpu_helpers import kv_to_dev, kv_to_host, to_dev

    oracle.build()
    rng = np.random.default_rng(31)
    blk_shape = (2, T, HKV, D)
    bb = int(np.prod(blk_shape)) * 2
    local = synth.normal_bf16_bits(rng, (L, LOCAL) + blk_shape)
    lent = synth.normal_bf16_bits(rng, (L, LENT) + blk_shape)
    staging = np.zeros((2, LENT) + blk_shape, np.uint16)
    g_local, g_lent, g_staging = kv_to_dev(local), kv_to_dev(lent), kv_to_dev(staging)
    orc = oracle.OracleSlice(L, T, bb, LOCAL, LENT, LENT, 2, LENT, max_seqs=MAXSEQ, max_blocks_per_seq=MAXBLK)
    s = B.Slice(L, HKV, LOCAL, LENT, LENT, local=g_local, lent=g_lent, staging=g_staging, max_seqs=MAXSEQ,
                max_blocks_per_seq=MAXBLK, pipeline_mode=pipeline_mode, static_split=static_split, decode_ctas=12)
    main, side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    scale = 1.0 / float(np.sqrt(D))

    arrivals = synth.bursty_arrivals(5, STEPS, rate=0.6, prompt_lo=3, prompt_hi=70, out_median=18.0, out_sigma=0.8,
                                     out_clip=50)
    waiting, active, remaining = [], [], {}
    next_id, taken, decode_steps, reclaims, preempted = 0, 0, 0, 0, 0

    def free_both(i):
        assert s.slice_free_seq(i) == orc.free_seq(i) == 0
        active.remove(i)
        del remaining[i]

    def alloc_both(i, hint=oracle.AUTO):
        rc, _ = s.slice_alloc_blocks(i, 1, B.TIER_AUTO)
        rc2, _ = orc.alloc_blocks(i, 1, hint)
        assert rc == rc2
        return rc

    for t in range(STEPS):
        waiting += [a for a in arrivals if a.step == t]
        # ---- admission: allocate the prompt's blocks and write the prompt's KV into them ----
        while waiting and len(active) < MAXSEQ:
            a = waiting[0]
            i = next_id
            need = synth.blocks_for(a.prompt_len)
            ok = True
            for _ in range(need):
                if alloc_both(i) != 0:
                    ok = False
                    break
            if not ok:
                if s.slice_get_block_table(i)[0] == 0:      # roll the partial allocation back on both sides
                    assert s.slice_free_seq(i) == orc.free_seq(i) == 0
                _tables_equal(s, orc, active)
                break
            waiting.pop(0)
            next_id += 1
            assert s.slice_set_seq_len(i, a.prompt_len) == orc.set_seq_len(i, a.prompt_len) == 0
            active.append(i)
            remaining[i] = a.output_len
            _, tab, _ = orc.block_table(i)
            for layer in range(L):
                for e in tab[:need].tolist():
                    blk = synth.normal_bf16_bits(rng, blk_shape)
                    if e >= 0:
                        local[layer, e] = blk
                        g_local[layer, e] = kv_to_dev(blk)
                    else:
                        lent[layer, ~e] = blk
                        g_lent[layer, ~e] = kv_to_dev(blk)
        # ---- the lender takes blocks back / lends them again ----
        if t % 10 == 5:
            take = int(rng.integers(4, 13))
            rc, mig = orc.reclaim(take, local, lent)
            rc2, mig2 = s.slice_reclaim(take, main)
            assert rc == rc2 and (rc != 0 or mig == mig2)
            if rc == 0:
                taken += take
                reclaims += 1
            torch.cuda.synchronize()
            _tables_equal(s, orc, active)
        if t % 10 == 0 and taken:
            assert s.slice_lend(taken) == orc.lend(taken) == 0
            taken = 0
            _tables_equal(s, orc, active)
        if not active:
            continue
        # ---- one decode step: every sequence grows by a token ----
        for i in list(active):
            if i not in remaining:
                continue
            ln = orc.block_table(i)[2]
            if ln % T == 0:
                while alloc_both(i) != 0:       # out of blocks: preempt the most recently admitted sequence
                    victim = active[-1]
                    free_both(victim)
                    preempted += 1
                    if victim == i:
                        break
                if i not in remaining:
                    continue
            assert s.slice_set_seq_len(i, ln + 1) == orc.set_seq_len(i, ln + 1) == 0
        if not active:
            continue
        _tables_equal(s, orc, active)
        seqs = np.array(active, np.int32)
        n = len(active)
        k_new = synth.normal_bf16_bits(rng, (L, n, HKV, D))
        v_new = synth.normal_bf16_bits(rng, (L, n, HKV, D))
        for layer in range(L):
            assert orc.append_kv(layer, seqs, k_new[layer], v_new[layer], HKV, D, local, lent, None) == 0
        if static_split:        # every layer in one launch
            assert s.slice_append_kv(B.ALL_LAYERS, seqs, to_dev(k_new), to_dev(v_new), main) == B.OK
        else:
            for layer in range(L):
                assert s.slice_append_kv(layer, seqs, to_dev(k_new[layer]), to_dev(v_new[layer]), main) == B.OK
        q = synth.normal_bf16_bits(rng, (L, n, HQ, D))
        gq = to_dev(q)
        gout = torch.zeros_like(gq)
        assert s.slice_decode_step(seqs, gq, HQ, scale, gout, False, True, main, side) == B.OK
        torch.cuda.synchronize()
        st = s.slice_stats()
        assert st["device_status"] == 0 and st["last_cuda_error"] == 0
        got = gout.view(torch.bfloat16).double().cpu().numpy()
        lens = np.array([orc.block_table(i)[2] for i in active], np.uint32)
        for layer in range(L):
            rc, resolved, k = orc.gather(layer, seqs, lent, staging)
            assert rc == 0
            rc, ref, _ = oracle.paged_attention(q[layer], local[layer], staging[layer % 2], resolved, lens, HQ, HKV, D, T, scale)
            assert rc == 0
            ok, max_abs, max_rel = attention_close(got[layer], ref, ATOL, RTOL)
            assert ok, (t, layer, max_abs, max_rel)
        decode_steps += 1
        for i in list(active):
            remaining[i] -= 1
            if remaining[i] <= 0:
                free_both(i)
        _tables_equal(s, orc, active)
    torch.cuda.synchronize()
    # the run must have exercised what it is for
    assert decode_steps >= 40 and reclaims >= 3 and next_id >= 10
    assert (kv_to_host(g_local) == local).all() and (kv_to_host(g_lent) == lent).all()
    s.slice_destroy()
