"""Random interleavings of the public calls against the oracle: sequences come and go, grow, the
lender takes and gives (with and without preempting requests), and attention is asked for through every entry point (whole pass in one
launch, per-layer prefetch + decode, write-back in between) on whatever state the earlier calls
left. Return codes must agree with the oracle's state machine; every attention result and, at the
end, every arena byte must agree with the oracle."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from paper_2609_27040_b200 import binding as B
from paper_2609_27040_b200 import synth
from tests.helpers import attention_close

pytestmark = pytest.mark.gpu

L, HQ, HKV, D, T = 3, 8, 2, 128, 16
LOCAL, LENT, MAXSEQ, MAXBLK = 28, 30, 6, 12


@pytest.mark.parametrize("seed,mode", [(1, 0), (2, 1), (3, 2), (4, 0), (5, 3)])
def test_random_call_sequences_match_the_oracle(seed, mode):
    import torch
    from tests.gpu_helpers import kv_to_dev, kv_to_host, to_dev

    oracle.build()
    rng = np.random.default_rng(seed)
    blk = (2, T, HKV, D)
    bb = int(np.prod(blk)) * 2
    local = synth.normal_bf16_bits(rng, (L, LOCAL) + blk)
    lent = synth.normal_bf16_bits(rng, (L, LENT) + blk)
    staging = np.zeros((2, LENT) + blk, np.uint16)
    g_local, g_lent, g_staging = kv_to_dev(local), kv_to_dev(lent), kv_to_dev(staging)
    orc = oracle.OracleSlice(L, T, bb, LOCAL, LENT, LENT, 2, LENT, max_seqs=MAXSEQ, max_blocks_per_seq=MAXBLK)
    s = B.Slice(L, HKV, LOCAL, LENT, LENT, local=g_local, lent=g_lent, staging=g_staging, max_seqs=MAXSEQ,
                max_blocks_per_seq=MAXBLK, pipeline_mode=mode, decode_ctas=int(rng.integers(2, 20)),
                static_split=int(seed % 2))
    main, side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    scale = 1.0 / float(np.sqrt(D))
    active, next_id, taken, attended, preempted = [], 0, 0, 0, 0

    def tables_equal():
        for i in active:
            rc, t, ln = s.slice_get_block_table(i)
            rc2, t2, ln2 = orc.block_table(i)
            assert rc == rc2 == 0 and ln == ln2 and t.tolist() == t2.tolist()
        assert s.slice_get_free_stack(B.TIER_LOCAL).tolist() == orc.free_stack(1).tolist()
        assert s.slice_get_free_stack(B.TIER_LENT).tolist() == orc.free_stack(2).tolist()

    def lens_of(ids):
        return np.array([orc.block_table(i)[2] for i in ids], np.uint32)

    def check(got, q, ids, layers):
        lens = lens_of(ids)
        for layer in layers:
            rc, resolved, k = orc.gather(layer, ids, lent, staging)
            assert rc == 0
            rc, ref, _ = oracle.paged_attention(q[layer], local[layer], staging[layer % 2], resolved, lens, HQ, HKV, D, T, scale)
            assert rc == 0
            ok, max_abs, max_rel = attention_close(got[layer], ref, 1e-2, 1e-2)
            assert ok, (layer, max_abs, max_rel)

    for step in range(90):
        op = rng.choice(["arrive", "grow", "free", "reclaim", "lend", "pass", "layers", "writeback"],
                        p=[0.14, 0.22, 0.05, 0.09, 0.06, 0.22, 0.17, 0.05])
        if op == "arrive" and len(active) < MAXSEQ:
            n = int(rng.integers(1, 90))
            need = synth.blocks_for(n)
            hint = int(rng.choice([oracle.AUTO, oracle.LOCAL, oracle.LENT]))
            rc, _ = s.slice_alloc_blocks(next_id, need, hint)
            rc2, _ = orc.alloc_blocks(next_id, need, hint)
            assert rc == rc2
            if rc == 0:
                assert s.slice_set_seq_len(next_id, n) == orc.set_seq_len(next_id, n) == 0
                _, tab, _ = orc.block_table(next_id)
                for layer in range(L):
                    for e in tab[:need].tolist():
                        b = synth.normal_bf16_bits(rng, blk)
                        if e >= 0:
                            local[layer, e] = b
                            g_local[layer, e] = kv_to_dev(b)
                        else:
                            lent[layer, ~e] = b
                            g_lent[layer, ~e] = kv_to_dev(b)
                active.append(next_id)
            next_id += 1
        elif op == "grow" and active:
            ids = [i for i in active if rng.random() < 0.7] or active[:1]
            grown = []
            for i in ids:
                ln = orc.block_table(i)[2]
                if ln % T == 0:
                    if len(orc.block_table(i)[1]) >= MAXBLK:
                        continue
                    rc, _ = s.slice_alloc_blocks(i, 1, B.TIER_AUTO)
                    rc2, _ = orc.alloc_blocks(i, 1, oracle.AUTO)
                    assert rc == rc2
                    if rc != 0:
                        continue
                assert s.slice_set_seq_len(i, ln + 1) == orc.set_seq_len(i, ln + 1) == 0
                grown.append(i)
            if grown:
                seqs = np.array(grown, np.int32)
                k_new = synth.normal_bf16_bits(rng, (L, len(grown), HKV, D))
                v_new = synth.normal_bf16_bits(rng, (L, len(grown), HKV, D))
                for layer in range(L):
                    assert orc.append_kv(layer, seqs, k_new[layer], v_new[layer], HKV, D, local, lent, None) == 0
                if rng.random() < 0.5:
                    assert s.slice_append_kv(B.ALL_LAYERS, seqs, to_dev(k_new), to_dev(v_new), main) == B.OK
                else:
                    for layer in range(L):
                        assert s.slice_append_kv(layer, seqs, to_dev(k_new[layer]), to_dev(v_new[layer]), main) == B.OK
        elif op == "free" and active:
            i = active.pop(int(rng.integers(len(active))))
            assert s.slice_free_seq(i) == orc.free_seq(i) == 0
        elif op == "reclaim" and rng.random() < 0.5:
            take, slab = int(rng.integers(1, 16)), int(rng.integers(1, 6))
            rc, victims, mig = orc.reclaim_preempt(take, slab, local, lent)      # evicts where there is no room
            rc2, victims2, mig2 = s.slice_reclaim_preempt(take, slab, main)
            assert rc == rc2 == 0 and victims == victims2 and mig == mig2
            active = [i for i in active if i not in victims]
            preempted += len(victims)
            taken = LENT - orc.lent_capacity
        elif op == "reclaim":
            take = int(rng.integers(1, 10))
            rc, mig = orc.reclaim(take, local, lent)
            rc2, mig2 = s.slice_reclaim(take, main)
            assert rc == rc2 and (rc != 0 or mig == mig2)
            taken = LENT - orc.lent_capacity          # a take larger than what is lent is clipped
        elif op == "lend" and taken:
            n = int(rng.integers(1, taken + 1))
            assert s.slice_lend(n) == orc.lend(n) == 0
            taken = LENT - orc.lent_capacity
        elif op == "pass" and active:
            ids = [i for i in active if rng.random() < 0.8] or active[:1]
            seqs = np.array(ids, np.int32)
            q = synth.normal_bf16_bits(rng, (L, len(ids), HQ, D))
            gq = to_dev(q)
            gout = torch.zeros_like(gq)
            assert s.slice_decode_step(seqs, gq, HQ, scale, gout, False, bool(rng.integers(2)), main, side) == B.OK
            torch.cuda.synchronize()
            check(gout.view(torch.bfloat16).double().cpu().numpy(), q, ids, range(L))
            attended += 1
        elif op == "layers" and active:
            ids = [i for i in active if rng.random() < 0.8] or active[:1]
            seqs = np.array(ids, np.int32)
            q = synth.normal_bf16_bits(rng, (L, len(ids), HQ, D))
            gq = to_dev(q)
            gout = torch.zeros_like(gq)
            layers = [int(x) for x in rng.permutation(L)[: int(rng.integers(1, L + 1))]]
            for layer in layers:
                assert s.prefetch_layer(layer, seqs, side) == B.OK
                assert s.paged_decode(layer, seqs, gq[layer], HQ, scale, gout[layer], None, main) == B.OK
            torch.cuda.synchronize()
            check(gout.view(torch.bfloat16).double().cpu().numpy(), q, ids, layers)
            attended += 1
        elif op == "writeback" and active:
            ids = list(active)
            seqs = np.array(ids, np.int32)
            layer = int(rng.integers(L))
            assert s.prefetch_layer(layer, seqs, side) == B.OK
            assert s.slice_writeback_layer(layer, seqs, main) == B.OK      # staged copy -> home: no change in bytes
        tables_equal()
        st = s.slice_stats()
        assert st["device_status"] == 0 and st["last_cuda_error"] == 0 and st["lent_capacity"] == orc.lent_capacity
        assert s.slice_preempt_stats()["preempt_reclaim"] == orc.preempt_state()["preempt_reclaim"] == preempted
    torch.cuda.synchronize()
    assert attended >= 5
    assert (kv_to_host(g_local) == local).all() and (kv_to_host(g_lent) == lent).all()
    s.slice_destroy()
