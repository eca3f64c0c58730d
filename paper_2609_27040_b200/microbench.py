"""Microbenchmarks of the copy paths: the gather/scatter kernels over a sweep of block counts
(the prefetch microbenchmark of the measurement plan) and the reclaim migration at serving-like
sizes. Prints one JSON line per case. Run on a B200:

    python -m paper_2609_27040_b200.microbench --what copy
    python -m paper_2609_27040_b200.microbench --what reclaim

Timing: CUDA events on the launching stream, 3 warm-up launches, inputs larger than L2 (or an L2
flush between launches for the small cases). GB/s counts bytes read + bytes written.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

BLOCK_BYTES = 65536
L2_BYTES = 126 << 20


def _time_us(fn, stream, reps, flush=None):
    import torch
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    total = 0.0
    for _ in range(reps):
        if flush is not None:
            flush.add_(1)                      # rewrites a buffer larger than L2
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        stream.wait_stream(torch.cuda.current_stream())
        e0.record(stream)
        fn()
        e1.record(stream)
        e1.synchronize()
        total += e0.elapsed_time(e1) * 1e3
    return total / reps


def copy_sweep(args):
    """Gather of n random 64 KB blocks out of an arena of 2n into a dense destination."""
    import torch
    from paper_2609_27040_b200 import binding as B
    stream = torch.cuda.Stream()
    flush = torch.zeros(160 << 20, dtype=torch.uint8, device="cuda")
    free, _ = torch.cuda.mem_get_info()
    for n in args.blocks:
        need = 3 * n * BLOCK_BYTES
        if need > 0.8 * free:
            print(json.dumps({"case": "copy", "blocks": n, "skipped": f"needs {need / 2**30:.1f} GiB"}), flush=True)
            continue
        src = torch.empty((2 * n, BLOCK_BYTES // 2), dtype=torch.int16, device="cuda")
        src.random_(-30000, 30000)
        dst = torch.zeros((n, BLOCK_BYTES // 2), dtype=torch.int16, device="cuda")
        rng = np.random.default_rng(n)
        idx = torch.from_numpy(rng.permutation(2 * n)[:n].astype(np.int32)).cuda()
        pos = torch.arange(n, dtype=torch.int32, device="cuda")
        moved = 2 * n * BLOCK_BYTES
        use_flush = flush if moved < 4 * L2_BYTES else None
        reps = 20 if n <= 100_000 else 5
        for kind, name in ((1, "copy_blocks_vector"), (2, "copy_blocks_bulk"), (3, "copy_blocks_bulk, 6 stages")):
            for ctas in args.ctas:
                def run():
                    assert B.slice_copy_blocks(dst, pos, src, idx, n, BLOCK_BYTES, kind, ctas, stream) == 0
                us = _time_us(run, stream, reps, use_flush)
                ok = bool(torch.equal(dst, src.index_select(0, idx.long()))) if n <= 100_000 else None
                print(json.dumps({"case": "copy", "kernel": name, "blocks": n, "ctas": ctas or "default", "us": round(us, 1),
                                  "gbs": round(moved / us / 1e3, 1), "bytes_moved": moved, "matches_index_select": ok,
                                  "l2": "flushed" if use_flush is not None else "larger than L2"}), flush=True)

        def ref():
            with torch.cuda.stream(stream):
                torch.index_select(src, 0, idx, out=dst)
        us = _time_us(ref, stream, reps, use_flush)
        print(json.dumps({"case": "copy", "kernel": "torch.index_select (reference line, not product code)", "blocks": n,
                          "us": round(us, 1), "gbs": round(moved / us / 1e3, 1)}), flush=True)
        del src, dst


def reclaim_bench(args):
    """The lender takes `take` block ids of a 32-layer slice whose lent part is fully in use: every
    taken id is migrated (all layers) to a free local id; then the ids are lent again."""
    import torch
    from paper_2609_27040_b200 import binding as B
    Lr, Hkv = 32, 8
    stream = torch.cuda.Stream()
    for take in args.take:
        lent_blocks = 2 * take
        local_blocks = take + 64
        shape = (2, 16, Hkv, 128)
        local = torch.empty((Lr, local_blocks) + shape, dtype=torch.bfloat16, device="cuda").normal_()
        lent = torch.empty((Lr, lent_blocks) + shape, dtype=torch.bfloat16, device="cuda").normal_()
        staging = torch.zeros((2, 1) + shape, dtype=torch.bfloat16, device="cuda")
        nseq = 64
        per_seq = lent_blocks // nseq
        s = B.Slice(Lr, Hkv, local_blocks, lent_blocks, 1, local=local, lent=lent, staging=staging, max_seqs=nseq,
                    max_blocks_per_seq=per_seq + 1)
        for i in range(nseq):
            rc, _ = s.slice_alloc_blocks(i, per_seq, B.TIER_LENT)
            assert rc == 0, rc
            assert s.slice_set_seq_len(i, per_seq * 16) == 0
        before = lent.clone()
        tabs_before = [s.slice_get_block_table(i)[1].copy() for i in range(nseq)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        rc, migrated = s.slice_reclaim(take, stream)
        e1.record(stream)
        e1.synchronize()
        assert rc == 0, rc
        ms = e0.elapsed_time(e1)
        # every moved block must hold the bytes it held before
        ok = True
        for i in range(0, nseq, 7):
            tab = s.slice_get_block_table(i)[1]
            for b in range(0, per_seq, 5):
                e0_, e1_ = int(tabs_before[i][b]), int(tab[b])
                new = local[:, e1_] if e1_ >= 0 else lent[:, ~e1_]
                ok = ok and bool(torch.equal(new, before[:, ~e0_]))
        moved = 2 * migrated * Lr * BLOCK_BYTES
        print(json.dumps({"case": "reclaim", "take_block_ids": take, "migrated_block_ids": int(migrated), "layers": Lr,
                          "ms": round(ms, 3), "bytes_moved": moved, "gbs": round(moved / ms / 1e6, 1),
                          "sampled_blocks_intact": ok,
                          "note": "host planning + table rewrite + one batched copy launch, from call to completion"}), flush=True)
        s.slice_destroy()
        del local, lent, before


def growth_bench(args):
    """Bursty KV growth at serving size: Poisson arrivals, one token per sequence per step, blocks
    allocated as sequences grow (local first, then lent), finished sequences freed, the lender taking
    2-8 GB back every 200 steps and lending it again 100 steps later. Where the lender's reclaim has
    no room to migrate into, requests are preempted: by the library (--victims slab: the slab with
    the fewest requests, slice_reclaim_preempt) or by the driver (--victims lifo: the most recently
    admitted sequence, then a retry); a sequence that cannot grow preempts the most recently admitted
    one (cause: out of memory). Preempted requests go back to the head of the queue with what they
    had generated. --cap-window T (steps) turns on the cap after a preemption (Section 5.3).
    Every step = one append launch (all layers) + one decode launch.
    KV contents are whatever the arenas hold (random): only shapes and placement matter for timing."""
    import time
    import torch
    from paper_2609_27040_b200 import binding as B, synth
    Lr, Hq, Hkv, max_batch = 32, 32, 8, 256
    total_ids = int(args.arena_gb * 2**30 / (Lr * BLOCK_BYTES))
    local_blocks = int(total_ids * 0.6)
    lent_blocks = total_ids - local_blocks
    shape = (2, 16, Hkv, 128)
    local = torch.empty((Lr, local_blocks) + shape, dtype=torch.bfloat16, device="cuda")
    lent = torch.empty((Lr, lent_blocks) + shape, dtype=torch.bfloat16, device="cuda")
    for l in range(Lr):
        local[l].normal_()
        lent[l].normal_()
    staging = torch.zeros((2, lent_blocks) + shape, dtype=torch.bfloat16, device="cuda")
    max_blocks = (2048 + 8192) // 16 + 2
    s = B.Slice(Lr, Hkv, local_blocks, lent_blocks, lent_blocks, local=local, lent=lent, staging=staging, max_seqs=max_batch,
                max_blocks_per_seq=max_blocks)
    main, side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    q = torch.empty((Lr, max_batch, Hq, 128), dtype=torch.bfloat16, device="cuda").normal_()
    out = torch.zeros_like(q)
    knew = torch.empty((Lr, max_batch, Hkv, 128), dtype=torch.bfloat16, device="cuda").normal_()
    rng = np.random.default_rng(args.seed)
    arrivals = synth.bursty_arrivals(args.seed, args.steps)
    by_step = {}
    for a in arrivals:
        by_step.setdefault(a.step, []).append(a)
    waiting, active, length, remaining = [], [], {}, {}
    next_id = taken = tokens = preempted = enospc = capped = 0
    assert s.slice_set_preempt_window(args.cap_window) == 0

    def requeue(victim, t):
        waiting.insert(0, synth.Arrival(t, length[victim], remaining[victim]))
        del length[victim], remaining[victim]
    alloc_s = 0.0
    reclaims, lent_frac = [], []
    scale = 1.0 / float(np.sqrt(128))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    e0.record(main)
    for t in range(args.steps):
        waiting += by_step.get(t, [])
        t_a = time.perf_counter()
        assert s.slice_set_time(t) == 0
        while waiting and len(active) < max_batch:
            a = waiting[0]
            need = synth.blocks_for(a.prompt_len)
            rc, _ = s.slice_alloc_blocks(next_id, need, B.TIER_AUTO)
            if rc in (B.ENOSPC, B.ECAPPED):  # a failing call changes nothing: the request keeps waiting
                capped += rc == B.ECAPPED
                break
            assert rc == 0, rc
            assert s.slice_set_seq_len(next_id, a.prompt_len) == 0
            waiting.pop(0)
            active.append(next_id)
            length[next_id], remaining[next_id] = a.prompt_len, a.output_len
            next_id += 1
        if t and t % 200 == 0:
            take = int(rng.uniform(2, 8) * 2**30 / (Lr * BLOCK_BYTES))
            r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            r0.record(main)
            h0 = time.perf_counter()
            n_victims = 0
            if args.victims == "slab":
                rc, victims, mig = s.slice_reclaim_preempt(take, args.slab, main)
                for victim in victims:
                    active.remove(victim)
                    requeue(victim, t)
                n_victims = len(victims)
            else:
                rc, mig = s.slice_reclaim(take, main)
                while rc == B.ENOSPC and active:  # no room for the blocks in use up there: preempt and retry
                    victim = active.pop()
                    assert s.slice_preempt_seq(victim, B.PREEMPT_RECLAIM) == 0
                    requeue(victim, t)
                    n_victims += 1
                    rc, mig = s.slice_reclaim(take, main)
            host_ms = (time.perf_counter() - h0) * 1e3
            preempted += n_victims
            r1.record(main)
            r1.synchronize()
            if rc == 0:
                taken = take
                reclaims.append({"step": t, "take_ids": take, "migrated_ids": int(mig), "preempted": n_victims,
                                 "host_ms": round(host_ms, 3), "ms": round(r0.elapsed_time(r1), 3),
                                 "gbs": round(2 * mig * Lr * BLOCK_BYTES / r0.elapsed_time(r1) / 1e6, 1)})
            else:
                reclaims.append({"step": t, "take_ids": take, "rc": rc})
        if t % 200 == 100 and taken:
            assert s.slice_lend(taken) == 0
            taken = 0
        for i in list(active):
            if i not in length:
                continue
            if length[i] % 16 == 0:
                while s.slice_alloc_blocks(i, 1, B.TIER_AUTO)[0] != 0:
                    enospc += 1
                    victim = active[-1]
                    assert s.slice_preempt_seq(victim, B.PREEMPT_OOM) == 0
                    active.remove(victim)
                    requeue(victim, t)
                    preempted += 1
                    if victim == i:
                        break
                if i not in length:
                    continue
            length[i] += 1
            assert s.slice_set_seq_len(i, length[i]) == 0
        alloc_s += time.perf_counter() - t_a
        if not active:
            continue
        seqs = np.array(active, np.int32)
        n = len(active)
        kn = knew if n == max_batch else knew[:, :n].contiguous()
        assert s.slice_append_kv(B.ALL_LAYERS, seqs, kn, kn, main) == 0
        assert s.slice_decode_step(seqs, q[:, :n].contiguous() if n != max_batch else q, Hq, scale, out[:, :n].contiguous() if n != max_batch else out,
                                   False, True, main, side) == 0
        tokens += n
        if t % 50 == 0:
            st = s.slice_stats()             # reads the device status word: synchronises
            lent_frac.append(round(st["lent_used"] / max(st["lent_used"] + st["local_used"], 1), 3))
        for i in list(active):
            remaining[i] -= 1
            if remaining[i] <= 0:
                assert s.slice_free_seq(i) == 0
                active.remove(i)
                del length[i], remaining[i]
    e1.record(main)
    e1.synchronize()
    wall = time.perf_counter() - wall0
    st = s.slice_stats()
    print(json.dumps({"case": "bursty_growth", "steps": args.steps, "arena_gb": args.arena_gb, "block_ids": total_ids,
                      "decoded_tokens": tokens, "tokens_per_s": round(tokens / wall, 1), "wall_s": round(wall, 3),
                      "gpu_stream_s": round(e0.elapsed_time(e1) / 1e3, 3), "sequences_admitted": next_id,
                      "host_allocator_us_per_step": round(alloc_s / args.steps * 1e6, 1),
                      "victims": args.victims, "slab_blocks": args.slab, "cap_window_steps": args.cap_window,
                      "enospc": enospc, "capped_admissions": capped, "preempted": preempted,
                      "preempted_by_cause": {k: v for k, v in s.slice_preempt_stats().items() if k.startswith("preempt_")},
                      "reclaims": reclaims, "lent_fraction_every_50_steps": lent_frac,
                      "device_status": st["device_status"], "plans_built": st.get("plans_built")}), flush=True)
    s.slice_destroy()


def transfer_size_sweep(args):
    """Effective bandwidth of a gather against the size of its contiguous pieces (Section 4.2: small
    fragments lower the effective bandwidth B, hence slabs and layer groups: pieces of S..mS, kS or
    kS..mkS bytes). The same total is gathered as n scattered pieces of c bytes each, for c from 4 KB
    to 16 MB (64 KB = one KV block of one layer; 640 KB = a slab of 10; 2.5 MB = a slab of 10 times a
    group of 4 layers), out of an arena twice as large, over both links: HBM to HBM and pinned host
    memory to HBM."""
    import torch
    from paper_2609_27040_b200 import binding as B
    stream = torch.cuda.Stream()
    flush = torch.zeros(160 << 20, dtype=torch.uint8, device="cuda")
    sizes = [4 << 10, 16 << 10, 64 << 10, 256 << 10, 640 << 10, 2560 << 10, 16 << 20]
    for link, total in (("hbm", 1 << 30), ("pinned_host", 256 << 20)):
        arena = torch.empty(2 * total // 2, dtype=torch.int16, device="cuda" if link == "hbm" else "cpu")
        arena.random_(-30000, 30000)
        if link != "hbm":
            arena = arena.pin_memory()
        dst = torch.zeros(total // 2, dtype=torch.int16, device="cuda")
        for c in sizes:
            n = total // c
            rng = np.random.default_rng(c)
            idx = torch.from_numpy(rng.permutation(2 * total // c)[:n].astype(np.int32)).cuda()
            pos = torch.arange(n, dtype=torch.int32, device="cuda")
            for kind, name in ((1, "copy_blocks_vector"), (2, "copy_blocks_bulk"), (3, "copy_blocks_bulk, 6 stages")):
                for ctas in ((0,) if link == "hbm" else (8, 0)):
                    def run():
                        assert B.slice_copy_blocks(dst, pos, arena, idx, n, c, kind, ctas, stream) == 0
                    us = _time_us(run, stream, 10 if link == "hbm" else 3, flush)
                    ok = None
                    if c >= 64 << 10:
                        got = dst[: n * c // 2].view(n, c // 2)
                        want = arena[: (2 * total // c) * c // 2].view(-1, c // 2).index_select(0, idx.long().to(arena.device))
                        ok = bool(torch.equal(got.cpu() if link != "hbm" else got, want))
                    print(json.dumps({"case": "transfer_size", "link": link, "kernel": name, "ctas": ctas or "default",
                                      "piece_bytes": c, "pieces": n, "us": round(us, 1),
                                      "gbs_read": round(n * c / us / 1e3, 1), "matches_index_select": ok}), flush=True)
        del arena, dst


def multislice_bench(args):
    """One compute process with several slices (Section 5: one per peer) at serving size. Every
    slice has a local half and a half in its peer's memory; each peer's own use of its half follows
    a square wave with its own period (busy: it takes memory back, reclaim by preemption; idle: it
    lends again) and is reported to the slice. Arriving requests are sent to a slice by --policy:
    gll (Section 5.2, smallest combined utilisation), random, or round_robin; a request whose slice
    has no room waits. Sequences grow on their slice; one that cannot grow preempts the most recently
    admitted one of the same slice. Every step = per slice with work one append launch and one
    decode launch. Reports tokens/s and the preemptions by cause, summed over the slices."""
    import time
    import torch
    from paper_2609_27040_b200 import binding as B, synth
    Lr, Hq, Hkv, max_batch, ns = 32, 32, 8, 256, args.slices
    ids = int(args.arena_gb * 2**30 / (Lr * BLOCK_BYTES)) // ns
    half = ids // 2
    shape = (2, 16, Hkv, 128)
    max_blocks = (2048 + 8192) // 16 + 2
    slices, keep = [], []
    for k in range(ns):
        local = torch.empty((Lr, half) + shape, dtype=torch.bfloat16, device="cuda")
        lent = torch.empty((Lr, half) + shape, dtype=torch.bfloat16, device="cuda")
        for l in range(Lr):
            local[l].normal_()
            lent[l].normal_()
        staging = torch.zeros((2, half) + shape, dtype=torch.bfloat16, device="cuda")
        keep.append((local, lent, staging))
        slices.append(B.Slice(Lr, Hkv, half, half, half, local=local, lent=lent, staging=staging, max_seqs=max_batch,
                              max_blocks_per_seq=max_blocks))
    main, side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    q = torch.empty((Lr, max_batch, Hq, 128), dtype=torch.bfloat16, device="cuda").normal_()
    out = torch.zeros_like(q)
    knew = torch.empty((Lr, max_batch, Hkv, 128), dtype=torch.bfloat16, device="cuda").normal_()
    rng = np.random.default_rng(args.seed)
    by_step = {}
    for a in synth.bursty_arrivals(args.seed, args.steps, rate=args.rate):
        by_step.setdefault(a.step, []).append(a)
    period = [240 + 90 * k for k in range(ns)]                 # peers are busy at different times
    busy_frac = [0.9, 0.6, 0.75, 0.5, 0.8, 0.7, 0.65, 0.85][:ns]
    peer_used = [int(0.1 * half)] * ns
    for k in range(ns):                                          # what the peer uses it does not lend
        assert slices[k].slice_reclaim(peer_used[k], main)[0] == 0
        assert slices[k].slice_set_peer_used(peer_used[k]) == 0
    waiting, active, home, length, remaining = [], [[] for _ in range(ns)], {}, {}, {}
    next_id = tokens = enospc = waits = rr = 0
    scale = 1.0 / float(np.sqrt(128))

    def requeue(victim, t):
        waiting.insert(0, synth.Arrival(t, length[victim], remaining[victim]))
        active[home[victim]].remove(victim)
        del length[victim], remaining[victim], home[victim]

    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    for t in range(args.steps):
        waiting += by_step.get(t, [])
        for k in range(ns):                                      # the peers' own demand
            want = int((busy_frac[k] if (t // period[k]) % 2 == 1 else 0.1) * half)
            if want > peer_used[k]:
                rc, victims, _ = slices[k].slice_reclaim_preempt(want - peer_used[k], args.slab, main)
                assert rc == 0, rc
                for v in victims:
                    requeue(v, t)
            elif want < peer_used[k]:
                assert slices[k].slice_lend(peer_used[k] - want) == 0
            peer_used[k] = want
            assert slices[k].slice_set_peer_used(want) == 0
        while waiting and sum(len(a) for a in active) < max_batch:
            a = waiting[0]
            if args.policy == "gll":
                k = B.slice_schedule_gll(slices)
            elif args.policy == "random":
                k = int(rng.integers(ns))
            else:
                k, rr = rr % ns, rr + 1
            rc, _ = slices[k].slice_alloc_blocks(next_id, synth.blocks_for(a.prompt_len), B.TIER_AUTO)
            if rc != 0:
                waits += 1
                break
            assert slices[k].slice_set_seq_len(next_id, a.prompt_len) == 0
            waiting.pop(0)
            active[k].append(next_id)
            home[next_id], length[next_id], remaining[next_id] = k, a.prompt_len, a.output_len
            next_id += 1
        for k in range(ns):
            for i in list(active[k]):
                if i not in length:
                    continue
                if length[i] % 16 == 0:
                    while slices[k].slice_alloc_blocks(i, 1, B.TIER_AUTO)[0] != 0:
                        enospc += 1
                        victim = active[k][-1]
                        assert slices[k].slice_preempt_seq(victim, B.PREEMPT_OOM) == 0
                        requeue(victim, t)
                        if victim == i:
                            break
                    if i not in length:
                        continue
                length[i] += 1
                assert slices[k].slice_set_seq_len(i, length[i]) == 0
            n = len(active[k])
            if not n:
                continue
            seqs = np.array(active[k], np.int32)
            kn = knew if n == max_batch else knew[:, :n].contiguous()
            assert slices[k].slice_append_kv(B.ALL_LAYERS, seqs, kn, kn, main) == 0
            assert slices[k].slice_decode_step(seqs, q if n == max_batch else q[:, :n].contiguous(), Hq, scale,
                                               out if n == max_batch else out[:, :n].contiguous(), False, True, main, side) == 0
            tokens += n
            for i in list(active[k]):
                remaining[i] -= 1
                if remaining[i] <= 0:
                    assert slices[k].slice_free_seq(i) == 0
                    active[k].remove(i)
                    del length[i], remaining[i], home[i]
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    ps = [sl.slice_preempt_stats() for sl in slices]
    st = [sl.slice_stats() for sl in slices]
    print(json.dumps({"case": "multislice", "policy": args.policy, "arrivals_per_step": args.rate, "slices": ns, "steps": args.steps, "arena_gb": args.arena_gb,
                      "block_ids_per_slice": ids, "decoded_tokens": tokens, "tokens_per_s": round(tokens / wall, 1),
                      "wall_s": round(wall, 3), "sequences_admitted": next_id, "admission_waits": waits,
                      "preempt_oom": sum(p["preempt_oom"] for p in ps), "preempt_reclaim": sum(p["preempt_reclaim"] for p in ps),
                      "migrated_blocks": sum(x["migrated_blocks"] for x in st),
                      "device_status": [x["device_status"] for x in st]}), flush=True)
    for sl in slices:
        sl.slice_destroy()


def link_point(f: float, seed: int = 0, layers: int = 8, reps: int = 10) -> dict:
    """One point of the link measurement: the Llama-3-8B-shaped batch on `layers` layers with a
    fraction f of every sequence's blocks in a lent arena in pinned host memory (lent_kind = 1, the
    prefetch crosses PCIe). Returns the lent bytes per layer, the time per layer of the one-launch
    pass and the link rate measured with the stand-alone gather from the same arena."""
    import dataclasses
    import torch
    from paper_2609_27040_b200 import binding as B, synth
    Lr = layers
    wl = dataclasses.replace(synth.WORKLOADS["llama3_8b_decode"], num_layers=Lr, lent_fraction=f)
    pl = synth.make_placement(wl, seed, slack_blocks=64)
    shape = (2, 16, wl.num_kv_heads, 128)
    local = torch.empty((Lr, pl.local_blocks) + shape, device="cuda", dtype=torch.bfloat16).normal_()
    lent = torch.empty((Lr, max(pl.lent_blocks, 1)) + shape, dtype=torch.bfloat16).normal_().pin_memory()
    staging = torch.zeros((2, max(pl.staging_blocks, 1)) + shape, device="cuda", dtype=torch.bfloat16)
    q = torch.empty((Lr, wl.batch, wl.num_q_heads, 128), device="cuda", dtype=torch.bfloat16).normal_()
    out = torch.zeros_like(q)
    s = B.Slice(Lr, wl.num_kv_heads, pl.local_blocks, pl.lent_blocks, pl.staging_blocks, local=local, lent=lent,
                staging=staging, max_seqs=wl.batch, max_blocks_per_seq=300, lent_kind=1,
                local_free_order=pl.local_free_order, lent_free_order=pl.lent_free_order)
    for i, hints in enumerate(pl.hints):
        for h in hints:
            assert s.slice_alloc_blocks(i, 1, int(h))[0] == 0
        assert s.slice_set_seq_len(i, int(pl.lengths[i])) == 0
    seqs = np.arange(wl.batch, dtype=np.int32)
    main, side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    scale = 1.0 / float(np.sqrt(128))
    m = pl.staging_blocks * BLOCK_BYTES
    link_gbs = None
    if m:
        def gather():
            assert s.prefetch_layer(3, seqs, main) == 0
            assert s.prefetch_layer(5, seqs, main) == 0      # same slot, other layer: always a real copy
        us = _time_us(gather, main, 5) / 2
        link_gbs = m / us / 1e3
    for _ in range(3):
        assert s.slice_decode_step(seqs, q, wl.num_q_heads, scale, out, False, True, main, side) == 0
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(main)
    for _ in range(reps):
        assert s.slice_decode_step(seqs, q, wl.num_q_heads, scale, out, False, True, main, side) == 0
    e1.record(main)
    e1.synchronize()
    row = {"f": f, "lent_bytes_per_layer": m, "us_per_layer": e0.elapsed_time(e1) * 1e3 / reps / Lr,
           "link_gbs": link_gbs, "device_status": s.slice_stats()["device_status"],
           "kv_bytes_per_layer": int(pl.lengths.sum()) * wl.kv_bytes_per_token}
    s.slice_destroy()
    del local, lent, staging
    torch.cuda.empty_cache()
    return row


def link_bench(args):
    """The paper's transparency condition (Section 2.3 / 4: a transfer of m bytes over a link of
    bandwidth B is hidden when it fits in the latency window L between two uses, B*L >= m) with a
    real bandwidth-limited link: the lent arena lives in pinned host memory (lent_kind = 1), so the
    prefetch crosses PCIe. For a sweep of lent fractions f: measured time per layer of the one-launch
    pass against the model max(T0, m/B), T0 = time per layer with nothing lent, m = lent bytes per
    layer, B = link rate measured with the stand-alone gather from the same arena."""
    from paper_2609_27040_b200 import capacity
    rows = [link_point(f, args.seed) for f in args.fractions]
    t0 = min(r["us_per_layer"] for r in rows if r["lent_bytes_per_layer"] == 0) if any(r["lent_bytes_per_layer"] == 0 for r in rows) else None
    rates = [r["link_gbs"] for r in rows if r["link_gbs"]]
    link = max(rates) if rates else None
    for r in rows:
        if t0 is not None and link:
            pred = capacity.layer_time(t0, r["lent_bytes_per_layer"], link * 1e3)   # us, bytes, bytes per us
            r.update({"model_us_per_layer": round(pred, 1), "stall_us_measured": round(r["us_per_layer"] - t0, 1),
                      "stall_us_model": round(pred - t0, 1), "measured_over_model": round(r["us_per_layer"] / pred, 3)})
        r["us_per_layer"] = round(r["us_per_layer"], 1)
        r["link_gbs"] = round(r["link_gbs"], 1) if r["link_gbs"] else None
        print(json.dumps({"case": "link", **r}), flush=True)
    if t0 is not None and link:
        bytes_layer = 614.3e6
        print(json.dumps({"case": "link_summary", "T0_us_per_layer": round(t0, 1), "link_gbs": round(link, 1),
                          "knee_lent_bytes_per_layer": round(link * 1e3 * t0), "knee_fraction_of_kv": round(link * 1e3 * t0 / bytes_layer, 4),
                          "model": "time per layer = max(T0, m / B_link): the transfer is hidden while B*L >= m"}), flush=True)


def layout_sweep(args):
    """Section 4.2 / Figure "Throughput under Different Group and Slab Size", on this machine: the
    one-launch pass over 16 layers of the Llama-3-8B-shaped batch with the slab allocator (slab sizes
    1..100, and the block-granular free stack with a seeded order as the scattered extreme), layer
    groups of 1 and 4, the layer-major and layer-group-major orders, 8 / 2 / 1 KV heads (64 / 16 /
    8 KB blocks), the lent arena in HBM and behind PCIe (pinned host memory). Blocks are allocated
    either request by request (a prompt's blocks at once) or interleaved over the requests (growth
    during decoding). Reports time per layer, the algorithmic rate and the mean length of the runs
    the fused gather could copy as one unit (neighbours in the arena and in the slot, <= 64 KB)."""
    import dataclasses
    import torch
    from paper_2609_27040_b200 import binding as B, synth
    Lr = 16      # more layers than the ring has layer slots (2 groups of up to 4), so every layer is fetched in every pass
    for link in args.links:
        for hkv in args.kv_heads:
            base = dataclasses.replace(synth.WORKLOADS["llama3_8b_decode"], num_layers=Lr, num_kv_heads=hkv,
                                       num_q_heads=4 * hkv, lent_fraction=0.4 if link == "hbm" else 0.02)
            bb = base.block_bytes
            for order in ("per_request", "interleaved"):
                for slab, group, layout in [(0, 1, 0), (1, 1, 0), (10, 1, 0), (10, 4, 0), (10, 4, 2), (10, 4, 1), (100, 4, 2), (100, 1, 0)]:
                    pl = synth.make_placement(base, args.seed, slack_blocks=64, permute=slab == 0)
                    nl, nr = pl.local_blocks, pl.lent_blocks
                    if slab:
                        nl, nr = -(-nl // slab) * slab, -(-nr // slab) * slab
                    shape = (2, 16, hkv, 128)
                    local = torch.empty((Lr, nl) + shape, device="cuda", dtype=torch.bfloat16).normal_()
                    if link == "hbm":
                        lent = torch.empty((Lr, nr) + shape, device="cuda", dtype=torch.bfloat16).normal_()
                    else:
                        lent = torch.empty((Lr, nr) + shape, dtype=torch.bfloat16).normal_().pin_memory()
                    staging = torch.zeros((2 * group, max(pl.staging_blocks, 1)) + shape, device="cuda", dtype=torch.bfloat16)
                    q = torch.empty((Lr, base.batch, base.num_q_heads, 128), device="cuda", dtype=torch.bfloat16).normal_()
                    out = torch.zeros_like(q)
                    s = B.Slice(Lr, hkv, nl, nr, pl.staging_blocks, local=local, lent=lent, staging=staging, max_seqs=base.batch,
                                max_blocks_per_seq=300, lent_kind=int(link != "hbm"), slab_blocks=slab, layer_group=group,
                                layout=layout, local_free_order=pl.local_free_order, lent_free_order=pl.lent_free_order)
                    if order == "per_request":
                        for i, hints in enumerate(pl.hints):
                            for h in hints:
                                assert s.slice_alloc_blocks(i, 1, int(h))[0] == 0
                    else:
                        for b in range(max(len(h) for h in pl.hints)):
                            for i, hints in enumerate(pl.hints):
                                if b < len(hints):
                                    assert s.slice_alloc_blocks(i, 1, int(hints[b]))[0] == 0
                    for i in range(base.batch):
                        assert s.slice_set_seq_len(i, int(pl.lengths[i])) == 0
                    # runs of lent blocks that are neighbours by id and in the staging order
                    ids = [~int(e) for i in range(base.batch) for e in s.slice_get_block_table(i)[1] if e < 0]
                    runs, cap = [], max(1, min(8, 65536 // bb))
                    for a, b2 in zip([None] + ids[:-1], ids):
                        if a is not None and b2 == a + 1 and runs[-1] < cap:
                            runs[-1] += 1
                        else:
                            runs.append(1)
                    seqs = np.arange(base.batch, dtype=np.int32)
                    main, side = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
                    scale = 1.0 / float(np.sqrt(128))
                    for _ in range(3):
                        assert s.slice_decode_step(seqs, q, base.num_q_heads, scale, out, False, True, main, side) == 0
                    torch.cuda.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    reps = 10
                    fetched0 = s.slice_stats()["prefetched_bytes"]
                    e0.record(main)
                    for _ in range(reps):
                        assert s.slice_decode_step(seqs, q, base.num_q_heads, scale, out, False, True, main, side) == 0
                    e1.record(main)
                    e1.synchronize()
                    us = e0.elapsed_time(e1) * 1e3 / reps / Lr
                    tokens = int(pl.lengths.sum())
                    fetched = (s.slice_stats()["prefetched_bytes"] - fetched0) / reps / Lr      # gathered per layer, as counted by the library
                    algo = tokens * base.kv_bytes_per_token + 2 * fetched
                    print(json.dumps({"case": "layouts", "link": link, "kv_heads": hkv, "block_kb": bb // 1024, "alloc": order,
                                      "slab": slab or "stack, seeded order", "group": group,
                                      "layout": ["layer-major", "slab-major", "layer-group-major"][layout],
                                      "us_per_layer": round(us, 1), "algorithmic_gbs": round(algo / us / 1e3, 1),
                                      "lent_mb_per_layer": round(pl.staging_blocks * bb / 1e6, 1), "gathered_mb_per_layer": round(fetched / 1e6, 1),
                                      "mean_blocks_per_copy_unit": round(float(np.mean(runs)), 2) if runs else None,
                                      "device_status": s.slice_stats()["device_status"]}), flush=True)
                    s.slice_destroy()
                    del local, lent, staging, q, out
                    torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--what", choices=["copy", "reclaim", "growth", "link", "size", "multislice", "layouts", "all"], default="all")
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--arena-gb", type=float, default=48.0)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--fractions", type=float, nargs="*", default=[0.0, 0.002, 0.005, 0.01, 0.02, 0.05, 0.1, 0.2])
    ap.add_argument("--blocks", type=int, nargs="*", default=[1_000, 10_000, 100_000, 400_000])
    ap.add_argument("--ctas", type=int, nargs="*", default=[0, 148, 592])
    ap.add_argument("--take", type=int, nargs="*", default=[954, 3815])
    ap.add_argument("--victims", choices=["slab", "lifo"], default="slab")
    ap.add_argument("--slab", type=int, default=10, help="blocks per slab for the victim rule (the paper's default)")
    ap.add_argument("--slices", type=int, default=3, help="multislice: slices of the one compute process (at most 8)")
    ap.add_argument("--rate", type=float, default=0.5, help="multislice: mean arrivals per step (Poisson)")
    ap.add_argument("--policy", choices=["gll", "random", "round_robin"], default="gll")
    ap.add_argument("--cap-window", type=int, default=0, help="steps a cap holds after a preemption by reclamation")
    ap.add_argument("--links", nargs="*", default=["hbm", "host"], help="layouts: where the lent arena lives")
    ap.add_argument("--kv-heads", type=int, nargs="*", default=[8, 2, 1], help="layouts: KV heads (block = 8 KB per head)")
    args = ap.parse_args()
    from paper_2609_27040_b200 import binding as B
    B.lib()                                    # fails loudly when the CUDA library is missing
    if args.what in ("copy", "all"):
        copy_sweep(args)
    if args.what in ("reclaim", "all"):
        reclaim_bench(args)
    if args.what == "growth":
        growth_bench(args)
    if args.what == "link":
        link_bench(args)
    if args.what == "size":
        transfer_size_sweep(args)
    if args.what == "multislice":
        multislice_bench(args)
    if args.what == "layouts":
        layout_sweep(args)


if __name__ == "__main__":
    main()
