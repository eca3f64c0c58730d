#!/usr/bin/env python
"""Benchmark of the memory-slice hot path: per-layer prefetch of lent KV blocks overlapped with
paged GQA decode attention, on synthetic Llama-3-8B-shaped decode batches.

    python bench.py --gpus N --steps K --warmup W            (one process per GPU under torchrun)
    python bench.py --impl reference ...                      (the CPU oracle, timed as it stands)

A step is one pass of the whole path over one batch: for every layer, the gather of that layer's
lent blocks into the staging ring and the attention over the local arena plus the ring slot. The
metric is decode tokens/s = sequences * steps / time. One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_27040_b200 import synth  # noqa: E402

METRIC = "decode_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="default 200 (reference arm: 5)")
    ap.add_argument("--warmup", type=int, default=None, help="default 10 (reference arm: 1)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama3_8b_decode", choices=sorted(synth.WORKLOADS) + ["prefetch_microbench"],
                    help="a decode workload, or prefetch_microbench: the gather / scatter sweep over launch sizes")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--copy-kind", type=int, default=0)
    ap.add_argument("--copy-ctas", type=int, default=0)
    ap.add_argument("--decode-ctas", type=int, default=0)
    ap.add_argument("--pipeline-mode", type=int, default=0,
                    help="0 one persistent launch per pass, 1 two streams with events, 2 one fused launch per layer, "
                         "3 a chain of launches, one per layer, each starting while the one before it runs")
    ap.add_argument("--static-split", type=int, default=0, help="1: no work stealing between CTAs")
    ap.add_argument("--prefetch-priority", type=int, default=0,
                    help="1: two partial buffers instead of four (CTAs in step, prefetch always ahead, slower pass)")
    ap.add_argument("--no-ablations", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parity-check", action="store_true", help="skip the oracle check of the last timed pass")
    ap.add_argument("--no-microbench", action="store_true", help="skip the short prefetch / migration microbenchmark table")
    ap.add_argument("--no-wrap", action="store_true", help="do not prefetch layer 0 of the next pass")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (debugging)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch (debugging)")
    ap.add_argument("--kv-heads", type=int, default=0,
                    help="override the KV heads, same query heads per KV head (profiling the few-KV-head kernel variants)")
    args = ap.parse_args()
    # The reference arm really spends what it reports (about four seconds per step): fewer steps by default.
    if args.steps is None:
        args.steps = 5 if args.impl == "reference" else 200
    if args.warmup is None:
        args.warmup = 1 if args.impl == "reference" else 10
    return args


def profile_traffic(wl, mode, prefetch_priority=0):
    """DRAM bytes per launch of the layer kernel as ncu counted them (dram__bytes_read.sum +
    dram__bytes_write.sum) in the capture recorded in profiles/ncu_traffic.json: the full batch on
    fewer layers than the bench runs (a full-size launch is too large to capture), scaled by the
    layers a launch spans, to which the traffic is proportional. A figure from that capture, not a
    measurement of this run; None for workloads, pipelines or knobs that were not captured."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if not os.path.exists(path):
        return None, None
    with open(path) as f:
        table = json.load(f)
    key = f"{wl.name}/batch{wl.batch}/pipeline{mode}/prefetch_priority{prefetch_priority}"
    rec = table.get("captures", {}).get(key)
    if not rec:
        return None, None
    return int(rec["dram_bytes_per_layer"] * wl.num_layers), rec


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------------------
# Workload construction (device)
# ---------------------------------------------------------------------------------------------
class DeviceWorkload:
    """Arenas, tables and query tensors of one workload on the current CUDA device."""

    def __init__(self, wl: synth.Workload, seed: int, flags: int = 0, copy_kind: int = 0, copy_ctas: int = 0,
                 decode_ctas: int = 0, pipeline_mode: int = 0, static_split: int = 0, steal_floor: int = 0,
                 prefetch_priority: int = 0, swap_out: int = 0):
        import torch
        from paper_2609_27040_b200 import binding as B
        self.wl, self.B = wl, B
        self.pl = pl = synth.make_placement(wl, seed, slack_blocks=64)
        shape = (2, wl.block_tokens, wl.num_kv_heads, wl.head_dim)
        need = (wl.num_layers * (pl.local_blocks + pl.lent_blocks) + wl.ring_slots * pl.staging_blocks) * wl.block_bytes
        free, _ = torch.cuda.mem_get_info()
        if need > 0.92 * free:
            raise RuntimeError(f"workload needs {need / 2**30:.1f} GiB, device has {free / 2**30:.1f} GiB free")
        gen = torch.Generator(device="cuda").manual_seed(seed)
        bf = torch.bfloat16
        self.local = torch.empty((wl.num_layers, pl.local_blocks) + shape, device="cuda", dtype=bf)
        self.lent = torch.empty((wl.num_layers, pl.lent_blocks) + shape, device="cuda", dtype=bf)
        for l in range(wl.num_layers):          # N(0,1) bf16 KV, layer by layer
            self.local[l].normal_(generator=gen)
            self.lent[l].normal_(generator=gen)
        self.staging = torch.zeros((wl.ring_slots, max(pl.staging_blocks, 1)) + shape, device="cuda", dtype=bf)
        self.q = torch.empty((wl.num_layers, wl.batch, wl.num_q_heads, wl.head_dim), device="cuda", dtype=bf)
        self.q.normal_(generator=gen)
        self.out = torch.zeros_like(self.q)
        self.main = torch.cuda.Stream()
        self.side = torch.cuda.Stream(priority=-1)
        torch.cuda.synchronize()
        self.max_blocks = int(max(len(h) for h in pl.hints)) + 4
        self.s = B.Slice(wl.num_layers, wl.num_kv_heads, pl.local_blocks, pl.lent_blocks, max(pl.staging_blocks, 1),
                         local=self.local, lent=self.lent, staging=self.staging, ring_slots=wl.ring_slots,
                         max_seqs=wl.batch, max_blocks_per_seq=self.max_blocks, flags=flags,
                         local_free_order=pl.local_free_order, lent_free_order=pl.lent_free_order,
                         copy_kind=copy_kind, copy_ctas=copy_ctas, decode_ctas=decode_ctas,
                         pipeline_mode=pipeline_mode, static_split=static_split, steal_floor=steal_floor,
                         prefetch_priority=prefetch_priority, swap_out=swap_out)
        t0 = time.perf_counter()
        for i, hints in enumerate(pl.hints):
            for h in hints:
                rc, _ = self.s.slice_alloc_blocks(i, 1, int(h))
                assert rc == 0, rc
            assert self.s.slice_set_seq_len(i, int(pl.lengths[i])) == 0
        self.alloc_s = time.perf_counter() - t0
        self.seqs = np.arange(wl.batch, dtype=np.int32)
        self.scale = 1.0 / float(np.sqrt(wl.head_dim))
        # algorithmic bytes
        self.tokens = int(pl.lengths.sum())
        self.attn_bytes_layer = (self.tokens * wl.kv_bytes_per_token + 2 * wl.batch * wl.num_q_heads * wl.head_dim * 2
                                 + 4 * pl.total_blocks)
        self.pref_bytes_layer = 2 * pl.staging_blocks * wl.block_bytes + 4 * pl.staging_blocks
        self.step_bytes = wl.num_layers * (self.attn_bytes_layer + self.pref_bytes_layer)

    def step(self, wrap=True, host_io=None):
        if host_io is None:
            rc = self.s.slice_decode_step(self.seqs, self.q, self.wl.num_q_heads, self.scale, self.out, False, wrap,
                                          self.main, self.side)
        else:
            qh, oh = host_io
            rc = self.s.slice_decode_step(self.seqs, qh, self.wl.num_q_heads, self.scale, oh, True, wrap,
                                          self.main, self.side)
        if rc != 0:
            raise RuntimeError(f"slice_decode_step: {self.B.slice_strerror(rc)}")

    def timed(self, steps, wrap=True, host_io=None):
        """K steps between CUDA events on the launching stream; both streams are joined at the end."""
        import torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(self.main)
        for _ in range(steps):
            self.step(wrap, host_io)
        self.main.wait_stream(self.side)
        e1.record(self.main)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / 1e3


class ClockSampler:
    """nvidia-smi samples of SM clock and throttle reasons while the timed regions run."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", uuid], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL,
                                         text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------
def oracle_layer_runner(wl: synth.Workload, seed: int):
    """Host data of ONE layer of the full batch (same placement rule as the device workload) and a
    function that runs the oracle on it once: gather of the lent blocks into a host staging slot, then
    fp64 paged attention of every sequence through the resolved table. Returns (run, tokens, threads)."""
    import oracle
    pl = synth.make_placement(wl, seed, slack_blocks=64)
    sub = list(range(wl.batch))
    n_local = sum(int((pl.hints[i] == synth.LOCAL).sum()) for i in sub)
    n_lent = sum(int((pl.hints[i] == synth.LENT).sum()) for i in sub)
    max_blocks = int(max(len(pl.hints[i]) for i in sub)) + 1
    orc = oracle.OracleSlice(1, wl.block_tokens, wl.block_bytes, n_local, n_lent, n_lent, 1, max(n_lent, 1),
                             max_seqs=len(sub), max_blocks_per_seq=max_blocks)
    for i in sub:
        for h in pl.hints[i]:
            assert orc.alloc_blocks(i, 1, int(h))[0] == 0
        assert orc.set_seq_len(i, int(pl.lengths[i])) == 0
    rng = np.random.default_rng(seed)
    shape = (2, wl.block_tokens, wl.num_kv_heads, wl.head_dim)
    local = synth.normal_bf16_bits(rng, (1, n_local) + shape)
    lent = synth.normal_bf16_bits(rng, (1, max(n_lent, 1)) + shape)
    staging = np.zeros((1, max(n_lent, 1)) + shape, np.uint16)
    q = synth.normal_bf16_bits(rng, (len(sub), wl.num_q_heads, wl.head_dim))
    lens = np.asarray([pl.lengths[i] for i in sub], np.uint32)

    def run():
        rc, resolved, k = orc.gather(0, sub, lent, staging)
        assert rc == 0
        rc, out, _ = oracle.paged_attention(q, local[0], staging[0], resolved, lens, wl.num_q_heads, wl.num_kv_heads,
                                            wl.head_dim, wl.block_tokens, 1.0 / np.sqrt(wl.head_dim), want_lse=False)
        assert rc == 0

    return run, int(lens.sum()), oracle.num_threads()


def oracle_step_seconds(run, layers: int) -> float:
    """One step of the oracle: the whole batch, `layers` times (every layer has the same shape; the
    oracle is run on one layer's host data again and again, so that a step costs 0.6 GB of host
    memory instead of 19 GB). The time is the time spent, nothing is extrapolated."""
    t0 = time.perf_counter()
    for _ in range(layers):
        run()
    return time.perf_counter() - t0


def run_reference(args, wl):
    """The reference arm: there is no reference implementation, so the CPU oracle is timed as it
    stands, on the same workload and metric. Every step runs what it reports."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    run, tokens, threads = oracle_layer_runner(wl, args.seed)
    for _ in range(args.warmup):
        oracle_step_seconds(run, wl.num_layers)
    t = sum(oracle_step_seconds(run, wl.num_layers) for _ in range(args.steps))
    value = wl.batch * args.steps / t
    sample = (f"each step = {wl.num_layers} x (oracle gather + fp64 paged attention of all {wl.batch} sequences, "
              f"{tokens} tokens, on one layer's host data); time as spent, nothing extrapolated")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.batch, "layers": wl.num_layers, "q_heads": wl.num_q_heads,
                   "kv_heads": wl.num_kv_heads, "lent_fraction": wl.lent_fraction, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def parity_check(wl, pl, local, lent, q, outs, scale, seed):
    """Outside every timed region: sampled outputs of the last timed pass against the CPU oracle.
    The oracle replays the placement on its own allocator (so the tables do not come from the CUDA
    library), the blocks of a sampled (layer, sequence) are copied back from the device arenas and
    its dense fp64 attention is compared with what the pass wrote, all query heads, within the stated
    bf16 tolerance. `outs` maps a label to an output tensor [layers][batch][Hq][128]. Raises when a
    sampled output is outside the tolerance: a throughput of wrong results is no result."""
    import oracle
    import torch
    from paper_2609_27040_b200 import binding as B
    oracle.build()
    orc = oracle.OracleSlice(1, wl.block_tokens, wl.block_bytes, pl.local_blocks, pl.lent_blocks, pl.lent_blocks, 1,
                             max(pl.staging_blocks, 1), max_seqs=wl.batch, max_blocks_per_seq=int(max(len(h) for h in pl.hints)) + 4,
                             local_free_order=pl.local_free_order, lent_free_order=pl.lent_free_order)
    for i, hints in enumerate(pl.hints):
        for h in hints:
            assert orc.alloc_blocks(i, 1, int(h))[0] == 0
    L = wl.num_layers
    layers = sorted({0, min(4, L - 1), min(5, L - 1), L // 2, L - 1})
    order = np.argsort(pl.lengths)
    rng = np.random.default_rng(seed)
    seqs = sorted({int(order[0]), int(order[-1])} | {int(x) for x in rng.choice(wl.batch, min(2, wl.batch), replace=False)})
    worst = {k: 0.0 for k in outs}
    worst_rel = {k: 0.0 for k in outs}

    def bits(t):
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)

    for layer in layers:
        for i in seqs:
            n = int(pl.lengths[i])
            tab = orc.block_table(i)[1][: synth.blocks_for(n)]
            blocks = torch.stack([local[layer, e] if e >= 0 else lent[layer, ~e] for e in tab.tolist()])
            blocks = B.kv_block_swizzle(blocks)              # block format -> canonical token rows
            K = blocks[:, 0].reshape(-1, wl.num_kv_heads, wl.head_dim)[:n]
            V = blocks[:, 1].reshape(-1, wl.num_kv_heads, wl.head_dim)[:n]
            rc, ref, _, _ = oracle.dense_attention(bits(q[layer, i]), bits(K), bits(V), wl.num_q_heads, wl.num_kv_heads,
                                                   wl.head_dim, scale)
            assert rc == 0
            for label, out in outs.items():
                got = out[layer, i].double().cpu().numpy()
                err = np.abs(got - ref)
                if not (np.isfinite(got).all() and (err <= 1e-2 + 1e-2 * np.abs(ref)).all()):
                    raise RuntimeError(f"parity check failed: {label}, layer {layer}, sequence {i}, max |err| {err.max():.3e}")
                worst[label] = max(worst[label], float(err.max()))
                big = np.abs(ref) >= 2.0 ** -6
                if big.any():
                    worst_rel[label] = max(worst_rel[label], float((err[big] / np.abs(ref[big])).max()))
    return {"layers": layers, "seqs": seqs, "heads": "all", "checked": sorted(outs), "against": "oracle.dense_attention (fp64)",
            "tolerance": "|err| <= 1e-2 + 1e-2*|ref|", "max_abs_err": max(worst.values()),
            "max_abs_err_by_pass": worst, "max_rel_err": max(worst_rel.values()), "ok": True}


# ---------------------------------------------------------------------------------------------
# Prefetch / migration microbenchmark (gather of randomly indexed 64 KB blocks into a ring, and back)
# ---------------------------------------------------------------------------------------------
def prefetch_microbench(totals=(1_000, 10_000, 100_000, 1_000_000), batches=(1, 8, 64, 512, 4096, 32768),
                        arena_blocks=262_144, max_launches=2048, seed=0, reference_line=True):
    """Gather of N randomly indexed KV blocks (16 tokens x 8 heads x 128 x bf16, K and V: 64 KB) from a
    lent arena into a ring of two staging slots, in launches of b blocks, and the scatter of the same
    blocks back to their ids. The arena holds min(N, arena_blocks) ids; the indices are seeded
    permutations of it (fresh ones concatenated when N is larger). Up to max_launches launches of a
    case are timed (CUDA events on the launching stream; the rate of a launch does not depend on how
    many follow). GB/s counts bytes read plus bytes written. Returns a list of rows."""
    import torch
    from paper_2609_27040_b200 import binding as B
    BB = 65536
    rows = []
    stream = torch.cuda.Stream()
    free, _ = torch.cuda.mem_get_info()
    cap_blocks = int(min(arena_blocks, 0.6 * free // BB))
    bmax = max(batches)
    ring = torch.zeros((2, bmax, BB // 2), dtype=torch.int16, device="cuda")
    arena = None
    for N in totals:
        A = min(N, cap_blocks)
        if arena is None or arena.shape[0] != A:
            del arena
            torch.cuda.empty_cache()
            arena = torch.empty((A, BB // 2), dtype=torch.int16, device="cuda")
            arena.random_(-30000, 30000)
        rng = np.random.default_rng(seed + N)
        idx_h = np.concatenate([rng.permutation(A) for _ in range(-(-N // A))])[:N].astype(np.int32)
        idx = torch.from_numpy(idx_h).cuda()
        for b in batches:
            if b > N:
                continue
            launches = min(N // b, max_launches)
            for direction in ("gather", "scatter"):
                def run(n_launch):          # the launches are issued by the library (one call), not one by one from here
                    rc = B.slice_copy_blocks_series(ring, 2, bmax * BB, arena, idx, n_launch * b, b, BB, direction == "scatter",
                                                    B.COPY_DEFAULT if b < 64 else B.COPY_BULK, 0, stream)
                    assert rc == 0
                run(min(launches, 8))
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                run(launches)
                e1.record(stream)
                e1.synchronize()
                sec = e0.elapsed_time(e1) / 1e3
                moved = 2 * launches * b * BB
                row = {"blocks_total": N, "blocks_per_launch": b, "direction": direction, "launches_timed": launches,
                       "us_per_launch": round(sec / launches * 1e6, 2), "gbs": round(moved / sec / 1e9, 1),
                       "arena_blocks": A, "l2": "arena fits in L2" if A * BB <= 126 << 20 else "larger than L2"}
                if direction == "gather" and b * launches <= 20000:      # byte check of what the last launches left in the ring
                    torch.cuda.synchronize()
                    j = launches - 1
                    row["ring_matches_index_select"] = bool(torch.equal(ring[j & 1][:b], arena.index_select(0, idx[j * b:(j + 1) * b].long())))
                rows.append(row)
        if reference_line and N >= 10_000:
            b = min(4096, N)
            launches = min(N // b, 64)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(stream):
                e0.record(stream)
                for j in range(launches):
                    torch.index_select(arena, 0, idx[j * b:(j + 1) * b], out=ring[j & 1][:b])
                e1.record(stream)
            e1.synchronize()
            sec = e0.elapsed_time(e1) / 1e3
            rows.append({"blocks_total": N, "blocks_per_launch": b, "direction": "gather",
                         "kernel": "torch.index_select (a reference line, not product code)",
                         "gbs": round(2 * launches * b * BB / sec / 1e9, 1)})
    del arena, ring
    torch.cuda.empty_cache()
    return rows


def run_prefetch_microbench(args):
    """`--workload prefetch_microbench`: the whole sweep, one JSON line."""
    import torch
    from paper_2609_27040_b200 import binding as B
    from paper_2609_27040_b200 import build as build_mod
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the path has no CPU fallback")
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    build_mod.build()
    B.lib()
    peak, peak_src = measured_peaks()
    rows = prefetch_microbench(seed=args.seed)
    best = max(r["gbs"] for r in rows if "kernel" not in r)
    line = {"metric": "prefetch_gather_scatter_gbs", "value": best, "unit": "GB/s", "n_gpus": 1, "steps": 1, "warmup": 1,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": "prefetch_microbench", "block_bytes": 65536, "ring_slots": 2,
                       "note": "value = best rate of the sweep; rows = every case"},
            "roofline": {"bound": "hbm", "achieved": best, "peak": peak, "unit": "GB/s", "frac": best / peak,
                         "peak_source": f"of {peak_src}", "traffic": None},
            "rows": rows}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
def reduce_over_ranks(t: float, t_e2e_step: float, launches: int, world: int, device: str):
    """Replicas only: the job's time is the slowest rank's (max over ranks, for the device-resident
    and the end-to-end figure alike), its launch count the sum. No other exchange between ranks."""
    if world <= 1:
        return t, t_e2e_step, launches
    import torch
    import torch.distributed as dist
    tt = torch.tensor([t, t_e2e_step], device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    ll = torch.tensor([launches], device=device, dtype=torch.int64)
    dist.all_reduce(ll)
    return float(tt[0]), float(tt[1]), int(ll[0])


def job_value(batch: int, world: int, steps: int, t: float) -> float:
    """Whole-job tokens/s: every replica decodes `batch` tokens per step; t is the max over ranks."""
    return batch * world * steps / t


def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2609_27040_b200 import binding as B
    from paper_2609_27040_b200 import build as build_mod

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build_mod.build()
    if world > 1:
        dist.barrier()
    B.lib()

    # Replicas only: every rank runs the same workload shape on its own GPU with its own seed.
    kw = dict(copy_kind=args.copy_kind, copy_ctas=args.copy_ctas, decode_ctas=args.decode_ctas,
              static_split=args.static_split, prefetch_priority=args.prefetch_priority)
    w = DeviceWorkload(wl, args.seed + rank, pipeline_mode=args.pipeline_mode, **kw)
    wrap = not args.no_wrap
    for _ in range(max(args.warmup, 3)):
        w.step(wrap)
    torch.cuda.synchronize()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid).replace("GPU-", ""))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: device-resident inputs ----
    st0 = w.s.slice_stats()
    barrier()
    t = w.timed(args.steps, wrap)
    barrier()
    st1 = w.s.slice_stats()
    launches = st1["kernel_launches"] - st0["kernel_launches"]

    # ---- end to end: pinned host q in, out back, every step ----
    qh = w.q.cpu().pin_memory()
    oh = torch.zeros_like(qh).pin_memory()
    for _ in range(3):
        w.step(wrap, (qh, oh))
    barrier()
    e2e_steps = max(3, min(args.steps, 50))
    t_e2e = w.timed(e2e_steps, wrap, (qh, oh))
    barrier()
    io_bytes = qh.numel() * qh.element_size()

    t, t_e2e_step, launches = reduce_over_ranks(t, t_e2e / e2e_steps, launches, world, "cuda")

    # ---- the dominant kernel inside the pipelined pass (profile events + per-CTA trace), rank 0 ----
    roof = None
    parity = None
    extra = {}
    if rank == 0:
        step_bytes, tokens, pl_blocks, k_blocks = w.step_bytes, w.tokens, w.pl.total_blocks, w.pl.staging_blocks
        attn_bytes_layer, pref_bytes_layer = w.attn_bytes_layer, w.pref_bytes_layer
        if not args.no_parity_check:
            # what the last timed pass left in `out` (device-resident run) and in the pinned host
            # buffer (end-to-end run), against the oracle
            parity = parity_check(wl, w.pl, w.local, w.lent, w.q, {"resident": w.out, "e2e_host": oh.view(torch.bfloat16)},
                                  w.scale, args.seed)
        del w
        torch.cuda.empty_cache()
        peak, peak_src = measured_peaks()
        L = wl.num_layers
        reps = max(3, min(args.steps, 20))
        wp = DeviceWorkload(wl, args.seed, flags=B.FLAG_PROFILE, pipeline_mode=args.pipeline_mode, **kw)
        for _ in range(3):
            wp.step(wrap)
        kernel_us, stall_mean, stall_max, launches_per_step = [], [], [], None
        for _ in range(reps):
            k0 = wp.s.slice_stats()["kernel_launches"]
            wp.step(wrap)
            tm = wp.s.slice_layer_times().astype(np.float64)         # synchronises
            launches_per_step = wp.s.slice_stats()["kernel_launches"] - k0
            if args.pipeline_mode in (0, 3):
                kernel_us.append(float(tm[L - 1, 3] - tm[0, 2]))     # one launch (or one chain) spans the pass
            else:
                kernel_us.append(float(np.nansum(tm[:, 4] - tm[:, 2])))
        del wp
        torch.cuda.empty_cache()
        # per-CTA device-timer trace in a pass of its own (the trace costs a few per cent)
        wp = DeviceWorkload(wl, args.seed, flags=B.FLAG_TRACE, pipeline_mode=args.pipeline_mode, **kw)
        for _ in range(3):
            wp.step(wrap)
        for _ in range(max(3, reps // 2)):
            wp.step(wrap)
            tr = wp.s.slice_cta_trace(0).astype(np.float64)
            wait_us = tr[:, :, 1] / 1e3                               # [layer][cta] ns the attention waited
            stall_mean.append(wait_us[1:].mean())
            stall_max.append(wait_us[1:].max(axis=1).mean())
        kernel_s = float(np.mean(kernel_us)) * 1e-6
        algo = step_bytes if args.pipeline_mode != 1 else L * attn_bytes_layer
        achieved = algo / kernel_s / 1e9
        combined = step_bytes * args.steps / t / 1e9
        name = {0: "slice_layer_kernel (one launch per pass: attention + gather of every layer)",
                1: "slice_layer_kernel (attention only; gather in copy_blocks_bulk<6> on a second stream, sharing the SMs)",
                2: "slice_layer_kernel (one launch per layer: attention + gather of the next layer)",
                3: "slice_layer_kernel (a chain of launches, one per layer, each starting while the one before it runs)"
                }[args.pipeline_mode]
        traffic, traffic_rec = profile_traffic(wl, args.pipeline_mode, args.prefetch_priority)
        roof = {"bound": "hbm", "kernel": name, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic,
                # DRAM bytes (ncu, scaled by layers) over this run's launch time: what HBM actually moved
                "achieved_dram": traffic / kernel_s / 1e9 if traffic else None,
                "frac_dram": traffic / kernel_s / 1e9 / peak if traffic else None,
                "frac_dram_of_nominal_8TBs": traffic / kernel_s / 1e9 / NOMINAL_HBM_GBS if traffic else None,
                "traffic_source": ({"file": "profiles/ncu_traffic.json", **{k: traffic_rec[k] for k in
                                    ("layers_captured", "dram_bytes_per_layer", "l2_hit_rate_pct", "dram_over_algorithmic")
                                    if k in traffic_rec}} if traffic_rec else None),
                "peak_source": f"of {peak_src}", "launches_per_step": launches_per_step,
                "launch_us": kernel_s * 1e6 / max(launches_per_step, 1) if args.pipeline_mode != 1 else None,
                "algorithmic_bytes_per_launch": algo // max(launches_per_step, 1) if args.pipeline_mode != 1 else attn_bytes_layer,
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "combined_over_step_time": {"achieved": combined, "frac": combined / peak,
                                            "frac_of_nominal_8TBs": combined / NOMINAL_HBM_GBS}}
        attn_layer_us = kernel_s * 1e6 / L
        extra = {"layer_us": attn_layer_us, "stall_us_per_layer": float(np.mean(stall_mean)),
                 "stall_us_per_layer_worst_cta": float(np.mean(stall_max)),
                 "stall_frac_of_layer": float(np.mean(stall_mean)) / attn_layer_us,
                 "stall_definition": "time a CTA's attention waits for the layer's prefetched blocks (device timer), "
                                     "mean over CTAs and layers; worst_cta = mean over layers of the slowest CTA. "
                                     "Attention and prefetch share ONE HBM here (the paper's prefetch crosses a link from "
                                     "another GPU's memory): while a CTA's attention waits, its copy thread and the other "
                                     "CTAs keep HBM at the rate the roofline object reports, so the wait is slack of the "
                                     "faster stream, not time lost by the step.",
                 "alloc_seconds_setup": wp.alloc_s}
        del wp
        torch.cuda.empty_cache()
        if not args.no_ablations:
            # Other pipelines on the same workload: one fused launch per layer; the same launches as a
            # chain in which each starts while the one before it runs; two kernels on two
            # streams; and the on-demand variant (gather and attention serialised on one stream), whose
            # profile events also give each kernel's duration with nothing running beside it.
            abl = {}
            for label, mode in (("fused_launch_per_layer", 2), ("chained_launch_per_layer", 3), ("two_streams", 1)):
                if mode == args.pipeline_mode:
                    continue
                wa = DeviceWorkload(wl, args.seed, pipeline_mode=mode, **kw)
                for _ in range(3):
                    wa.step(wrap)
                ta = wa.timed(reps, wrap)
                abl[label] = {"tokens_per_s": wl.batch * reps / ta, "ms_per_step": ta / reps * 1e3,
                              "hbm_gbs_combined": step_bytes * reps / ta / 1e9}
                del wa
                torch.cuda.empty_cache()
            # Swap-out beside swap-in (Section 2.3): the ring as a write-back cache, every staged layer written
            # back to the lent arena by the copy threads of the same launch while it is attended to.
            for label, swap in ((("swap_out_write_back", 1), ("swap_out_tail_blocks_only", 2)) if args.pipeline_mode == 0 else ()):
                wa = DeviceWorkload(wl, args.seed, pipeline_mode=0, swap_out=swap, **kw)
                for _ in range(3):
                    wa.step(wrap)
                ta = wa.timed(reps, wrap)
                swap_bytes = step_bytes + L * (wa.pref_bytes_layer if swap == 1 else 2 * wl.batch * wl.block_bytes)
                abl[label] = {"tokens_per_s": wl.batch * reps / ta, "ms_per_step": ta / reps * 1e3,
                              "hbm_gbs_combined": swap_bytes * reps / ta / 1e9,
                              "note": ("swap_out = 1: attention + gather + write-back of every staged layer (algorithmic "
                                       "bytes: attention + 4 x the lent bytes), one launch per pass" if swap == 1 else
                                       "swap_out = 2: the write-back takes only the staged tail blocks, the ones an append "
                                       "can have changed (at most one block per sequence and layer), one launch per pass")}
                del wa
                torch.cuda.empty_cache()
            # Two kernels on two streams with events, the pipeline the paper's description maps to most
            # directly: its event-defined stall, max(0, end of prefetch(l) - end of attention(l-1)).
            wt = DeviceWorkload(wl, args.seed, flags=B.FLAG_PROFILE, pipeline_mode=1, **kw)
            for _ in range(3):
                wt.step(wrap)
            ev_stall = []
            for _ in range(3):
                wt.step(wrap)
                tm = wt.s.slice_layer_times().astype(np.float64)
                ev_stall.append(np.nanmean(np.clip(tm[1:, 1] - tm[:-1, 4], 0.0, None)))
            abl.setdefault("two_streams", {})["event_stall_us_per_layer"] = float(np.mean(ev_stall))
            abl["two_streams"]["event_stall_definition"] = "max(0, end of prefetch(l) - end of attention(l-1)) from CUDA events"
            del wt
            torch.cuda.empty_cache()
            # Ways to keep attention from waiting for prefetched blocks, each at a price in tokens/s:
            # lock step (idle CTAs steal down to the last block of every layer, so all CTAs change
            # layers together), prefetch priority (the copy threads keep 4 instead of 3 loads in
            # flight and win the bandwidth they need), and both.
            if args.pipeline_mode == 0:
                for label, opts in (("lock_step_stealing", {"steal_floor": 1}), ("prefetch_priority", {"prefetch_priority": 1}),
                                    ("prefetch_priority_lock_step", {"steal_floor": 1, "prefetch_priority": 1})):
                    wa = DeviceWorkload(wl, args.seed, flags=B.FLAG_TRACE, pipeline_mode=0, **{**kw, **opts})
                    for _ in range(3):
                        wa.step(wrap)
                    ta = wa.timed(reps, wrap)
                    wa.step(wrap)
                    tr = wa.s.slice_cta_trace(0).astype(np.float64)
                    abl[label] = {"tokens_per_s": wl.batch * reps / ta, "ms_per_step": ta / reps * 1e3,
                                  "hbm_gbs_combined": step_bytes * reps / ta / 1e9,
                                  "stall_us_per_layer": float((tr[1:, :, 1] / 1e3).mean()),
                                  "note": "traced run (a few per cent slower than an untraced one)"}
                    del wa
                    torch.cuda.empty_cache()
            # The same one-launch pass as a decoder can drive it: the queries of layer l+1 are released
            # only when the output of layer l is complete (here they ARE that output, aliased in
            # memory: q = X[l], out = X[l+1]); the caller's stream only waits and releases, through
            # stream-ordered memory operations, so no kernel has to fit beside the persistent one.
            # A second form leaves 8 SMs free and has a kernel of the caller (an elementwise negation)
            # compute q[l+1] from out[l] on them.
            for label, alias, prio in ((("layer_dependent_q", True, args.prefetch_priority),
                                        ("layer_dependent_q_caller_kernel", False, args.prefetch_priority))
                                       if args.pipeline_mode == 0 else ()):
                kwa = {**kw, "prefetch_priority": prio}
                if not alias:
                    kwa["decode_ctas"] = max(1, torch.cuda.get_device_properties(0).multi_processor_count - 8)
                try:
                    wa = DeviceWorkload(wl, args.seed, flags=B.FLAG_TRACE, pipeline_mode=0, **kwa)
                    X = torch.zeros((L + 1,) + tuple(wa.q.shape[1:]), device="cuda", dtype=torch.bfloat16)
                    X[0].copy_(wa.q[0])
                    caller = torch.cuda.Stream()
                    if not alias:
                        torch.neg(wa.out[0], out=wa.q[1])        # loads the kernel's code before any pass runs
                    torch.cuda.synchronize()

                    def dependent_step():
                        rc = wa.s.slice_step_begin(wa.seqs, X[:L] if alias else wa.q, wl.num_q_heads, wa.scale,
                                                   X[1:] if alias else wa.out, wrap, wa.main)
                        if rc != 0:
                            raise RuntimeError(f"slice_step_begin: {B.slice_strerror(rc)}")
                        assert wa.s.slice_step_submit_q(0, caller) == 0
                        for l in range(L - 1):
                            assert wa.s.slice_step_wait_out(l, caller) == 0
                            if not alias:
                                with torch.cuda.stream(caller):
                                    torch.neg(wa.out[l], out=wa.q[l + 1])
                            assert wa.s.slice_step_submit_q(l + 1, caller) == 0

                    for _ in range(3):
                        dependent_step()
                    torch.cuda.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(wa.main)
                    for _ in range(reps):
                        dependent_step()
                    e1.record(wa.main)
                    torch.cuda.synchronize()
                    ta = e0.elapsed_time(e1) / 1e3
                    if wa.s.slice_stats()["device_status"] != 0:
                        raise RuntimeError("layer-dependent pass: a bounded device wait expired")
                    tr = wa.s.slice_cta_trace(0).astype(np.float64)
                    abl[label] = {
                        "tokens_per_s": wl.batch * reps / ta, "ms_per_step": ta / reps * 1e3,
                        "hbm_gbs_combined": step_bytes * reps / ta / 1e9,
                        "stall_us_per_layer": float((tr[1:, :wa.s.cfg.decode_ctas or None, 1] / 1e3).mean()),
                        "decode_ctas": int(wa.s.cfg.decode_ctas) or "one per SM", "prefetch_priority": prio,
                        "note": "slice_step_begin: every layer's attention waits for its queries, which are released only "
                                "after the previous layer's output is complete (" +
                                ("q[l+1] = out[l], aliased in memory: the caller's stream only waits and releases"
                                 if alias else "q[l+1] = -out[l], computed by a kernel of the caller on the 8 SMs left free"
                                               ) + "); traced run"}
                    del wa, X
                    torch.cuda.empty_cache()
                except RuntimeError as err:      # an ablation must not cost the bench line
                    abl[label] = {"error": str(err)}
                    torch.cuda.synchronize()
                    torch.cuda.empty_cache()
            # Performance transparency (Sections 2.3, 4): a layer's lent data comes in during the latency
            # window before the layer is used. A decoder leaves such a window by itself: between out[l]
            # and q[l+1] lie the projections and the MLP of the block. Here a spinning kernel of the
            # caller stands for them (window_us per layer, on an SM the pass leaves free), and the time
            # from a layer's queries to its output is compared with the same batch with nothing lent.
            if args.pipeline_mode == 0 and wl.lent_fraction > 0:
                try:
                    import dataclasses
                    windows_us = (0.0, 50.0, 100.0, 150.0)
                    props = torch.cuda.get_device_properties(0)
                    sms = props.multi_processor_count
                    cycles_per_us = getattr(props, "clock_rate", 1965000) * 1e-3                 # SM cycles
                    res = {}
                    for name, wlx in (("lent", wl), ("all_local", dataclasses.replace(wl, lent_fraction=0.0))):
                        wa = DeviceWorkload(wlx, args.seed, flags=B.FLAG_TRACE, pipeline_mode=0, **{**kw, "decode_ctas": sms - 1})
                        X = torch.zeros((L + 1,) + tuple(wa.q.shape[1:]), device="cuda", dtype=torch.bfloat16)
                        X[0].copy_(wa.q[0])
                        caller = torch.cuda.Stream()
                        with torch.cuda.stream(caller):
                            torch.cuda._sleep(1000)                 # loads the spinning kernel before any pass runs
                        torch.cuda.synchronize()

                        def windowed_step(spin):
                            rc = wa.s.slice_step_begin(wa.seqs, X[:L], wl.num_q_heads, wa.scale, X[1:], wrap, wa.main)
                            if rc != 0:
                                raise RuntimeError(f"slice_step_begin: {B.slice_strerror(rc)}")
                            assert wa.s.slice_step_submit_q(0, caller) == 0
                            for l in range(L - 1):
                                assert wa.s.slice_step_wait_out(l, caller) == 0
                                if spin:
                                    with torch.cuda.stream(caller):
                                        torch.cuda._sleep(spin)
                                assert wa.s.slice_step_submit_q(l + 1, caller) == 0

                        for w_us in windows_us:
                            spin = int(w_us * cycles_per_us)
                            for _ in range(2):
                                windowed_step(spin)
                            torch.cuda.synchronize()
                            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                            n_w = max(3, reps // 2)
                            e0.record(wa.main)
                            for _ in range(n_w):
                                windowed_step(spin)
                            e1.record(wa.main)
                            torch.cuda.synchronize()
                            if wa.s.slice_stats()["device_status"] != 0:
                                raise RuntimeError("windowed layer-dependent pass: a bounded device wait expired")
                            tr = wa.s.slice_cta_trace(0).astype(np.float64)[:, :sms - 1]
                            seen = np.where(tr[:, :, 7] > 0, tr[:, :, 7], np.inf).min(axis=1)  # first CTA to have the layer's q
                            done = tr[:, :, 5].max(axis=1)                                       # last CTA to finish its last run
                            res[(name, w_us)] = {"ms_per_step": e0.elapsed_time(e1) / n_w,
                                                 "q_to_last_block_us_per_layer": float(np.mean((done - seen)[1:-1]) / 1e3),
                                                 "stall_us_per_layer": float((tr[1:, :, 1] / 1e3).mean())}
                        del wa, X
                        torch.cuda.empty_cache()
                    abl["transparency_with_a_window"] = {
                        "decode_ctas": sms - 1, "lent_fraction": wl.lent_fraction,
                        "windows": [{"window_us_per_layer": w_us, "lent": res[("lent", w_us)], "all_local": res[("all_local", w_us)],
                                     "layer_time_ratio_lent_over_all_local":
                                         res[("lent", w_us)]["q_to_last_block_us_per_layer"] / res[("all_local", w_us)]["q_to_last_block_us_per_layer"],
                                     "step_time_ratio_lent_over_all_local":
                                         res[("lent", w_us)]["ms_per_step"] / res[("all_local", w_us)]["ms_per_step"]} for w_us in windows_us],
                        "note": "slice_step_begin with a spinning kernel of the caller between out[l] and q[l+1] (the rest of a "
                                "decoder block); q_to_last_block = from the first CTA seeing a layer's queries to the last CTA "
                                "finishing its last run of the layer (device timer, mean over the inner layers); a ratio of 1 "
                                "means the lent part of the KV cost the layer nothing: the prefetch fitted in the window"}
                except RuntimeError as err:
                    abl["transparency_with_a_window"] = {"error": str(err)}
                    torch.cuda.synchronize()
                    torch.cuda.empty_cache()
            ws = DeviceWorkload(wl, args.seed, flags=B.FLAG_PROFILE, pipeline_mode=1, **kw)
            for _ in range(2):
                assert ws.s.slice_decode_step(ws.seqs, ws.q, wl.num_q_heads, ws.scale, ws.out, False, wrap, ws.main, ws.main) == 0
            iso_attn, iso_pref = [], []
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t_serial = 0.0
            for _ in range(max(3, reps // 2)):
                e0.record(ws.main)
                assert ws.s.slice_decode_step(ws.seqs, ws.q, wl.num_q_heads, ws.scale, ws.out, False, wrap, ws.main, ws.main) == 0
                e1.record(ws.main)
                tm = ws.s.slice_layer_times().astype(np.float64)
                t_serial += e0.elapsed_time(e1) / 1e3
                iso_attn.append(tm[:, 4] - tm[:, 2])
                iso_pref.append(tm[:, 1] - tm[:, 0])
            n_ser = max(3, reps // 2)
            iso_us, iso_pref_us = float(np.nanmean(np.stack(iso_attn))), float(np.nanmean(np.stack(iso_pref)))
            abl["serialised_prefetch"] = {"tokens_per_s": wl.batch * n_ser / t_serial, "ms_per_step": t_serial / n_ser * 1e3,
                                          "note": "on-demand variant: prefetch not overlapped with attention"}
            extra["ablations"] = abl
            alts = {k: v for k, v in abl.items() if "stall_us_per_layer" in v}
            if alts:
                # The 70 % gate is about what HBM moves: algorithmic bytes times the DRAM-to-algorithmic
                # ratio of the ncu capture of the same configuration (L2 serves part of the staged
                # blocks), where one was captured; the algorithmic figure is kept beside it.
                def dram_ratio(prio):
                    rec = profile_traffic(wl, 0, prio)[1]
                    return rec.get("dram_over_algorithmic") if rec else None

                def frac(v):
                    return v["stall_us_per_layer"] / (v["ms_per_step"] * 1e3 / L)

                def hbm(gbs, prio):
                    r = dram_ratio(prio)
                    return {"algorithmic_bytes": gbs / NOMINAL_HBM_GBS,
                            "dram_bytes": gbs * r / NOMINAL_HBM_GBS if r else None,
                            "dram_bytes_source": "ncu capture, profiles/ncu_traffic.json" if r else "unmeasured"}

                def gate(gbs, prio):
                    h = hbm(gbs, prio)
                    return (h["dram_bytes"] if h["dram_bytes"] is not None else h["algorithmic_bytes"]) >= 0.70

                prio_of = {"lock_step_stealing": 0, "prefetch_priority": 1, "prefetch_priority_lock_step": 1,
                           "layer_dependent_q": -1, "layer_dependent_q_caller_kernel": -1}  # DRAM traffic of these: not captured
                ok = [k for k, v in alts.items() if frac(v) < 0.05 and gate(v["hbm_gbs_combined"], prio_of.get(k, 0))]
                pick = max(ok, key=lambda k: alts[k]["tokens_per_s"]) if ok else min(alts, key=lambda k: frac(alts[k]))
                default_stall = extra["stall_frac_of_layer"]
                # every configuration that meets both targets, with its tokens/s (the two-stream pipeline by
                # its event-defined stall and the algorithmic rate: its DRAM traffic was not captured)
                all_ok = {k: round(alts[k]["tokens_per_s"], 1) for k in ok}
                ts = abl.get("two_streams", {})
                if "event_stall_us_per_layer" in ts and ts["event_stall_us_per_layer"] / (ts["ms_per_step"] * 1e3 / L) < 0.05 \
                        and ts["hbm_gbs_combined"] / NOMINAL_HBM_GBS >= 0.70:
                    all_ok["two_streams"] = round(ts["tokens_per_s"], 1)
                extra["targets"] = {
                    "all_configurations_meeting_both": all_ok,
                    "hbm_frac_of_nominal_8TBs": {"target": 0.70, "default_pipeline": hbm(combined, args.prefetch_priority),
                                                 pick: hbm(alts[pick]["hbm_gbs_combined"], prio_of.get(pick, 0))},
                    "stall_frac_of_layer": {"target": 0.05, "default_pipeline": default_stall, pick: frac(alts[pick])},
                    "default_pipeline_meets": {"hbm": gate(combined, args.prefetch_priority), "stall": default_stall < 0.05},
                    "both_met_by": pick if ok else None,
                    "default_tokens_per_s": wl.batch * args.steps / t, "both_met_tokens_per_s": alts[pick]["tokens_per_s"] if ok else None,
                    "note": "the default pipeline maximises tokens/s and misses the stall target: attention and prefetch "
                            "share one HBM, attention takes its share first and then waits while the copy threads use "
                            "the rest; the named configuration meets both targets at the lower tokens/s stated"}
            # The prefetch / migration microbenchmark in short (the whole sweep: --workload prefetch_microbench).
            if not args.no_microbench:
                extra["prefetch_microbench"] = prefetch_microbench(totals=(100_000,), batches=(1, 8, 64, 512, 4096, 32768),
                                                                   arena_blocks=100_000, max_launches=512, seed=args.seed)
            extra["kernels_alone"] = {
                "attention_only_layer_kernel": {"us_per_launch": iso_us, "algorithmic_bytes": attn_bytes_layer,
                                                "achieved_gbs": attn_bytes_layer / (iso_us * 1e-6) / 1e9,
                                                "frac": attn_bytes_layer / (iso_us * 1e-6) / 1e9 / peak,
                                                "note": "one launch per layer, prefetch serialised before it"},
                "copy_blocks_bulk_gather": {"us_per_launch": iso_pref_us, "kernel": "copy_blocks_bulk<6> (6 x 16 KB ring per CTA, one CTA per SM)", "algorithmic_bytes": pref_bytes_layer,
                                              "achieved_gbs": pref_bytes_layer / (iso_pref_us * 1e-6) / 1e9,
                                              "frac": pref_bytes_layer / (iso_pref_us * 1e-6) / 1e9 / peak}}
            del ws
            torch.cuda.empty_cache()
    clocks = sampler.stop()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        import oracle
        oracle.build()
        run, sample_tokens, threads = oracle_layer_runner(wl, args.seed)
        run()                                                   # page the data in
        step_s = min(oracle_step_seconds(run, wl.num_layers) for _ in range(2))
        cpu = {"value": wl.batch / step_s, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"one whole step, best of 2: {wl.num_layers} x (oracle gather + fp64 paged attention of all "
                         f"{wl.batch} sequences, {sample_tokens} tokens, on one layer's host data); {step_s:.2f} s per step"}

    value = job_value(wl.batch, world, args.steps, t)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": t / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.batch, "layers": wl.num_layers, "q_heads": wl.num_q_heads,
                   "kv_heads": wl.num_kv_heads, "head_dim": wl.head_dim, "block_tokens": wl.block_tokens,
                   "len_range": [wl.len_lo, wl.len_hi], "lent_fraction": wl.lent_fraction, "ring_slots": wl.ring_slots,
                   "tokens_in_batch": tokens, "blocks": pl_blocks, "lent_blocks": k_blocks,
                   "parallelism": "replicas" if world > 1 else "single", "pipeline_mode": args.pipeline_mode,
                   "l2": "inputs larger than L2: every step streams %.1f GB of KV" % (step_bytes / 1e9)},
        "hbm_gbs_combined": step_bytes * world * args.steps / t / 1e9,
        "roofline": roof, "cpu_baseline": cpu, "parity_checked": parity,
        "e2e": {"value": wl.batch * world / t_e2e_step, "unit": UNIT, "h2d_bytes_per_step": io_bytes,
                "d2h_bytes_per_step": io_bytes, "ms_per_step": t_e2e_step * 1e3},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    line.update(extra)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.workload == "prefetch_microbench":
        run_prefetch_microbench(args)
        return
    wl = synth.WORKLOADS[args.workload]
    if args.layers or args.batch or args.kv_heads:
        import dataclasses
        hkv = args.kv_heads or wl.num_kv_heads
        wl = dataclasses.replace(wl, num_layers=args.layers or wl.num_layers, batch=args.batch or wl.batch, num_kv_heads=hkv,
                                 num_q_heads=wl.num_q_heads // wl.num_kv_heads * hkv)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
