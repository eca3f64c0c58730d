"""The multi-GPU form of the bench is N independent replicas; the only exchange between ranks is the
reduction of their timings. Checked here with two gloo ranks on the CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    dist.barrier()
    # rank 1 is the slower replica in the device-resident figure, rank 0 in the end-to-end one
    t = [2.0, 3.0][rank]
    e2e = [0.9, 0.5][rank]
    out = bench.reduce_over_ranks(t, e2e, 10 + rank, world, "cpu")
    dist.barrier()
    if rank == 0:
        print(json.dumps({"t": out[0], "e2e": out[1], "launches": out[2],
                          "value": bench.job_value(64, world, 30, out[0])}))
    dist.destroy_process_group()
""") % ROOT


def test_two_rank_reduction_takes_the_slowest_rank_and_sums_launches():
    import json
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-400:] for o in outs]
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["t"] == 3.0 and line["e2e"] == 0.9 and line["launches"] == 21
    assert line["value"] == 64 * 2 * 30 / 3.0           # whole-job tokens/s over the slowest rank's time
    assert outs[1][0].strip() == ""                      # only rank 0 prints


def test_single_rank_passes_values_through():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(1.5, 0.25, 7, 1, "cpu") == (1.5, 0.25, 7)
    assert bench.job_value(64, 1, 10, 2.0) == 320.0
