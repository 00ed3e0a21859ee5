"""The multi-GPU path of the benchmark is replicas only: ranks decode disjoint sequences and the
report is reduced over the ranks.  Covered here with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # per-rank figures: rank r took (10 + r) ms, emitted 100 * (r + 1) tokens with 7 launches
    maxed, summed = bench.reduce_over_ranks([10.0 + rank, 2.0 - rank], [100.0 * (rank + 1), 7.0], "cpu")
    out.put((rank, maxed, summed, bench.rank_sequences(rank, 4)))
    dist.barrier()
    dist.destroy_process_group()


def test_report_is_reduced_over_two_gloo_ranks_and_sequences_are_disjoint():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, maxed, summed, seqs in res:
        assert maxed == [11.0, 2.0]                 # slowest rank decides the time
        assert summed == [300.0, 14.0]              # tokens and launches add up
    assert res[0][3] == [0, 1, 2, 3] and res[1][3] == [4, 5, 6, 7]


def test_single_process_passes_through():
    import bench
    assert bench.reduce_over_ranks([1.5], [2.0, 3.0], "cpu") == ([1.5], [2.0, 3.0])


def test_gpus_flag_must_agree_with_the_launcher():
    """Started by a launcher (RANK set) with a world size that differs from --gpus, the benchmark
    stops with a message instead of silently timing one replica."""
    import subprocess
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"], env=env,
                       capture_output=True, text=True, timeout=120)
    assert r.returncode != 0 and "--gpus 2 but WORLD_SIZE is 1" in r.stderr
