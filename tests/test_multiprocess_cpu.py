"""The N > 1 path of the benchmark is N independent replicas (the method has no exchange step), joined only by
barriers and by the reduction of the per-rank figures.  These tests run that host logic with two gloo ranks
on the CPU: the slowest rank sets every time, the bytes add up, and the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        times, nbytes = bench.aggregate_over_ranks([1.0 + rank, 5.0 - rank, 0.25 * (rank + 1)], 1000.0 * (rank + 1),
                                                   dist, torch.device("cpu"))
        out.put((rank, times, nbytes))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reduce_to_the_slowest_time_and_the_summed_bytes():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 500
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, times, nbytes in got:
        assert times == [2.0, 5.0, 0.5]          # max over the two ranks of each entry
        assert nbytes == 3000.0                  # 1000 + 2000


def test_single_process_reduction_is_the_identity():
    import torch
    sys.path.insert(0, ROOT)
    import bench
    times, nbytes = bench.aggregate_over_ranks([3.0, 4.0], 7.0, None, torch.device("cpu"))
    assert times == [3.0, 4.0] and nbytes == 7.0


@pytest.mark.parametrize("rank,expect_line", [(0, True), (1, False)])
def test_reference_arm_prints_on_rank_zero_only(rank, expect_line):
    """Under torchrun every rank starts `bench.py --impl reference`; only rank 0 times the oracle and prints."""
    env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank))
    proc = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                           "--steps", "1", "--warmup", "3", "--workload", "cfg1"],
                          env=env, capture_output=True, text=True, timeout=600)
    assert proc.returncode == 0, proc.stderr[-2000:]
    lines = [l for l in proc.stdout.splitlines() if l.startswith("{")]
    if not expect_line:
        assert lines == []
        return
    line = json.loads(lines[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["value"] > 0 and line["n_gpus"] == 2
