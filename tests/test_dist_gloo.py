"""The multi-rank host logic of the benchmark on two gloo ranks (CPU): sharding by whole windows,
per-rank batches, max-over-ranks timing and the whole-job throughput."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2603_25463_b200 import dist as cd, synth
    wl = synth.WORKLOADS["llamagen384"]
    mine = cd.rank_workload(wl, rank)
    assert mine.rows == wl.rows and mine.seed != cd.rank_workload(wl, 1 - rank).seed
    b, e = cd.shard_rows(1000 * 16 + 16, 16, rank, world)  # 1001 windows over 2 ranks
    ms = 2.0 if rank == 0 else 3.5
    slow = cd.max_over_ranks(ms, world)
    tput = cd.job_throughput(e - b, 10, ms, world)
    with open(os.path.join(out_dir, "r%d.txt" % rank), "w") as f:
        f.write("%d %d %.6f %.6f\n" % (b, e, slow, tput))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks(tmp_path):
    world, port = 2, 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [open(tmp_path / ("r%d.txt" % i)).read().split() for i in range(world)]
    b0, e0, b1, e1 = int(r[0][0]), int(r[0][1]), int(r[1][0]), int(r[1][1])
    assert b0 == 0 and e0 == b1 and e1 == 1001 * 16  # contiguous, complete
    assert e0 % 16 == 0 and (e0 - b0) // 16 == 501 and (e1 - b1) // 16 == 500  # whole windows, balanced
    for i in range(world):
        assert float(r[i][2]) == 3.5  # the slowest rank's time, on every rank
        assert abs(float(r[i][3]) - 1001 * 16 * 10 / 3.5e-3) < 1e-3 * 1001 * 16 * 10 / 3.5e-3


def test_shard_rows_edge_cases():
    sys.path.insert(0, ROOT)
    from paper_2603_25463_b200 import dist as cd
    assert cd.shard_rows(0, 8, 0, 4) == (0, 0)
    spans = [cd.shard_rows(3 * 8, 8, r, 4) for r in range(4)]  # fewer windows than ranks
    assert spans == [(0, 8), (8, 16), (16, 24), (24, 24)]
