"""The N>1 path of the benchmark on CPU: two gloo ranks, each with its own batch shard and its
own timing; the reported time is the maximum over ranks and the rate the whole job's.  There is
no collective on the data path (images are independent), so this reduction is all there is."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 2.0 + 3.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, device="cpu")
    # every rank draws its own shard: different seeds, same shapes
    from paper_1805_12549_b200 import synth
    x = synth.smoothed_noise((("bench", "c64@32", rank), "x"), 2, 8, 8, 16)
    out[rank] = (ms, bench.whole_job_rate(256, world, ms), float(x.sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_rank_and_the_whole_job():
    world, port = 2, 29531 + os.getpid() % 200
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 5.0
    assert abs(res[0][1] - 2 * 256 / 5.0e-3) < 1e-6
    assert res[0][2] != res[1][2]                    # the shards differ


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25, device="cpu") == 1.25
    assert bench.whole_job_rate(64, 1, 2.0) == 32000.0
