"""World-size-2 gloo test of the multi-GPU bookkeeping of bench.py: the path has
no exchange step, so ranks are independent replicas; the job time is the max
over ranks and the job throughput the sum of the ranks' tokens over that time."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 5.0 + 3.0 * rank          # rank 1 is the slow one
    value, ms = bench.replica_throughput(1000, ms_local)
    mx = bench.max_over_ranks(float(rank))
    # replicas draw different seeds: same structure, different logits
    from paper_2605_17862_b200 import synth
    wl = synth.tiny(scale=1 / 16)
    wl.seed += 100 * rank
    ch = synth.gen_chunk(wl, 0)
    sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(sums, ch["student"].double().sum().reshape(1))
    out[rank] = (value, ms, mx, float(sums[0]), float(sums[1]))
    dist.destroy_process_group()


def test_replica_bookkeeping_world_size_2():
    world, port = 2, 29500 + os.getpid() % 1000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        value, ms, mx, s0, s1 = res[rank]
        assert ms == 8.0 and mx == 1.0
        assert abs(value - 2 * 1000 / 8e-3) < 1e-6
        assert s0 != s1
    assert res[0][3:] == res[1][3:]


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5) == 3.5
    value, ms = bench.replica_throughput(100, 2.0)
    assert ms == 2.0 and abs(value - 100 / 2e-3) < 1e-9
