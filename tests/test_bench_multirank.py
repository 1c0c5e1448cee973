"""The N>1 path of bench.py on CPU: two gloo ranks take the max of their device times and
rank 0 aggregates whole-job throughput (replicas: no data-path collective)."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(2.0 + rank, world)  # rank 1 is slower
    out[rank] = (ms, bench.aggregate_tokens_per_s(16384, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_max_and_aggregate():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29511 + os.getpid() % 200, out), nprocs=world, join=True)
        assert out[0] == out[1]
        ms, tok = out[0]
        assert ms == 3.0 and abs(tok - 2 * 16384 / 3e-3) < 1e-6


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25, 1) == 1.25
    assert bench.dist_env()[1] >= 1
    ab = bench.algorithmic_bytes(bench.get_workload("c4"))
    assert ab["fwd"] == 4 * 4 * 16 * 4096 * 64 * 2 and ab["bwd"] == 7 * 4 * 16 * 4096 * 64 * 2
