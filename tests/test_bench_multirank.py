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


def test_roofline_counts_the_methods_bytes_only():
    """The roofline object divides the method's bytes (4 tensors forward, 7 backward, each once)
    by the summed kernel time -- not the bytes the implementation chooses to re-read -- and
    reports the whole-call fractions and the captured DRAM traffic next to it."""
    sys.path.insert(0, ROOT)
    import bench
    w = bench.get_workload("c4")
    peaks = {"hbm_gbs": 6550.7, "bf16_tflops": 1646.4, "source": "measured"}
    tensor = 4 * 16 * 4096 * 64 * 2
    r = bench.roofline_record(w, peaks, kernels_ms=0.1452, kernel="k", fwd_ms=0.050, bwd_ms=0.100, step_ms=0.150)
    assert r["algorithmic_bytes"] == 11 * tensor
    assert r["algorithmic_bytes_per_token_head"] == {"fwd": 8 * 64, "bwd": 14 * 64}
    assert abs(r["frac"] - 11 * tensor / 0.1452e-3 / 1e9 / 6550.7) < 1e-12
    assert abs(r["frac_of_nominal_8TBs"] - 11 * tensor / 0.1452e-3 / 1e9 / 8000.0) < 1e-12
    assert abs(r["calls"]["fwd"]["frac"] - 4 * tensor / 0.050e-3 / 1e9 / 6550.7) < 1e-12
    assert abs(r["calls"]["bwd"]["frac"] - 7 * tensor / 0.100e-3 / 1e9 / 6550.7) < 1e-12
    assert abs(r["calls"]["step"]["frac"] - 11 * tensor / 0.150e-3 / 1e9 / 6550.7) < 1e-12
    assert r["bound"] == "hbm" and r["peak"] == 6550.7 and r["peak_source"] == "measured"
    # DRAM traffic from the committed capture: above the method's bytes (re-reads), below 1.5x
    assert 1.0 < r["traffic_over_algorithmic"] < 1.5 and "not measured in this run" in r["traffic_source"]
    # a forward-only workload counts four tensors and has no backward entry
    r2 = bench.roofline_record(bench.get_workload("c2"), peaks, 0.03, "k", 0.034, None, 0.034)
    assert r2["algorithmic_bytes"] == 4 * 32 * 12 * 512 * 64 * 2 and "bwd" not in r2["calls"]
