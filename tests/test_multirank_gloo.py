"""The N > 1 path of the benchmark is N independent replicas: no data-path collective, only the
whole-job aggregation (max of the ranks' times, sum of their tokens).  Covered here with two gloo
ranks on the CPU."""
import os
import sys
import tempfile

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank: int, world: int, init_file: str, out_dir: str):
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"file://{init_file}", rank=rank, world_size=world)
    try:
        # rank r "ran" for 10 + 5 r ms and processed 1000 (r + 1) tokens
        ms, tokens = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1))
        with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
            f.write(f"{ms} {tokens}")
    finally:
        dist.destroy_process_group()


def test_replica_aggregation_two_gloo_ranks():
    world = 2
    with tempfile.TemporaryDirectory() as td:
        init_file = os.path.join(td, "rendezvous")
        mp.spawn(_rank_main, args=(world, init_file, td), nprocs=world, join=True)
        for r in range(world):
            ms, tokens = map(float, open(os.path.join(td, f"r{r}.txt")).read().split())
            assert ms == 15.0            # the slowest rank's time
            assert tokens == 3000.0      # all ranks' tokens


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(12.5, 77.0) == (12.5, 77.0)
