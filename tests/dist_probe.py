"""Run under torchrun on CPU (gloo): exercises the rendezvous, barrier and max-over-ranks code of
bench.py that the multi-GPU replicas path uses."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

import bench  # noqa: E402

world, rank, local = bench.dist_setup(int(os.environ["WORLD_SIZE"]))
assert world == int(os.environ["WORLD_SIZE"]) and rank == int(os.environ["RANK"])
bench.barrier(world)
got = bench.max_over_ranks(10.0 + rank, world, torch.device("cpu"))
assert got == 10.0 + world - 1, got
bench.barrier(world)
if rank == 0:
    print(f"probe ok world={world}")
import torch.distributed as dist  # noqa: E402
dist.destroy_process_group()
