"""Worker of tests/test_dist_gloo.py: two CPU processes exercise the benchmark's multi-process host logic."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import torch
import torch.distributed as dist

import bench

rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
bench.init_dist()
assert dist.get_backend() == "gloo" and dist.get_world_size() == world == 2
dist.barrier()
# the job's time is the slowest rank's
assert bench.max_over_ranks(10.0 + rank, world) == 11.0
# every rank decodes a different sequence, reproducibly
mine = bench.rank_prompt(1024, 32, rank)
both = [torch.zeros(32, dtype=torch.int32) for _ in range(world)]
dist.all_gather(both, mine)
assert not torch.equal(both[0], both[1])
assert torch.equal(both[rank], bench.rank_prompt(1024, 32, rank))
dist.barrier()
dist.destroy_process_group()
open(os.path.join(sys.argv[1], f"ok.{rank}"), "w").write("ok")
