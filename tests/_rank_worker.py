"""Worker of test_multirank_cpu.py: one of the ranks of a torchrun launch with the gloo backend (no GPU)."""
import json
import os
import sys

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2512_07090_b200 import workloads as W  # noqa: E402

rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
wl = W.WORKLOADS["c2"]
seed = bench.rank_seed(wl.seed, rank)
wl.seed = seed
ids = wl.make_ids(batch=1, seq=64)
slow = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")
dist.barrier()
json.dump({"rank": rank, "world": world, "seed": seed, "ids": ids[0, :16].tolist(), "max_ms": slow},
          open(os.path.join(sys.argv[1], f"rank{rank}.json"), "w"))
dist.destroy_process_group()
