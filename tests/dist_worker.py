"""Worker for the world_size-2 gloo test: each rank reports a different elapsed time; every rank must see the
maximum, draw a different batch, and compute the same whole-job rate."""
import json
import sys

import torch.distributed as dist

from paper_1910_06188_b200 import dist_util, synth

if __name__ == "__main__":
    world, rank, local = dist_util.env_world()
    dist.init_process_group("gloo")
    ms = 2.0 + 3.0 * rank                      # rank 1 is slower
    slowest = dist_util.max_over_ranks(ms)
    cfg = dist_util.rank_config(4, rank)
    x = synth.activation(4, 8, synth.seed_for(cfg, 0))
    rate = dist_util.whole_job_rate(1000.0, world, slowest)
    gathered = [None] * world
    dist.all_gather_object(gathered, dict(rank=rank, slowest=slowest, rate=rate, first=float(x[0, 0]), cfg=cfg))
    if rank == 0:
        print(json.dumps(gathered))
    dist.destroy_process_group()
    sys.exit(0)
