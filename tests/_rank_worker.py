"""Worker of the two-rank CPU test: the host-side logic bench.py runs on every rank of a multi-GPU
(replicas only) run, on the gloo backend.  Launched by torch.distributed.run."""
import json
import os
import sys
from dataclasses import replace

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from vvs_synth.configs import CONFIGS  # noqa: E402


def main() -> None:
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    wl = CONFIGS[1]
    seed = bench.replica_seed(wl.seed, rank)
    trial = bench.host_trial(replace(wl, seed=seed), 0)
    fills = torch.tensor(trial["cache_len"][:1].astype(np.int64))
    all_fills = [torch.zeros_like(fills) for _ in range(world)]
    dist.all_gather(all_fills, fills)
    dist.barrier()
    # the slowest rank decides the time of the whole job
    ms_total, ms_e2e = bench.max_over_ranks([10.0 + rank, 20.0 - rank], world)
    drafts = float(trial["n_draft"].sum())
    # repeated timed regions: the rank-dependent region times must make every rank stop after the same
    # region (the stop rule sees only all-reduced times), or the barriers deadlock
    calls = []

    def region(steps):
        calls.append(steps)
        return 40.0 + 30.0 * rank + len(calls)      # rank 1 is slower: 71, 72, ...

    regions = bench.timed_regions(region, 4, world, dist.barrier, min_ms=500.0, device="cpu")
    if rank == 0:
        out = {"fills": [int(f[0]) for f in all_fills], "ms_total": ms_total, "ms_e2e": ms_e2e,
               "value": bench.aggregate_value(world, drafts, 4, ms_total), "drafts": drafts, "world": world,
               "regions": regions, "region_calls": calls}
        with open(os.environ["VVS_RANK_TEST_OUT"], "w") as f:
            json.dump(out, f)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
