"""One rank of the two-process test of the replica logic (gloo, CPU); rank 0 prints one JSON line."""
import json
import os
import sys

import numpy as np
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2507_23777_b200 import inputs, replicas  # noqa: E402


def main():
    world, rank, local = replicas.env_ranks()
    dist.init_process_group("gloo")
    assert dist.get_world_size() == world and dist.get_rank() == rank
    cfg = inputs.config(0)
    seed = replicas.replica_seed(cfg["seed"], rank, world)
    cond = inputs.make_cond(dict(cfg, seed=seed), 1)
    # every rank decodes its own mesh: rank r commits 100 + r tokens in 10 (r + 1) ms
    job = replicas.reduce_totals(tokens=100 + rank, meshes=1, ms=10.0 * (rank + 1), ms_e2e=20.0 * (rank + 1))
    digest = float(np.abs(cond).sum())
    all_digests = [None] * world
    dist.all_gather_object(all_digests, (seed, digest))
    dist.barrier()
    if rank == 0:
        print(json.dumps({"world": job.world, "tokens": job.tokens, "meshes": job.meshes, "ms": job.ms,
                          "ms_e2e": job.ms_e2e, "value": job.tokens_per_s_per_mesh(), "ranks": all_digests}))
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
