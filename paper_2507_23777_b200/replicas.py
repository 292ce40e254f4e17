"""Host logic of a multi-GPU run: N independent replicas of the decoding loop, one process per GPU.

Meshes are independent problems (Algorithm 1 has no step that exchanges data between sequences), so a
job on N GPUs is N replicas, each with meshes of its own; the only communication is the reduction of the
timings and token counts for the report.  Everything here works on any ``torch.distributed`` backend:
NCCL with CUDA tensors in a GPU run, gloo with CPU tensors in the tests.
"""
from __future__ import annotations

import os
from dataclasses import dataclass


def env_ranks():
    """(world, rank, local_rank) as the launcher exported them; (1, 0, 0) for a plain run."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(seed: int, rank: int, world: int) -> int:
    """Seed of the meshes (conditions, Philox key) of one replica: replicas of one job never share meshes,
    a single-GPU run keeps the configured seed.  The model weights keep the configured seed on every rank."""
    return seed + 1000 * rank if world > 1 else seed


@dataclass
class JobTotals:
    tokens: int          # committed tokens, all ranks
    meshes: int          # meshes decoded, all ranks
    ms: float            # slowest rank's device time of the timed region
    ms_e2e: float        # slowest rank's time of the end-to-end region
    world: int

    def tokens_per_s_per_mesh(self) -> float:
        """Whole-job rate divided by the meshes one replica decodes at a time: the per-mesh rate when one GPU
        decodes one mesh, times N (weak scaling)."""
        return self.tokens / (self.ms / 1e3) / (self.meshes / self.world)


def reduce_totals(tokens: int, meshes: int, ms: float, ms_e2e: float, device="cpu") -> JobTotals:
    """Sum of the counts and maximum of the times over the ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return JobTotals(int(tokens), int(meshes), float(ms), float(ms_e2e), 1)
    s = torch.tensor([tokens, meshes], dtype=torch.int64, device=device)
    t = torch.tensor([ms, ms_e2e], dtype=torch.float64, device=device)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return JobTotals(int(s[0]), int(s[1]), float(t[0]), float(t[1]), dist.get_world_size())
