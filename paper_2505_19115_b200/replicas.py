"""Host-side plumbing of the multi-process benchmark: the path does not shard (one GPU per rank, every
rank runs its own replica of the workload), so the only things ranks share are a barrier around the
timed region, the maximum of their times, and distinct input seeds.  No data-path collective."""
import os

import torch


def env_rank_world():
    """(rank, world_size, local_rank) from the launcher's environment (1 process when absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(base: int, rank: int) -> int:
    """Input seed of a rank's replica: distinct per rank, reproducible."""
    return base + 100 * rank


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The slowest rank's time: what a job that waits for all replicas experiences."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, world: int, seconds: float) -> float:
    """Whole-job throughput of `world` replicas that each processed units_per_rank in `seconds` (the max over ranks)."""
    return units_per_rank * world / seconds
