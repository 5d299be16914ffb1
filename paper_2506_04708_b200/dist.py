"""Multi-GPU plumbing of the benchmark: independent replicas, one process per GPU.

The step shards by sequence and its only coupling is the shared N-gram table, so several GPUs run
independent replicas (each rank its own sequences and its own table) with no collective on the data path.
What is shared is the measurement: every rank times the same number of steps, the slowest rank's time
counts, and rank 0 reports the units of all ranks over that time.
"""
import os


def env_ranks():
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) when run directly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(seed: int, rank: int) -> int:
    """Every replica draws its own streams, logits and uniforms."""
    return seed + 7919 * rank


def init(backend: str, device=None):
    """Joins the process group (rendezvous from MASTER_ADDR / MASTER_PORT); returns torch.distributed or None."""
    rank, world, _ = env_ranks()
    if world == 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kw)
    return dist


def barrier(dist):
    if dist is not None:
        dist.barrier()


def max_over_ranks(dist, value: float, device="cpu") -> float:
    """The slowest rank's figure (a time), known to every rank."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step: int, world: int, steps: int, max_ms_total: float) -> float:
    """Units processed by all ranks per second, over the slowest rank's time."""
    return units_per_rank_per_step * world * steps / (max_ms_total * 1e-3)
