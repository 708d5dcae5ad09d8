"""Host-side logic for running N independent replicas of a boundary, one process per GPU.

The codec has no exchange step between samples (Algorithm 1 works on one sample at a time),
so data parallelism only splits the id space: every rank owns its own shard of sample ids
with its own copy pair of m, and no tensor crosses ranks.  What the ranks do share is the
clock: a run is as slow as its slowest rank.
"""
from dataclasses import replace


def shard_for_rank(cfg, rank: int, world: int):
    """The boundary that `rank` of `world` owns: same shapes and quantizer, its own id shard.

    Shard r covers global sample ids [r * n_samples, (r + 1) * n_samples); inside the rank the
    ids are local (0 .. n_samples - 1) and the input recipe is keyed by the shard (stream = r),
    so two ranks never see the same activations."""
    if not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside world of {world}")
    return replace(cfg, stream=cfg.stream + rank)


def global_sample_id(cfg, rank: int, local_id: int) -> int:
    return rank * cfg.n_samples + local_id


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The largest `value` over all ranks (every rank gets it); identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, slowest_ms: float) -> float:
    """Units per second of the whole job: every rank did units_per_rank in slowest_ms."""
    return world * units_per_rank / (slowest_ms * 1e-3)
