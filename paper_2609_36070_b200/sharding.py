"""Host-side logic of the multi-GPU path: token-sharded replicas.

Every token's output depends only on its own row of x (paper, Section 2.1 equation), so N GPUs that each hold all
weights and their own batch need no data-path exchange; the only communication is a barrier and the max over ranks
of the step time.  This module holds that logic so that it can be tested with `gloo` ranks on CPU.
"""
from dataclasses import replace

from . import inputs


def rank_config(cfg: inputs.MoEConfig, rank: int) -> inputs.MoEConfig:
    """The workload of one rank: same shapes and weights, its own token stream (seed offset)."""
    return cfg if rank == 0 else replace(cfg, seed=cfg.seed + 1000 * rank)


def rank_tokens(cfg: inputs.MoEConfig, rank: int):
    """x[T,H] (bf16 bits) of one rank."""
    return inputs.make_x(rank_config(cfg, rank))


def shard_rows(total_rows: int, world: int, rank: int):
    """Contiguous token range [begin, end) of `rank` when one batch of total_rows is split over `world` ranks."""
    base, rem = divmod(total_rows, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Step time of the job = the slowest rank's (paper, Section 4.1: latency of the slowest rank)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput with a fixed batch per GPU (weak scaling)."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)
