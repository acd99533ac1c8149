"""Host-side logic for running N independent replicas of the router, one process per GPU.

The capacity constraint couples every token of a batch (the column sums of P run over all tokens, Eq. 7),
so one routing problem does not shard: under data parallelism each rank routes its own batch with its own
capacity C = ceil(cf * T * k / E) (Sec. 2.3) and no data crosses ranks.  What the ranks share is only the
measurement: a barrier around the timed region and the maximum of the per-rank times.
"""
from __future__ import annotations

import os
from dataclasses import dataclass


@dataclass(frozen=True)
class RankInfo:
    rank: int
    local_rank: int
    world: int


def rank_info(env=None) -> RankInfo:
    """Rank, local rank and world size as the launcher exports them (absent = a single process)."""
    env = os.environ if env is None else env
    world = int(env.get("WORLD_SIZE", "1"))
    rank = int(env.get("RANK", "0"))
    local = int(env.get("LOCAL_RANK", str(rank)))
    if world < 1 or not (0 <= rank < world) or local < 0:
        raise ValueError(f"inconsistent launcher environment: RANK={rank} LOCAL_RANK={local} WORLD_SIZE={world}")
    return RankInfo(rank, local, world)


def replica_seed(info: RankInfo, base_seed: int = 0) -> int:
    """Every replica routes a different synthetic batch."""
    return base_seed + info.rank


def init_group(info: RankInfo, backend: str, **kw):
    """Join the process group (rendezvous through MASTER_ADDR / MASTER_PORT); no-op for one process."""
    if info.world == 1:
        return False
    import torch.distributed as dist
    dist.init_process_group(backend, rank=info.rank, world_size=info.world, **kw)
    return True


def barrier(info: RankInfo):
    if info.world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(info: RankInfo, value: float, device="cpu") -> float:
    """The slowest rank's time: what a job of N replicas takes."""
    if info.world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(info: RankInfo, tokens_per_rank_per_step: int, ms_per_step_max: float) -> float:
    """Whole-job throughput: every rank routed its own batch in the time the slowest one needed."""
    return info.world * tokens_per_rank_per_step / (ms_per_step_max * 1e-3)


def shutdown(info: RankInfo):
    if info.world > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()
