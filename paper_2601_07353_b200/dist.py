"""Host-side plumbing for running the path on several GPUs of one node.

Sequences are independent in every step of the path (expansion, tree, attention, acceptance are
all per sequence), so more GPUs means more replicas: each rank owns its own sequences and its own
KV cache and there is no exchange on the data path.  What is left for ``torch.distributed`` is the
rendezvous, a barrier on each side of the timed region, and the max-over-ranks of the measured
time.  Everything here works with the ``gloo`` backend on CPU tensors as well, which is how it is
tested without GPUs.
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import List

import torch
import torch.distributed as td


@dataclass
class RankInfo:
    rank: int
    world: int
    local_rank: int

    @property
    def is_main(self) -> bool:
        return self.rank == 0


def env_rank_info() -> RankInfo:
    """Rank, world size and local rank as torchrun exports them (1 process if unset)."""
    return RankInfo(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
                    int(os.environ.get("LOCAL_RANK", "0")))


def init(info: RankInfo, backend: str) -> None:
    """Joins the process group when there is more than one rank (MASTER_ADDR/PORT from the env)."""
    if info.world > 1 and not td.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29517")
        td.init_process_group(backend=backend, rank=info.rank, world_size=info.world)


def shutdown() -> None:
    if td.is_initialized():
        td.destroy_process_group()


def barrier(info: RankInfo) -> None:
    if info.world > 1:
        td.barrier()


def max_over_ranks(value: float, info: RankInfo, device="cpu") -> float:
    """The slowest rank's figure: what a multi-GPU time has to be reported as."""
    if info.world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    td.all_reduce(t, op=td.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, info: RankInfo, device="cpu") -> float:
    if info.world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    td.all_reduce(t, op=td.ReduceOp.SUM)
    return float(t.item())


def rank_sequence_ids(info: RankInfo, sets: int, batch: int) -> List[List[int]]:
    """Sequence ids of this rank's input sets: ``sets`` lists of ``batch`` ids.

    Ranks and sets never share a sequence id, so every replica works on its own trees; set s of
    rank r holds ids ``(r * sets + s) * batch .. + batch - 1``.
    """
    base = info.rank * sets
    return [list(range((base + s) * batch, (base + s + 1) * batch)) for s in range(sets)]


def whole_job_rate(units_per_rank: float, seconds_max: float, info: RankInfo) -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling)."""
    return units_per_rank * info.world / seconds_max
