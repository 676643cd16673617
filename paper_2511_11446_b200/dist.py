"""Multi-GPU plumbing. The quantized-linear path shards by rows (tokens are independent: DAQ is per
token and the GEMM is row-wise), so ranks run independent batches with replicated weights and there
is NO collective on the data path; torch.distributed is used only for the timing barrier and the
max-over-ranks reduction of the measured time."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init(backend: str | None = None):
    """Initialises the process group when launched by torchrun (WORLD_SIZE > 1). Returns
    (rank, local_rank, world_size)."""
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"),
                                rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def shard_rows(M: int, rank: int, world: int, multiple: int = 1):
    """Contiguous row range [lo, hi) of rank `rank` when M rows are split over `world` ranks in
    units of `multiple` rows; the ranges partition [0, M)."""
    units = (M + multiple - 1) // multiple
    base, rem = divmod(units, world)
    lo_u = rank * base + min(rank, rem)
    hi_u = lo_u + base + (1 if rank < rem else 0)
    return min(M, lo_u * multiple), min(M, hi_u * multiple)


def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own batch: a distinct stream of the counter-based generator."""
    return (base_seed + 0x1000 * rank) & 0xFFFFFFFF
