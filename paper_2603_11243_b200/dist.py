"""Multi-process plumbing: one process per GPU, utterances sharded across ranks.

Utterances are independent units of the decision path (every output is per utterance or per
frame), so the path shards by utterance with no exchange step: each rank runs the whole path on
its own batch, and only the timing (maximum over ranks) and the processed-unit count (sum over
ranks) are combined, with two small all-reduces outside the data path.
"""
import os
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def env_rank() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment (1-process defaults)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    """Joins the process group when a launcher started this process (RANK and WORLD_SIZE in the
    environment, a world of one included, so that a single GPU exercises the same calls); a plain
    `python bench.py` stays without one.  With NCCL the rank's GPU is selected first and named
    to the group, so that no collective has to guess the device."""
    rank, local_rank, world = env_rank()
    launched = "RANK" in os.environ and "WORLD_SIZE" in os.environ
    if launched and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
            dist.init_process_group(backend=backend, rank=rank, world_size=world,
                                    device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def finalize() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()


def rank_seed(seed: int, rank: int) -> int:
    """Seed of the batch a rank generates: rank 0 keeps the workload's own seed."""
    return seed + 100003 * rank


def partition_by_bytes(costs: Sequence[int], world: int) -> List[Tuple[int, int]]:
    """Contiguous ranges [lo, hi) of utterances, one per rank, balanced by a per-utterance cost
    (bytes of logits): range r ends at the first utterance where the running cost reaches
    (r+1)/world of the total.  Used when one given batch is split (strong scaling)."""
    total = sum(costs)
    out, lo, acc, b = [], 0, 0, 0
    for r in range(world):
        target = total * (r + 1) / world
        while b < len(costs) and (acc + costs[b] <= target or r == world - 1):
            acc += costs[b]
            b += 1
        out.append((lo, b))
        lo = b
    return out


def reduce_max_sum(local_max: float, local_sum: float, device) -> Tuple[float, float]:
    """Maximum of `local_max` and sum of `local_sum` over all ranks."""
    if not dist.is_initialized():
        return local_max, local_sum
    m = torch.tensor([local_max], dtype=torch.float64, device=device)
    s = torch.tensor([local_sum], dtype=torch.float64, device=device)
    dist.all_reduce(m, op=dist.ReduceOp.MAX)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return float(m.item()), float(s.item())


def all_gather_rows(local: torch.Tensor) -> torch.Tensor:
    """[R, ...] stack of every rank's `local` tensor (same shape on all ranks), rank-major: the one
    exchange of vocabulary-parallel verification (each rank's [M, 3] partial statistics, 12 bytes
    per row).  Without a process group the result is the local tensor with a leading 1."""
    if not dist.is_initialized():
        return local.unsqueeze(0).contiguous()
    parts = [torch.empty_like(local) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, local.contiguous())
    return torch.stack(parts).contiguous()


def vocab_shard(V_total: int, rank: int, world: int, multiple: int = 8) -> Tuple[int, int]:
    """(col0, V_local) of rank's slice when V_total columns are split as evenly as possible in
    units of `multiple` columns (the last rank takes the remainder)."""
    units = (V_total + multiple - 1) // multiple
    lo = (units * rank // world) * multiple
    hi = V_total if rank == world - 1 else (units * (rank + 1) // world) * multiple
    return lo, max(0, min(hi, V_total) - lo)

