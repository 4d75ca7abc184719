"""Multi-GPU plumbing of the benchmark: one process per GPU, launched by
torch.distributed.run.  Sequences are independent (every equation of the
verification rule is per sequence and per round), so ranks shard the batch and
exchange no data; the only collectives are the barrier around the timed region
and the MAX reduction of the elapsed time."""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch


@dataclass
class Ranks:
    rank: int
    world: int
    local_rank: int
    backend: str          # "" when world == 1 (no process group)

    @property
    def is_main(self) -> bool:
        return self.rank == 0


def init_from_env(backend: str = "nccl") -> Ranks:
    """Reads RANK / WORLD_SIZE / LOCAL_RANK (set by torch.distributed.run) and
    creates the process group when there is more than one rank."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world == 1:
        return Ranks(0, 1, local, "")
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    import torch.distributed as dist
    if not dist.is_initialized():
        kw = {}
        if backend == "nccl":
            torch.cuda.set_device(local)
            kw["device_id"] = torch.device("cuda", local)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return Ranks(rank, world, local, backend)


def barrier(r: Ranks) -> None:
    if r.world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(r: Ranks, value: float) -> float:
    """Largest `value` over all ranks (the job's elapsed time is the slowest rank's)."""
    if r.world == 1:
        return float(value)
    import torch.distributed as dist
    dev = torch.device("cuda", r.local_rank) if r.backend == "nccl" else torch.device("cpu")
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(r: Ranks, value: float) -> float:
    if r.world == 1:
        return float(value)
    import torch.distributed as dist
    dev = torch.device("cuda", r.local_rank) if r.backend == "nccl" else torch.device("cpu")
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def shard_sequences(total_B: int, r: Ranks) -> range:
    """Contiguous block of the global batch that this rank verifies."""
    per, extra = divmod(total_B, r.world)
    lo = r.rank * per + min(r.rank, extra)
    return range(lo, lo + per + (1 if r.rank < extra else 0))


def shard_vocab(V: int, r: Ranks, align: int = 8):
    """(offset, width) of this rank's slice of the vocabulary; slice starts are multiples of `align`
    tokens so that every slice keeps 16-byte structure."""
    per = -(-V // r.world)
    per = -(-per // align) * align
    lo = min(V, r.rank * per)
    return lo, min(V, lo + per) - lo


def all_gather_partials(r: Ranks, partial: torch.Tensor) -> torch.Tensor:
    """All-gathers the per-row partial states of a vocabulary-parallel step: [rows, 4] on every rank ->
    [world, rows, 4] on every rank (16 bytes per row and rank: latency-bound, one NCCL call)."""
    if r.world == 1:
        return partial.unsqueeze(0)
    import torch.distributed as dist
    out = torch.empty((r.world,) + tuple(partial.shape), dtype=partial.dtype, device=partial.device)
    dist.all_gather(list(out.unbind(0)), partial.contiguous())   # one slot of `out` per rank, in rank order
    return out


def finalize(r: Ranks) -> None:
    if r.world > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()
