"""Data-parallel sharding of units (sequence x layer pairs) over ranks.

Units are independent, so the retention pass shards with no data-path collective: every rank runs
the whole pass on its own units.  The only communication is the benchmark's timing reduction --
except in the prompt-global mode (Alg. 1 (A): one window mass per prompt, averaged over all its
layers), where a prompt's layers may sit on several ranks and their partial sums must be added.
"""
from __future__ import annotations


def shard_units(n_units: int, rank: int, world: int) -> range:
    """Contiguous, balanced slice of ``range(n_units)`` owned by ``rank`` (sizes differ by at most one)."""
    if not 0 <= rank < world:
        raise ValueError("rank out of range")
    base, extra = divmod(n_units, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def max_over_ranks(value: float, group=None) -> float:
    """MAX all-reduce of a host scalar (elapsed time) over the process group; identity without one."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def allreduce_prompt_mass(pmass, group=None):
    """SUM all-reduce, in place, of the per-prompt window mass [prompts, L] over the ranks that hold the
    prompts' layers (the method's one exchange step: between ckv_prompt_mass and ckv_global_scores).
    Every rank must hold the same prompts in the same order.  Identity without a process group."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(pmass, op=dist.ReduceOp.SUM, group=group)
    return pmass
