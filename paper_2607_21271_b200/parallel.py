"""Data-parallel plumbing of the EQ-Linear path: token sharding and the one exchange step.

The forward pass and the data gradient are independent per token, so tokens are split over ranks and the
spectral weight is replicated.  The weight and bias gradients are sums over tokens, so their per-rank
partial results are summed over ranks (one all-reduce of T*C_out*C_in + C_out floats).  torch.distributed is
plumbing only; the arithmetic of the layer stays in the CUDA library.
"""

from __future__ import annotations


def shard_tokens(N: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous, balanced token range [begin, end) of `rank` out of `world` (sizes differ by at most 1)."""
    if world < 1 or not 0 <= rank < world or N < 0:
        raise ValueError("bad shard arguments")
    base, extra = divmod(N, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def grad_buffers(Co: int, Ci: int, T: int, device):
    """One contiguous float32 buffer holding dw [Co, Ci, T] followed by db [Co], and views of both: the exchange step is
    then a single all-reduce (at ~1 MB it is bound by launch latency, so one call instead of two matters)."""
    import torch

    n = Co * Ci * T
    pad = (-n) % 4                                   # keeps db 16-byte aligned, as the library requires
    flat = torch.zeros(n + pad + Co, dtype=torch.float32, device=device)
    return flat, flat[:n].view(Co, Ci, T), flat[n + pad:n + pad + Co]


def allreduce_weight_grads(dw, db=None, group=None, flat=None, async_op=False):
    """Sum dw (and db) over the ranks of `group`, in place.  No-op without an initialised process group.
    With `flat` (the buffer of grad_buffers that dw and db are views of) one all-reduce covers both; with
    `async_op` (flat form only) the collective's work handle is returned instead of being waited for."""
    import torch.distributed as dist

    if not dist.is_available() or not dist.is_initialized():
        return None
    if flat is not None:
        if dist.get_world_size(group) == 1 and not async_op:
            return None
        return dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group, async_op=async_op) if async_op else \
            dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    if dist.get_world_size(group) == 1:
        return None
    dist.all_reduce(dw, op=dist.ReduceOp.SUM, group=group)
    if db is not None:
        dist.all_reduce(db, op=dist.ReduceOp.SUM, group=group)
    return None
