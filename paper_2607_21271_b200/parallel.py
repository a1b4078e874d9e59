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


def dp_training_step(fwd, weight_grad, data_grad, flat, group=None, side_stream=None, mark=None):
    """One data-parallel training step of the layer, in the order that hides its one exchange step.

    forward -> weight gradient -> START the all-reduce of the flat dw|db buffer -> data gradient -> wait for the
    collective.  The weight gradient goes first because it is the only result other ranks need; its sum over ranks then
    travels while the data gradient (which needs no exchange) is computed, and the step ends only once the summed
    gradients are in place.  `fwd`, `weight_grad` and `data_grad` are callables that enqueue (GPU) or run (CPU) the
    three passes.  On CUDA, pass `side_stream`: the collective is issued there behind an event recorded after the
    weight gradient, so that it overlaps the data-gradient kernel, and the current stream waits for it at the end.
    `mark(i)`, if given, is called at the phase boundaries (0: start, 1: after fwd, 2: after the weight gradient and the
    start of the exchange, 3: after the data gradient) so that a caller can record timing events.
    Returns the list of phase names in the order they ran."""
    import torch

    order = []
    if mark:
        mark(0)
    fwd()
    order.append("fwd")
    if mark:
        mark(1)
    weight_grad()
    order.append("bwd_weight")
    work = None
    if side_stream is not None:
        ready = torch.cuda.Event()
        ready.record()
        with torch.cuda.stream(side_stream):
            side_stream.wait_event(ready)
            work = allreduce_weight_grads(None, None, group=group, flat=flat, async_op=True)
    else:
        work = allreduce_weight_grads(None, None, group=group, flat=flat, async_op=True)
    order.append("allreduce_start")
    if mark:
        mark(2)
    data_grad()
    order.append("bwd_data")
    if mark:
        mark(3)
    if work is not None:
        work.wait()                     # CUDA: the current stream waits for the collective; CPU: blocks until it is done
    order.append("allreduce_done")
    return order
