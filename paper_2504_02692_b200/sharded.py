"""One layer on several GPUs: token-sharded statistics, row-sharded quantization.

The solve shards naturally with ONE exchange step.  Tokens are independent in the statistics
(Algorithm 1, the statistics step: H and dXX^T are sums over tokens), so every rank accumulates its share of the
token batches into its own state; one all-reduce (sum, float32, 2 n^2 elements) gives every rank the
full sums.  The factor and P depend only on the sums and are recomputed on every rank (cheaper than
broadcasting two n x n matrices and free of a second exchange).  Rows of W are independent in the
loop (Section 4, Step 1), so every rank quantizes a slab of rows; nothing further is exchanged —
the caller gathers codes and grids if it wants them in one place.

Everything here is plumbing around the C ABI: index arithmetic and one ``torch.distributed``
all-reduce on views of the caller-owned state buffer (NCCL on GPUs; the host-side logic is
covered by gloo tests on CPU tensors).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def token_shard(n_batches: int, rank: int, world: int) -> range:
    """Contiguous, balanced share of the token batches for ``rank`` (earlier ranks take the extras)."""
    base, extra = divmod(n_batches, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def row_shard(m: int, rank: int, world: int, multiple: int = 32) -> tuple[int, int]:
    """Rows ``[r0, r1)`` of W for ``rank``: balanced in units of ``multiple`` rows (the quantize kernels
    take 32 rows per warp group), the last rank takes the ragged tail."""
    units = (m + multiple - 1) // multiple
    base, extra = divmod(units, world)
    u0 = rank * base + min(rank, extra)
    u1 = u0 + base + (1 if rank < extra else 0)
    return min(u0 * multiple, m), min(u1 * multiple, m)


def allreduce_sums(H: torch.Tensor, D: torch.Tensor, tokens: int, group=None) -> int:
    """Sums the per-rank partial statistics in place on every rank; returns the total token count.
    ``H`` / ``D``: the n x n float32 sums (any device that the process group's backend serves)."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return int(tokens)
    dist.all_reduce(H, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(D, op=dist.ReduceOp.SUM, group=group)
    t = torch.tensor([tokens], dtype=torch.int64, device=H.device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return int(t.item())


def allreduce_statistics(state, group=None) -> int:
    """The exchange step for a ``LayerState`` after this rank's gptaq_accumulate calls: orders the
    stream after the pending products, all-reduces H and dXX^T in the state buffer and sets the total
    token count on the handle (so that gptaq_factor normalises by it).  Returns the total.
    ``state`` needs ``H()``, ``D()`` (views of the sums, current on the stream the collective runs on),
    ``tokens()`` and ``set_tokens(total)``."""
    H, D = state.H(), state.D()          # views; H() / D() flush the handle's internal stream first
    total = allreduce_sums(H, D, state.tokens(), group)
    state.set_tokens(total)
    return total
