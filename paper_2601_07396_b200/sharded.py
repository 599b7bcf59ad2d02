"""Row-sharded calibration (Eq. 4 over several GPUs): every rank accumulates the Gram matrix of
its own rows of the stack, the ranks sum the D x D partial sums with one all-reduce, and every
rank runs the same eigen-solve on the total -- so all ranks end with the same basis, bit for bit.
The step kernels need none of this: blocks and rows are independent there.

Plumbing only (``torch.distributed`` for the exchange); the arithmetic is the library's.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch

from . import binding as sc


def shard_rows(M: int, rank: int, world: int) -> Tuple[int, int]:
    """Rows [lo, hi) of an M-row stack that rank ``rank`` of ``world`` owns: contiguous, disjoint,
    covering, sizes differing by at most one."""
    if not (0 <= rank < world) or M < 0:
        raise ValueError("need 0 <= rank < world and M >= 0")
    base, extra = divmod(M, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def gram_view(workspace: torch.Tensor, D: int) -> torch.Tensor:
    """The D x D fp64 Gram matrix inside a calibration workspace, as a tensor sharing its memory."""
    off, nbytes = sc.svdcache_calibrate_gram_region(D)
    return workspace[off:off + nbytes].view(torch.float64).view(D, D)


def allreduce_gram(G: torch.Tensor, group=None) -> torch.Tensor:
    """Sum of the ranks' partial Gram matrices, in place (NCCL for device tensors, gloo for host
    ones).  Without an initialised process group, or with one rank, G is the total already."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(G, op=dist.ReduceOp.SUM, group=group)
    return G


def calibrate_sharded(stack_shard: torch.Tensor, k: int, workspace: Optional[torch.Tensor] = None, group=None,
                      strict: bool = True):
    """Calibration of a stack whose rows are spread over the ranks of ``group``; ``stack_shard`` holds
    this rank's rows (device, M_local x D; M_local may be 0).  Returns (Vk, lambda, trace, info), the
    same on every rank."""
    M, D = stack_shard.shape
    if workspace is None:
        workspace = torch.empty(sc.svdcache_calibrate_workspace_bytes(D, k), dtype=torch.uint8, device=stack_shard.device)
    sc.svdcache_calibrate_begin(D, k, workspace)
    if M > 0:
        sc.svdcache_calibrate_accumulate(stack_shard, workspace)
    torch.cuda.current_stream().synchronize()
    allreduce_gram(gram_view(workspace, D), group)
    return sc.svdcache_calibrate_finish(D, k, workspace, strict=strict)
