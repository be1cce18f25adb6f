"""Tensor-parallel use of the layer path: the output features of a linear layer split across ranks.

With dY = [dY^(0) | dY^(1) | ...] split by columns, every per-sequence gradient is the row stack
G_i = [G_i^(0); G_i^(1); ...] of the ranks' own d_out_local x d_in blocks, so

    K_ij = <G_i, G_j> = sum_r <G_i^(r), G_j^(r)>      (the layer NTK of Alg. 2 is a sum over parameter blocks)

and the rows of dW = sum_i c_i G_i belonging to rank r need only G^(r).  Each rank therefore runs the
three calls on its own columns of dY with ONE exchange in between: a sum of the B x B float32
matrix K over the ranks (<= 256 KB).  Every rank then solves the same small system and keeps its
rows of dW.  X is replicated (as it is after the all-gather or in the column-parallel layers of a
Megatron-style block); a row-parallel layer (X split by columns) is the same computation with the
roles of the column blocks swapped: G_i = [G_i^(0) | G_i^(1)], K again the sum.

The exchange is `torch.distributed.all_reduce` (NCCL between GPUs; any backend for the host-side
tests).  Nothing here touches the data except through the library's calls and that collective.
"""

from __future__ import annotations

import torch
import torch.distributed as dist


def allreduce_K(K: torch.Tensor, group=None) -> torch.Tensor:
    """Sums the ranks' partial K in place (no-op outside a process group or with one rank)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(K, op=dist.ReduceOp.SUM, group=group)
    return K


def shard_columns(d: int, rank: int, world: int, multiple: int = 8) -> tuple[int, int]:
    """[begin, end) of the columns rank `rank` owns: contiguous blocks whose widths are multiples of
    `multiple` (the bf16 kernels want widths divisible by 8), the first ranks one block wider."""
    if d % multiple or d // multiple < world:
        raise ValueError(f"cannot split {d} columns into {world} shards of multiples of {multiple}")
    blocks = d // multiple
    base, extra = divmod(blocks, world)
    begin = (rank * base + min(rank, extra)) * multiple
    return begin, begin + (base + (1 if rank < extra else 0)) * multiple


def isopo_layer_tp(X, dY_local, seq_offsets, A, variant, lam, group=None, path=None, pqr_regs=None):
    """One layer on this rank's columns of dY: local partial K, all-reduce, the transform (identical
    on every rank), this rank's rows of dW.  Returns binding.LayerResult with the full K, the
    coefficients and dW_local [d_out_local, d_in].  All ranks must pass the same `path` resolution,
    which holds when their shards have equal width (AUTO looks at the local sizes)."""
    from . import binding as b

    off = b._offsets(seq_offsets)
    B = off.shape[0] - 1
    dev = X.device
    path = b.PATH_AUTO if path is None else path
    ws = b.alloc_workspace(b._dtype_code(X), X.shape[0], X.shape[1], dY_local.shape[1], B, path, dev)
    K = torch.empty((B, B), dtype=torch.float32, device=dev)
    c = torch.empty(B, dtype=torch.float32, device=dev)
    dW = torch.empty((dY_local.shape[1], X.shape[1]), dtype=torch.float32, device=dev)
    info = torch.zeros(1, dtype=torch.int32, device=dev)
    b.isopo_layer_gram(X, dY_local, off, K, ws, info, path)
    allreduce_K(K, group)
    b.isopo_transform_advantages(K, A, variant, lam, c, info, pqr_regs)
    b.isopo_weight_grad(X, dY_local, c, off, dW, ws, info, path, 0.0)
    return b.LayerResult(K, c, dW, int(info.item()))
