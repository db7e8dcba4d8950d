"""Token-sharded data parallelism of the split-FP4 layer: host-side plumbing only.

The path shards over tokens (rows of X and dY): forward and the input gradient are independent per shard
given the replicated weight operand, every shard splits and quantizes its own rows, and the weight gradient
is the one quantity that needs an exchange: a sum over shards (torch.distributed all-reduce, NCCL on GPUs).
"""
import torch
import torch.distributed as dist


def shard_rows(total_rows, rank, world, multiple=64):
    """Contiguous row range [start, stop) of `rank`; every shard but the last is a multiple of `multiple` rows
    (the block-scaled kernels need whole 16-element blocks, the tiled scale layout whole groups of 64)."""
    per = -(-total_rows // world)
    per = -(-per // multiple) * multiple
    start = min(rank * per, total_rows)
    stop = min(start + per, total_rows)
    return start, stop


def allreduce_weight_grad_(dw):
    """Sums the per-shard weight gradients in place across the default process group (no-op for one rank)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(dw, op=dist.ReduceOp.SUM)
    return dw
