"""One product split over the GPUs of a node by columns of W.

The columns of W (the outputs) are independent, so rank g of G holds columns [g m / G, (g + 1) m / G) as a format of its
own (its own stream, offset index and Huffman code), x is replicated on every rank, each rank multiplies its slice with
the ordinary kernels, and one all-gather of the output slices finishes the product.  The exchange is a library
collective (torch.distributed, NCCL on GPUs): the slices land in local memory, no kernel reads a peer's memory.

All ranks quantize the whole matrix the same way first (prune, share weights), so that the sharded product is the
product of the same quantized matrix as the unsharded format; the shards are then coded without further quantization.
"""
from __future__ import annotations

import numpy as np

from .binding import QUANT_NONE, Format


def column_bounds(m: int, world: int):
    """[lo, hi) of every rank: contiguous, in rank order, sizes differing by at most one column."""
    return [((m * g) // world, (m * (g + 1)) // world) for g in range(world)]


def quantized_matrix(kind: str, W: np.ndarray, **params) -> np.ndarray:
    """The pruned and weight-shared matrix the format of W stands for (host, via the library's own decode)."""
    f = Format(kind, W, **params)
    try:
        return f.decode_host()
    finally:
        f.close()


def gather_columns(y_local, bounds, rank: int, group=None, dist=None):
    """All-gather of the output slices.  y_local: torch tensor [hi - lo] or [hi - lo, B] of this rank; returns [m] or
    [m, B] on every rank.  Slices may differ in size by a column, so they travel padded to the widest."""
    import torch
    if dist is None:
        import torch.distributed as dist
    world = len(bounds)
    if world == 1:
        return y_local
    widest = max(hi - lo for lo, hi in bounds)
    tail = tuple(y_local.shape[1:])
    padded = torch.zeros((widest,) + tail, dtype=y_local.dtype, device=y_local.device)
    padded[: y_local.shape[0]] = y_local
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded, group=group)
    return torch.cat([p[: hi - lo] for p, (lo, hi) in zip(parts, bounds)], dim=0)


class ColumnSharded:
    """This rank's shard of a HAC or sHAC format of W, split by columns over the ranks of `group`."""

    def __init__(self, kind: str, W: np.ndarray, rank: int, world: int, group=None, seg_symbols=0, ri_bits=0, **quant):
        self.kind, self.rank, self.world, self.group = kind, rank, world, group
        self.n, self.m = W.shape
        self.bounds = column_bounds(self.m, world)
        lo, hi = self.bounds[rank]
        if hi <= lo:
            raise ValueError("more ranks than columns")
        Wq = quantized_matrix(kind, W, **quant) if quant else np.ascontiguousarray(W, dtype=np.float32)
        self.format = Format(kind, Wq[:, lo:hi], quantizer=QUANT_NONE, seg_symbols=seg_symbols, ri_bits=ri_bits)

    def upload(self, device="cuda"):
        self.format.upload(device)
        return self

    def dot(self, x, dist=None):
        """x: torch float32 CUDA tensor [n] or [n, B], the same on every rank.  Returns y [m] or [m, B] on every rank."""
        y_local = self.format.dot(x)
        return gather_columns(y_local, self.bounds, self.rank, self.group, dist)
