"""A GWQ linear layer whose output rows are split over the ranks of a process group.

The path shards by rows: rank r owns the contiguous rows [row0, row1) of W, i.e. its code rows, its scale and
zero-point rows and its CSR rows; x is replicated.  The outlier location of Eq. "o" (Section 3.2) ranks the whole
matrix, so every rank selects on the whole (replicated) W and G and then cuts its own rows out of the result;
packing and the product are independent per rank, and ONE collective, an all-gather of y, puts the product together.
No arithmetic of the method lives here: selection, packing and the product are the library's calls
(``local_ops``), this module only computes the row ranges and moves y.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def row_range(N: int, world: int, rank: int, align: int = 128):
    """Rows [row0, row1) of rank `rank`: contiguous, in units of `align` rows (the tile height of the tensor-core
    kernels) as evenly as the units divide, the ragged last unit going to the last rank that owns any."""
    units = (N + align - 1) // align
    u0, u1 = units * rank // world, units * (rank + 1) // world
    return min(N, u0 * align), min(N, u1 * align)


def all_gather_rows(y_local: torch.Tensor, N: int, group=None) -> torch.Tensor:
    """y_local [M, rows of this rank] on every rank -> y [M, N] on every rank.  The ranks own different numbers of
    rows, so the pieces are padded to the largest shard for the collective and cut back afterwards."""
    world = dist.get_world_size(group)
    M = y_local.shape[0]
    ranges = [row_range(N, world, r) for r in range(world)]
    widest = max(r1 - r0 for r0, r1 in ranges)
    padded = y_local.new_zeros((M, widest))
    padded[:, :y_local.shape[1]] = y_local
    pieces = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(pieces, padded, group=group)
    y = y_local.new_empty((M, N))
    for (r0, r1), piece in zip(ranges, pieces):
        y[:, r0:r1] = piece[:, :r1 - r0]
    return y


class RowShardedLinear:
    """One rank's part of a row-sharded layer.  `local_ops` supplies the three steps on this rank's device:
    select(W, G, frac) -> S, rows(S, row0, row1) -> S_local, pack(W_local, S_local, bits, group) -> P, and
    linear(P, x) -> y_local (on a GPU these are the binding's gwq_* calls)."""

    def __init__(self, W, G, frac: float, bits: int, group: int, local_ops, process_group=None):
        self.group = process_group
        self.N = W.shape[0]
        self.rank, self.world = dist.get_rank(process_group), dist.get_world_size(process_group)
        self.row0, self.row1 = row_range(self.N, self.world, self.rank)
        self.ops = local_ops
        self.P = None
        if self.row1 > self.row0:
            S = local_ops.select(W, G, frac)                       # the whole matrix: the ranking is global
            S_local = local_ops.rows(S, self.row0, self.row1)
            self.P = local_ops.pack(W[self.row0:self.row1], S_local, bits, group)

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        M = x.shape[0]
        if self.P is not None:
            y_local = self.ops.linear(self.P, x)
        else:
            y_local = x.new_zeros((M, 0), dtype=torch.float32)
        return all_gather_rows(y_local, self.N, self.group)


class CudaOps:
    """The library's calls on the current CUDA device."""

    @staticmethod
    def select(W, G, frac):
        from . import binding as gwq
        return gwq.gwq_select_outliers(W, G, frac)

    @staticmethod
    def rows(S, row0, row1):
        from . import binding as gwq
        return gwq.gwq_outliers_rows(S, row0, row1)

    @staticmethod
    def pack(W_local, S_local, bits, group):
        from . import binding as gwq
        return gwq.gwq_pack(W_local.contiguous(), S_local, bits, group)

    @staticmethod
    def linear(P, x):
        from . import binding as gwq
        return gwq.gwq_linear(P, x, out_dtype=torch.float32)
