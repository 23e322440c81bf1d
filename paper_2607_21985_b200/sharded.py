"""Row-tile sharding of the decode product over the ranks of a torch.distributed process group.

The paper leaves multi-GPU execution as future work (Sec. 6).  y = W x splits by rows without any
change to the method: rank k packs the row tiles spdp_row_shard gives it as its own Tiled-CBC matrix,
every rank holds the whole activation vector x and applies the same dynamic-pruning test to it, and
the partial outputs are disjoint slices of y.  One collective follows the local product: an
all-gather of the slices (NCCL over NVLink on GPUs; any backend works, the CPU tests use gloo).
No kernel ever reads another GPU's memory.

Row sharding leaves each row's summation order inside a rank's kernel, so a row's value does not
depend on the other ranks; it does depend on how that rank's matrix is cut over its CTAs.

Plumbing only: the product itself is whatever `local_product` computes (the CUDA library's
spdp_spmspv on a GPU; the tests inject the CPU oracle to exercise the collective path without one).
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import spdp


class RowShardedMatrix:
    """This rank's share of W and the buffers of the gathered output.

    pack(rows_of_W) -> handle is called with the rank's row slice [first_row, first_row + rows);
    local_product(handle, x, y_slice) must fill y_slice (a view of `rows` entries)."""

    def __init__(self, M: int, K: int, row_slice_of, pack, local_product, *, device, dtype=torch.float16, group=None):
        self.group = group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.M, self.K = M, K
        self.first_row, self.rows = spdp.spdp_row_shard(M, self.world, self.rank)
        shards = [spdp.spdp_row_shard(M, self.world, r) for r in range(self.world)]
        self.chunk = max(rows for _, rows in shards)                 # equal-size slots for the all-gather
        self.shards = shards
        self.local_product = local_product
        self.handle = pack(row_slice_of(self.first_row, self.rows)) if self.rows > 0 else None
        self.gathered = torch.zeros(self.world * self.chunk, dtype=dtype, device=device)
        self.mine = self.gathered[self.rank * self.chunk:(self.rank + 1) * self.chunk]

    def spmspv(self, x, *args):
        """y = W x over the active columns; returns the full y (M entries) on every rank."""
        if self.rows > 0:
            self.local_product(self.handle, x, self.mine[:self.rows], *args)
        if self.world > 1:
            dist.all_gather_into_tensor(self.gathered, self.mine, group=self.group)
        if all(rows == self.chunk for _, rows in self.shards):
            return self.gathered[:self.M]
        return torch.cat([self.gathered[r * self.chunk:r * self.chunk + rows] for r, (_, rows) in enumerate(self.shards)])
