"""The exchange step between data-parallel ranks (Eq. 2 "Sync", Eq. 12 third line).

Every rank compresses the gradients of its own workers; what crosses the wire is the payload
(neighborhood indices, values, per-layer counts).  The per-layer keep ratios come from the
replicated weights, so every rank keeps the same number of neighborhoods per layer and the
messages have one fixed size: the exchange is a single all-gather of one packed buffer per
rank (NCCL over NVLink on GPUs, gloo in the CPU tests), after which each rank aggregates all
the payloads on its own memory with rsdgc_decompress_accumulate() / rsdgc_decompress_assign().
Workers are summed in the order of their global id (rank-major) on every rank, so all replicas
end up with bit-identical dense gradients.
"""
from __future__ import annotations

from typing import List, Tuple

import torch


def _round16(n: int) -> int:
    return (n + 15) & ~15


class PayloadExchange:
    """Packed send / receive buffers of the payload all-gather.

    One worker's message is ``counts`` (n_layers int32), ``idx`` (idx_capacity int32) and ``val``
    (val_capacity values of ``val_dtype``), each section padded to 16 bytes.  ``local_views(w)``
    are tensors inside the send buffer: hand them to the compress call and nothing has to be
    copied before the all-gather."""

    def __init__(self, n_layers: int, idx_capacity: int, val_capacity: int, n_local_workers: int, world: int,
                 rank: int, device, val_dtype: torch.dtype = torch.float32, always_gather: bool = False):
        self.n_layers, self.ni, self.nv = int(n_layers), int(idx_capacity), int(val_capacity)
        self.n_local, self.world, self.rank = int(n_local_workers), int(world), int(rank)
        self.val_dtype = val_dtype
        esz = torch.empty(0, dtype=val_dtype).element_size()
        self._off_idx = _round16(4 * self.n_layers)
        self._off_val = self._off_idx + _round16(4 * self.ni)
        self.msg_bytes = self._off_val + _round16(esz * self.nv)
        self.send = torch.zeros(self.n_local * self.msg_bytes, dtype=torch.uint8, device=device)
        # with one rank the gathered payloads are the local ones: no second buffer, no copy
        # (always_gather: run the collective all the same, e.g. to time or test it on one GPU)
        self._skip = self.world == 1 and not always_gather
        self.recv = self.send if self._skip else torch.zeros(self.world * self.n_local * self.msg_bytes,
                                                                  dtype=torch.uint8, device=device)

    def _views(self, buf: torch.Tensor, slot: int) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        base = slot * self.msg_bytes
        esz = torch.empty(0, dtype=self.val_dtype).element_size()
        counts = buf[base:base + 4 * self.n_layers].view(torch.int32)
        idx = buf[base + self._off_idx:base + self._off_idx + 4 * self.ni].view(torch.int32)
        val = buf[base + self._off_val:base + self._off_val + esz * self.nv].view(self.val_dtype)
        return idx, val, counts

    def local_views(self, w: int) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """(idx, val, counts) of local worker ``w`` inside the send buffer."""
        return self._views(self.send, w)

    def gathered_views(self) -> List[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]]:
        """(idx, val, counts) of every worker of every rank, by global worker id."""
        return [self._views(self.recv, s) for s in range(self.world * self.n_local)]

    def exchange(self) -> None:
        """All-gather of the packed payloads (asynchronous on the current stream with NCCL)."""
        if self._skip:
            return
        import torch.distributed as dist

        dist.all_gather_into_tensor(self.recv, self.send)

    def aggregate(self, plan, dense: torch.Tensor, scale: float = 1.0, assign: bool = False) -> None:
        """dense (+)= scale * sum over all workers of all ranks (device tensors only)."""
        plan.decompress_accumulate(self.gathered_views(), dense, scale, assign=assign)
