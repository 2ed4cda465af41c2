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

from typing import List, Sequence, Tuple

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


# ---------------------------------------------------------------------------------------------
# the exchange overlapped with the compression: layer groups
# ---------------------------------------------------------------------------------------------

def keep_count(n_tiles: int, ratio: float, keep_at_least_one: bool = True) -> int:
    """k_l = ceil(K_l * ratio_l) limited to [0 or 1, K_l] (Eq. 11), the product taken in binary64 on the
    binary32 ratio: the number the compression kernels arrive at, computed on the host so that message
    sizes are known before anything is compressed."""
    import math
    import struct

    r32 = struct.unpack("f", struct.pack("f", float(ratio)))[0]
    x = math.ceil(float(n_tiles) * r32)
    k = 0 if x <= 0 else (n_tiles if x >= n_tiles else int(x))
    if keep_at_least_one and k < 1:
        k = 1
    return min(k, n_tiles)


def split_layers(shapes: Sequence[Tuple[int, int, int, int]], n_groups: int) -> List[Tuple[int, int]]:
    """Contiguous layer ranges [lo, hi) of about equal element counts (at most n_groups, none empty)."""
    sizes = [r * c for r, c, _, _ in shapes]
    total, out, lo, acc = sum(sizes), [], 0, 0
    n_groups = max(1, min(int(n_groups), len(shapes)))
    for l, n in enumerate(sizes):
        acc += n
        left_layers, left_groups = len(shapes) - (l + 1), n_groups - (len(out) + 1)
        if left_groups > 0 and (acc >= total * (len(out) + 1) / n_groups or left_layers == left_groups):
            out.append((lo, l + 1))
            lo = l + 1
    out.append((lo, len(shapes)))
    return [g for g in out if g[0] < g[1]]


class GroupedExchange:
    """Eq. 2's Sync overlapped with the compression (the paper names the exchange, Eq. 2 and Eq. 12's
    third line; how it is scheduled is this library's): the layers are cut into groups, every group has
    its own plan, and while group i + 1 is compressed on the caller's stream the payloads of group i
    travel on a second stream.  A message holds exactly what is sent: per worker the counts, sum_l k_l
    tile indices and sum_l k_l * nh_l * nw_l values of the group (k_l follows from the replicated ratios,
    so every rank knows every size before the exchange).  Aggregation runs group by group over all ranks'
    workers in global worker order on local memory, so every replica gets bit-identical dense gradients,
    identical to the ungrouped result.  NCCL moves the bytes (gloo in the CPU tests); the kernels only
    touch local memory.

    ``plans``: one binding.Plan per group (host-only plans suffice for the layout and the exchange).
    """

    def __init__(self, shapes: Sequence[Tuple[int, int, int, int]], groups: Sequence[Tuple[int, int]], plans,
                 n_local_workers: int, world: int, rank: int, device, val_dtype: torch.dtype = torch.float32,
                 keep_at_least_one: bool = True, always_gather: bool = False):
        self.shapes, self.groups, self.plans = list(shapes), list(groups), list(plans)
        self.n_local, self.world, self.rank, self.device = int(n_local_workers), int(world), int(rank), device
        self.val_dtype, self.clamp = val_dtype, keep_at_least_one
        self._skip = self.world == 1 and not always_gather
        self.exchanges: List[PayloadExchange] = []
        self._comm = None
        self._sent = self._done = None

    def set_ratios(self, ratios: Sequence[float]) -> None:
        """Sizes the messages for the given per-layer ratios (host values; call when the ratios change)."""
        self.exchanges = []
        for (lo, hi), plan in zip(self.groups, self.plans):
            ks = [keep_count(li.n_tiles, ratios[lo + j], self.clamp) for j, li in enumerate(plan.layers)]
            ni = sum(ks)
            nv = sum(k * li.nh * li.nw for k, li in zip(ks, plan.layers))
            self.exchanges.append(PayloadExchange(hi - lo, ni, nv, self.n_local, self.world, self.rank, self.device,
                                                  self.val_dtype, always_gather=not self._skip))

    def message_bytes(self) -> int:
        """Bytes one rank sends per step (all groups, all local workers)."""
        return sum(ex.msg_bytes * self.n_local for ex in self.exchanges)

    def local_views(self, group: int, w: int):
        return self.exchanges[group].local_views(w)

    def gathered_views(self, group: int):
        return self.exchanges[group].gathered_views()

    def exchange_group(self, group: int) -> None:
        """The all-gather of one group's payloads on the current stream."""
        self.exchanges[group].exchange()

    def step(self, grads, residuals, ratios_dev, workspaces, dense, scale: float = 1.0, assign: bool = True) -> None:
        """One iteration on the GPU.  Per group g: ``grads[g]`` / ``residuals[g]`` are lists with one arena per
        local worker, ``ratios_dev[g]`` the group's ratios, ``workspaces[g]`` n_local * workspace_bytes bytes,
        ``dense[g]`` the group's dense arena.  Group g + 1 is compressed while group g's payloads travel."""
        main = torch.cuda.current_stream()
        if self._comm is None:
            self._comm = torch.cuda.Stream()
            self._sent = [torch.cuda.Event() for _ in self.groups]
            self._done = [torch.cuda.Event() for _ in self.groups]
        for g, (plan, ex) in enumerate(zip(self.plans, self.exchanges)):
            views = [ex.local_views(w) for w in range(self.n_local)]
            plan.reserve_workers(self.n_local)
            plan.compress_workers(grads[g], residuals[g], ratios_dev[g], [v[0] for v in views], [v[1] for v in views],
                                  [v[2] for v in views], workspaces[g])
            if not self._skip:
                self._sent[g].record(main)
                with torch.cuda.stream(self._comm):
                    self._comm.wait_event(self._sent[g])
                    ex.exchange()
                    self._done[g].record(self._comm)
        for g, (plan, ex) in enumerate(zip(self.plans, self.exchanges)):
            if not self._skip:
                main.wait_event(self._done[g])
            ex.aggregate(plan, dense[g], scale, assign=assign)
