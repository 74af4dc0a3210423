"""One bucket's gradient exchange across the ranks of a torch.distributed group (Sec. 3.3 of the paper):

    send pass (Algorithm 1 steps 1-2)  ->  all-to-all of the packed parts  ->  local average (Eq. 8)

Rank r compresses its whole local gradient into P = world_size parts; part j travels to rank j; rank j averages
the P copies of part j it then holds and owns that shard of the averaged gradient (the sharded data-parallel
layout the paper assumes; the all-gather of updated weights that follows is the framework's own).  The paper
replaces reduce-scatter by all-to-all because codes cannot be summed hop by hop without leaving their range.

Two transports, both with every arithmetic step in the library's kernels:

  "collective"  the send pass fills a local buffer, one all_to_all_single (NCCL) moves the parts, the receive
                pass reads the local receive area.
  "peer_store"  the receive areas live in symmetric memory; the send pass stores part j straight into slot r of
                rank j's area through NVLink (loco_compensate_quantize_pack_scatter), one small all_reduce orders
                "everybody has stored" before "anybody reads", the receive pass reads local memory only.  No
                kernel of this library waits on another rank; two areas alternate from one exchange to the next so
                that a rank that is already one exchange ahead cannot overwrite slots that a slower rank is still
                reading.

Only plumbing lives here (buffers, pointers, the order of calls).  This module needs the CUDA library and a GPU per
rank; nothing in it has a CPU fallback.
"""
from __future__ import annotations

from typing import List, Optional

import torch
import torch.distributed as dist

from . import loco

TRANSPORTS = ("collective", "peer_store")


def slot_offset(cfg: "loco.Config", n: int, src_rank: int) -> int:
    """Byte offset, inside a rank's receive area, of the slot that holds the part sent by src_rank."""
    if not 0 <= src_rank < cfg.num_partitions:
        raise ValueError("source rank outside the group")
    return src_rank * loco.loco_partition_bytes(cfg, n)


def area_bytes(cfg: "loco.Config", n: int) -> int:
    """Bytes of one receive area: one slot per rank of the group."""
    return cfg.num_partitions * loco.loco_partition_bytes(cfg, n)


def area_index(seq: int) -> int:
    """Which of the two receive areas the seq-th exchange through a transport uses (peer_store)."""
    return seq & 1


def scatter_table(peer_area_ptrs: List[int], cfg: "loco.Config", n: int, my_rank: int) -> List[int]:
    """Destination of every part of rank my_rank's send pass: slot my_rank of each peer's receive area."""
    if len(peer_area_ptrs) != cfg.num_partitions:
        raise ValueError("one receive area per rank is needed")
    off = slot_offset(cfg, n, my_rank)
    return [int(p) + off for p in peer_area_ptrs]


def shard_elems(cfg: "loco.Config", n: int, rank: int) -> int:
    """Elements of the averaged gradient that rank owns after the exchange."""
    return loco.loco_partition_elems(cfg, n, rank)


class Transport:
    """The communication buffers of one rank, shared by all its buckets of at most n_max elements: buckets are
    exchanged one after the other on one stream, so they can take turns in the same memory.  `seq` counts the
    exchanges made through this object; the peer_store transport alternates its two areas on it."""

    def __init__(self, cfg: "loco.Config", n_max: int, group: Optional[dist.ProcessGroup] = None,
                 kind: str = "collective", device: Optional[torch.device] = None):
        if kind not in TRANSPORTS:
            raise ValueError("transport must be one of %s" % (TRANSPORTS,))
        if not dist.is_initialized():
            raise RuntimeError("torch.distributed is not initialised")
        self.group = group if group is not None else dist.group.WORLD
        self.world = dist.get_world_size(self.group)
        self.rank = dist.get_rank(self.group)
        if cfg.num_partitions != self.world:
            raise ValueError("num_partitions (%d) must equal the group's size (%d)" % (cfg.num_partitions, self.world))
        if device is None:
            device = torch.device("cuda", torch.cuda.current_device())
        self.cfg, self.n_max, self.kind, self.device = cfg, n_max, kind, device
        self.seq = 0
        nbytes = max(area_bytes(cfg, n_max), 16)
        if kind == "collective":
            self.comm = torch.empty(nbytes, dtype=torch.uint8, device=device)
            self.areas = [torch.empty(nbytes, dtype=torch.uint8, device=device)]
            self.peer_ptrs = None
        else:
            import os
            # this transport only stores through plain peer pointers: no NVLink multicast object is needed for it
            os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")
            import torch.distributed._symmetric_memory as symm_mem
            self.areas, self.peer_ptrs, self._handles = [], [], []
            for _ in range(2):
                area = symm_mem.empty(nbytes, dtype=torch.uint8, device=device)
                handle = symm_mem.rendezvous(area, self.group)
                self.areas.append(area)
                self._handles.append(handle)
                self.peer_ptrs.append([int(p) for p in handle.buffer_ptrs])
            self._token = torch.zeros(1, dtype=torch.float32, device=device)


class BucketExchange:
    """Error state of one bucket on one rank plus the transport it uses.  step() runs one iteration and leaves this
    rank's shard of the averaged gradient in `out` (shard_elems() values of cfg.out_dtype)."""

    def __init__(self, cfg: "loco.Config", n: int, group: Optional[dist.ProcessGroup] = None,
                 transport: str = "collective", device: Optional[torch.device] = None,
                 shared: Optional[Transport] = None):
        self.t = shared if shared is not None else Transport(cfg, n, group, transport, device)
        if n > self.t.n_max or cfg != self.t.cfg:
            raise ValueError("the shared transport was made for another configuration or a smaller bucket")
        self.cfg, self.n = cfg, n
        self.rank, self.world = self.t.rank, self.t.world
        self.part = loco.loco_partition_bytes(cfg, n)
        self.state = loco.State(cfg, n, device=self.t.device)
        self.tables = None
        if self.t.kind == "peer_store":
            self.tables = [scatter_table(ptrs, cfg, n, self.rank) for ptrs in self.t.peer_ptrs]

    def shard_elems(self) -> int:
        return shard_elems(self.cfg, self.n, self.rank)

    def _slots(self, area: torch.Tensor):
        return [area[slot_offset(self.cfg, self.n, w):slot_offset(self.cfg, self.n, w) + self.part] for w in range(self.world)]

    def step(self, grad: torch.Tensor, step_k: int, out: torch.Tensor) -> None:
        """All work is enqueued on the current stream; nothing synchronises the host."""
        t = self.t
        if t.kind == "collective":
            loco.loco_compensate_quantize_pack(self.state, grad, t.comm, step_k)
            area = t.areas[0]
            nbytes = self.world * self.part
            dist.all_to_all_single(area[:nbytes], t.comm[:nbytes], group=t.group)
        else:
            a = area_index(t.seq)
            area = t.areas[a]
            loco.loco_compensate_quantize_pack_scatter(self.state, grad, self.tables[a], step_k)
            dist.all_reduce(t._token, group=t.group)            # every rank's stores are complete once this has run
        t.seq += 1
        loco.loco_unpack_dequant_reduce(self.cfg, self._slots(area), self.n, out, first_partition=self.rank,
                                        partition_count=1)
