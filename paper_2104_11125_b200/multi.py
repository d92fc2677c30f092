"""Learner-per-GPU deployment of the CLT-k step (Algorithm 1 with one learner per process).

Each rank owns one learner: its gradient, its memory, a replica of the weights.
Iteration t runs, on every rank,

    leader = t mod world                    (the cyclic leader of Eq. 2-3)
    leader:   idx = select(g, m)            scalecom_select
    all:      broadcast(idx, src=leader)    k int32 indices
    all:      own = compress(g, m, idx)     scalecom_compress: Eq. 3 gather + Eq. 4 memory update
    all:      rows = all_gather(own)        world x k floats, rank order
    all:      val = reduce_rows(rows)       scalecom_reduce_rows: Algorithm 1 line 10, and in the same
              theta[idx] -= lr * val        kernel line 12

The gathered rows are exchanged with an all-gather and summed locally in rank
order, not with an all-reduce: the sum then has one fixed order on every rank,
so the replicas stay bit-identical to one another and to the single-process
step over the same learners.  The traffic per rank is k indices in and
world * k values in, independent of d; no kernel waits on another rank -- every
exchange is a torch.distributed collective between kernel launches.

With exchange="peer" the all-gather is fused into the compressing kernel instead: every rank maps the
other ranks' gathered-rows buffers (CUDA IPC; the ranks of a node must number the devices alike) and
scalecom_compress_scatter stores each kept value straight into this rank's row of every buffer while the pass
runs.  What remains between the calls is a fence -- a one-word all-reduce -- so that nobody reduces rows
that are still being written; two buffers are used in turn, so that a fast rank's next step cannot overwrite
rows a slow rank is still reading.  The kernels still wait for nobody.

With exchange="peer-flags" the fence goes too: the compressing kernel, once its last block is through, stores
the step's tag into a flag word beside its row in every rank's buffer, and the reducing kernel polls its own
rank's flag words (bounded; TIMEOUT in the handle's status when a sender never arrives) before it reads the
rows.  The index broadcast is then the only collective of the step.  Here a kernel does wait for other ranks'
kernels, so the ranks must be on different GPUs.

Both peer forms store through pointers into other GPUs' memory, which is only legal once the storing
device has peer access to the owning device.  Before anything is mapped, every rank therefore checks that
each peer on another device of the same host is reachable (torch.cuda.can_device_access_peer) and enables
the access explicitly with scalecom_enable_peer_access; the ranks agree on the outcome, and if any pair lacks
access (or a peer sits on another host) all of them fall back to exchange="collective" with a warning.

This module only orders calls; all arithmetic is in the library's kernels.
"""
from __future__ import annotations

import socket
import warnings
from typing import Callable, Optional, Sequence, Tuple

import torch
import torch.distributed as dist

from . import binding


class LearnerRank:
    """One learner of a `world`-learner job.  `engine` is the object whose select / compress /
    reduce_rows are called (a binding.Context by default, created here)."""

    def __init__(self, d: int, k: int, beta: float, lr: float, group: Optional[dist.ProcessGroup] = None,
                 selector: int = binding.SELECTOR_TOPK, layers: Optional[Tuple[Sequence[int], Sequence[int]]] = None,
                 engine=None, device: Optional[torch.device] = None, exchange: str = "collective",
                 can_access_peer: Optional[Callable[[int, int], bool]] = None):
        if not dist.is_initialized():
            raise RuntimeError("torch.distributed must be initialised before a LearnerRank is made")
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.d, self.k, self.lr = int(d), int(k), float(lr)
        self._flat_gather = dist.get_backend(group) == "nccl"
        if engine is None:
            engine = binding.Context(d, 1, k, beta, lr, stream=torch.cuda.current_stream())
            engine.set_option(binding.OPT_SELECTOR, selector)
            if layers is not None:
                engine.set_layers(*layers)
            device = torch.device("cuda", torch.cuda.current_device())
        self.engine = engine
        dev = device if device is not None else torch.device("cpu")
        self.idx = torch.empty(self.k, dtype=torch.int32, device=dev)
        self.own = torch.empty(self.k, dtype=torch.float32, device=dev)
        self.rows = torch.empty(self.world * self.k, dtype=torch.float32, device=dev)
        self.val = torch.empty(self.k, dtype=torch.float32, device=dev)
        if exchange not in ("collective", "peer", "peer-flags"):
            raise ValueError("exchange must be 'collective', 'peer' or 'peer-flags'")
        self.exchange = exchange
        self._can_access_peer = can_access_peer if can_access_peer is not None else torch.cuda.can_device_access_peer
        if exchange != "collective":
            peer_devices = self._reachable_peer_devices(dev)
            if peer_devices is None:
                warnings.warn("scalecom: exchange=%r needs peer access between all ranks' devices on one host; "
                              "at least one pair lacks it, every rank falls back to exchange='collective'" % exchange)
                self.exchange = "collective"
            else:
                if not isinstance(self.engine, binding.Context):
                    raise ValueError("exchange='peer' needs the CUDA engine")
                for other in peer_devices:                  # the device whose kernels store gets the access
                    self.engine.enable_peer_access(other)
                self._map_peer_rows(dev)

    def _reachable_peer_devices(self, dev: torch.device):
        """The other devices this rank's kernels would store to (device indices, same host), or None when any rank
        of the group reports a peer it cannot reach.  Every rank returns None together."""
        mine = (socket.gethostname(), dev.type, dev.index if dev.index is not None else -1 - self.rank)
        keys = [None] * self.world
        dist.all_gather_object(keys, mine, group=self.group)
        others, ok = [], True
        for r, (host, kind, index) in enumerate(keys):
            if r == self.rank or (host, kind, index) == mine:
                continue                                    # this rank, or a rank sharing this device
            if host != mine[0] or kind != "cuda" or mine[1] != "cuda" or not self._can_access_peer(mine[2], index):
                ok = False
            elif index not in others:
                others.append(index)
        verdicts = [None] * self.world
        dist.all_gather_object(verdicts, ok, group=self.group)
        return others if all(verdicts) else None

    def _map_peer_rows(self, dev: torch.device) -> None:
        """Two gathered-rows buffers [2][world][k] per rank and their flag words [2][world], each mapped into
        every other rank (one allocation: the flags are the tail of the rows' tensor)."""
        from torch.multiprocessing.reductions import reduce_tensor
        nrow = 2 * self.world * self.k
        self._shared = torch.zeros(nrow + 2 * self.world, dtype=torch.float32, device=dev)
        self._flag = torch.zeros(1, dtype=torch.int32, device=dev)
        torch.cuda.synchronize(dev)

        def split(buf):
            return buf[:nrow].view(2, self.world, self.k), buf[nrow:].view(torch.int32).view(2, self.world)

        self.rows2, self.flags2 = split(self._shared)
        if self.world == 1:
            self.peer_rows, self.peer_flags = [self.rows2], [self.flags2]
            return
        handles = [None] * self.world
        dist.all_gather_object(handles, reduce_tensor(self._shared), group=self.group)
        self.peer_rows, self.peer_flags, self._mapped = [], [], []
        for r, (rebuild, args) in enumerate(handles):
            buf = self._shared if r == self.rank else rebuild(*args)
            self._mapped.append(buf)
            rows, flags = split(buf)
            self.peer_rows.append(rows)
            self.peer_flags.append(flags)
        dist.barrier(group=self.group)                  # everyone has mapped everyone before the first store

    def _fence(self) -> None:
        """Returns (in stream order) once every rank's kernels issued so far have finished."""
        if self._flat_gather:                           # NCCL: ordered on the stream, no host wait
            dist.all_reduce(self._flag, group=self.group)
        else:
            torch.cuda.current_stream().synchronize()
            dist.barrier(group=self.group)

    def leader(self, t: int) -> int:
        return int(t) % self.world

    def step(self, grad: torch.Tensor, mem: torch.Tensor, weights: Optional[torch.Tensor], t: int
             ) -> Tuple[torch.Tensor, torch.Tensor]:
        """One iteration; mem (and weights, if given) are updated in place.  Returns (idx, val):
        views of buffers that the next step overwrites."""
        leader = self.leader(t)
        if self.rank == leader:
            self.engine.select(grad, mem, self.idx)
        src = leader if self.group is None else dist.get_global_rank(self.group, leader)
        dist.broadcast(self.idx, src=src, group=self.group)
        # the leader's handle still holds its selection: no need to hand the list back to it
        own_list = None if self.rank == leader else self.idx
        if self.exchange != "collective":
            b = int(t) & 1
            dst = [rows[b, self.rank] for rows in self.peer_rows]
            if self.exchange == "peer":
                self.engine.compress_scatter(grad, mem, own_list, self.own, dst)
                self._fence()
                self.engine.reduce_rows(self.rows2[b].view(-1), self.val, self.idx, weights)
            else:
                tag = int(t) + 1                        # never 0, new at every step
                self.engine.compress_scatter(grad, mem, own_list, self.own, dst,
                                             [flags[b, self.rank:self.rank + 1] for flags in self.peer_flags], tag)
                self.engine.reduce_rows(self.rows2[b].view(-1), self.val, self.idx, weights, self.flags2[b], tag)
            return self.idx, self.val
        self.engine.compress(grad, mem, own_list, self.own)
        if self._flat_gather:
            dist.all_gather_into_tensor(self.rows, self.own, group=self.group)
        else:                                   # (gloo has no flat all-gather)
            dist.all_gather(list(self.rows.view(self.world, self.k).unbind(0)), self.own, group=self.group)
        self.engine.reduce_rows(self.rows, self.val, self.idx, weights)
        return self.idx, self.val

    def close(self) -> None:
        """Drop the mappings of the peers' buffers (every rank, together), then the handle."""
        if getattr(self, "peer_rows", None) is not None and self.world > 1:
            torch.cuda.synchronize()
            self.peer_rows = self.peer_flags = self._mapped = None
            dist.barrier(group=self.group)              # nobody frees a buffer that a peer still has mapped
        self.peer_rows = self.peer_flags = None
        if isinstance(self.engine, binding.Context):
            self.engine.close()

    def exchange_bytes(self) -> int:
        """Payload that crosses the interconnect per rank and step: the k broadcast indices and the
        (world - 1) foreign rows of the all-gather."""
        return 0 if self.world == 1 else 4 * self.k + 4 * self.k * (self.world - 1)
