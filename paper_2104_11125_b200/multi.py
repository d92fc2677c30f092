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

This module only orders calls; all arithmetic is in the library's kernels.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import torch
import torch.distributed as dist

from . import binding


class LearnerRank:
    """One learner of a `world`-learner job.  `engine` is the object whose select / compress /
    reduce_rows are called (a binding.Context by default, created here)."""

    def __init__(self, d: int, k: int, beta: float, lr: float, group: Optional[dist.ProcessGroup] = None,
                 selector: int = binding.SELECTOR_TOPK, layers: Optional[Tuple[Sequence[int], Sequence[int]]] = None,
                 engine=None, device: Optional[torch.device] = None):
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
        self.engine.compress(grad, mem, self.idx, self.own)
        if self._flat_gather:
            dist.all_gather_into_tensor(self.rows, self.own, group=self.group)
        else:                                   # (gloo has no flat all-gather)
            dist.all_gather(list(self.rows.view(self.world, self.k).unbind(0)), self.own, group=self.group)
        self.engine.reduce_rows(self.rows, self.val, self.idx, weights)
        return self.idx, self.val

    def exchange_bytes(self) -> int:
        """Payload that crosses the interconnect per rank and step: the k broadcast indices and the
        (world - 1) foreign rows of the all-gather."""
        return 0 if self.world == 1 else 4 * self.k + 4 * self.k * (self.world - 1)
