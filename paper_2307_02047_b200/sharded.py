"""Tensor-sharded CAME step across data-parallel ranks (optimizer-state sharding).

Tensors are independent in Algorithm 2 (no term couples two parameter tensors), so the step
shards by tensor with no change to the arithmetic: every tensor has one owner rank that holds
its optimizer state; per step the gradients are summed onto the owner, the owner runs the
ordinary single-GPU step on its tensors with ``grad_scale = 1/world`` (the mean of the ranks'
gradients, folded into the kernels' scalars), and the updated parameters are broadcast back.
The only data that crosses ranks is gradients in and parameters out; nothing inside the
kernels waits on another rank.

Communication uses ``torch.distributed`` (NCCL on GPUs; gloo works for CPU tests with an
injected local stepper).
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence


def partition_by_bytes(sizes: Sequence[int], world: int) -> List[int]:
    """Owner rank of every tensor: largest first, each to the least-loaded rank (ties -> lowest
    rank), which keeps the per-rank byte totals within one tensor of each other."""
    assert world >= 1
    load = [0] * world
    owner = [0] * len(sizes)
    for i in sorted(range(len(sizes)), key=lambda k: (-sizes[k], k)):
        r = min(range(world), key=lambda k: (load[k], k))
        owner[i] = r
        load[r] += sizes[i]
    return owner


class ShardedCame:
    """``params``/``grads``: this rank's full replicas (same shapes on every rank).

    ``make_local(params_owned, grads_owned)`` builds the object that steps the owned tensors
    (``.step(**hparams)``, optional ``.close()``); the default is the CUDA ``CameOptimizer``.
    """

    def __init__(self, params, grads, make_local: Optional[Callable] = None, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.params, self.grads = list(params), list(grads)
        sizes = [p.numel() * (p.element_size() * 2 + g.element_size())
                 for p, g in zip(self.params, self.grads)]
        self.owner = partition_by_bytes(sizes, self.world)
        self.mine = [i for i, r in enumerate(self.owner) if r == self.rank]
        if make_local is None:
            from . import binding
            make_local = lambda p, g: binding.CameOptimizer(p, g, device=p[0].device.index or 0)
        self.local = make_local([self.params[i] for i in self.mine],
                                [self.grads[i] for i in self.mine]) if self.mine else None

    def _global_rank(self, r: int) -> int:
        return self.dist.get_global_rank(self.group, r) if self.group is not None else r

    def step(self, **hp) -> None:
        dist = self.dist
        works = [dist.reduce(g, dst=self._global_rank(self.owner[i]), op=dist.ReduceOp.SUM,
                             group=self.group, async_op=True) for i, g in enumerate(self.grads)]
        for w in works:
            w.wait()
        if self.local is not None:
            scale = float(hp.get("grad_scale", 1.0)) / self.world
            self.local.step(**dict(hp, grad_scale=scale))
        works = [dist.broadcast(p, src=self._global_rank(self.owner[i]), group=self.group,
                                async_op=True) for i, p in enumerate(self.params)]
        for w in works:
            w.wait()

    def close(self) -> None:
        if self.local is not None and hasattr(self.local, "close"):
            self.local.close()
