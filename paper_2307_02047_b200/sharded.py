"""Tensor-sharded CAME step across data-parallel ranks (optimizer-state sharding).

Tensors are independent in Algorithm 2 (no term couples two parameter tensors), so the step
shards by tensor with no change to the arithmetic: every tensor has one owner rank that holds
its optimizer state.  Per step

  1. gradients in:  every rank's gradients are summed onto the owners with a REDUCE-SCATTER
     over flat, byte-balanced buckets.  Rank r's tensors are laid end to end (each starting on a
     32-byte boundary) in "segment r"; all segments are padded to one length and cut into
     buckets of ``bucket_elems`` elements, so bucket b is a [world, chunk] array whose row r is
     slice b of segment r, and one reduce-scatter per bucket leaves slice b of the summed
     segment on its owner.  The sum is accumulated in fp32 whatever the gradient storage type
     (bf16 gradients are widened while they are packed).
  2. the owner runs the ordinary single-GPU step on its tensors, reading the summed fp32
     gradients in place, with ``grad_scale = 1/world`` (the mean of the ranks' gradients, folded
     into the kernels' scalars);
  3. parameters out: the owners' updated parameters travel back with one ALL-GATHER per bucket
     of the same layout, and every rank copies the slices it does not own into its replicas.

A step therefore issues 2 x (number of buckets) collectives, whatever the number of tensors.
The only data that crosses ranks is gradients in and parameters out; nothing inside the
kernels waits on another rank, and no kernel is handed another GPU's memory.

Communication uses ``torch.distributed`` (NCCL on GPUs; gloo works for CPU tests with an
injected local stepper -- gloo has no reduce-scatter, so there the bucket is all-reduced and
the owner keeps its row).
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence, Tuple

ALIGN_ELEMS = 8          # tensors start on 32-byte boundaries inside a segment (fp32 elements)


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


def segment_layout(numels: Sequence[int], owner: Sequence[int], world: int, bucket_elems: int
                   ) -> Tuple[List[int], int, int, int]:
    """Offsets of the tensors inside their owners' segments, and the bucket geometry.

    Returns ``(offset, seg_len, chunk, n_buckets)``: ``offset[i]`` is where tensor i starts in
    segment ``owner[i]``; every segment is ``seg_len = n_buckets * chunk`` elements long."""
    fill = [0] * world
    offset = [0] * len(numels)
    for i, n in enumerate(numels):
        r = owner[i]
        offset[i] = fill[r]
        fill[r] += (n + ALIGN_ELEMS - 1) // ALIGN_ELEMS * ALIGN_ELEMS
    longest = max(max(fill), ALIGN_ELEMS)
    chunk = min(max(bucket_elems // ALIGN_ELEMS * ALIGN_ELEMS, ALIGN_ELEMS), longest)
    n_buckets = (longest + chunk - 1) // chunk
    return offset, n_buckets * chunk, chunk, n_buckets


def bucket_pieces(numels: Sequence[int], owner: Sequence[int], offset: Sequence[int], chunk: int,
                  n_buckets: int) -> List[List[Tuple[int, int, int, int, int]]]:
    """For every bucket the pieces of tensors that fall into it:
    ``(tensor, lo, hi, rank, dst)`` = elements [lo, hi) of the flattened tensor go to row
    ``rank`` of the bucket at column ``dst``."""
    out: List[List[Tuple[int, int, int, int, int]]] = [[] for _ in range(n_buckets)]
    for i, n in enumerate(numels):
        start, end = offset[i], offset[i] + n
        b = start // chunk
        while start < end:
            stop = min(end, (b + 1) * chunk)
            out[b].append((i, start - offset[i], stop - offset[i], owner[i], start - b * chunk))
            start = stop
            b += 1
    return out


class ShardedCame:
    """``params``/``grads``: this rank's full replicas (same shapes on every rank).

    ``make_local(params_owned, grads_owned)`` builds the object that steps the owned tensors
    (``.step(**hparams)``, optional ``.close()``); ``grads_owned`` are fp32 views, shaped like
    the parameters, into this rank's summed-gradient segment.  The default is the CUDA
    ``CameOptimizer``.  ``bucket_elems``: elements per rank per collective (default 64 Mi:
    256 MB of fp32 per rank and bucket).
    """

    def __init__(self, params, grads, make_local: Optional[Callable] = None, group=None,
                 bucket_elems: int = 1 << 26):
        import torch
        import torch.distributed as dist
        self.torch, self.dist, self.group = torch, dist, group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.params, self.grads = list(params), list(grads)
        numels = [p.numel() for p in self.params]
        sizes = [p.numel() * (p.element_size() * 2 + g.element_size())
                 for p, g in zip(self.params, self.grads)]
        self.owner = partition_by_bytes(sizes, self.world)
        self.mine = [i for i, r in enumerate(self.owner) if r == self.rank]
        self.offset, self.seg_len, self.chunk, self.n_buckets = segment_layout(
            numels, self.owner, self.world, bucket_elems)
        self.pieces = bucket_pieces(numels, self.owner, self.offset, self.chunk, self.n_buckets)
        dev = self.params[0].device
        pdt = self.params[0].dtype
        # the sum of the ranks' gradients is accumulated in (at least) fp32
        self.acc_dtype = torch.float64 if self.grads[0].dtype == torch.float64 else torch.float32
        self.grad_seg = torch.zeros(self.seg_len, dtype=self.acc_dtype, device=dev)
        self.param_seg = torch.zeros(self.seg_len, dtype=pdt, device=dev)
        self.stage_g = [torch.zeros((self.world, self.chunk), dtype=self.acc_dtype, device=dev)
                        for _ in range(min(2, self.n_buckets))]
        self.stage_p = [torch.zeros((self.world, self.chunk), dtype=pdt, device=dev)
                        for _ in range(min(2, self.n_buckets))]
        self.has_reduce_scatter = dist.get_backend(group) == "nccl"
        if make_local is None:
            from . import binding
            make_local = lambda p, g: binding.CameOptimizer(p, g, device=p[0].device.index or 0)
        owned_g = [self.grad_seg[self.offset[i]:self.offset[i] + numels[i]].view(self.params[i].shape)
                   for i in self.mine]
        self.local = make_local([self.params[i] for i in self.mine], owned_g) if self.mine else None
        self.collectives_per_step = 2 * self.n_buckets

    # -- gradients in ------------------------------------------------------------------------
    def _reduce_gradients(self) -> None:
        dist = self.dist
        works = [None] * len(self.stage_g)
        for b in range(self.n_buckets):
            k = b % len(self.stage_g)
            if works[k] is not None:
                works[k].wait()                       # the bucket that used this staging buffer
            st = self.stage_g[k]
            for (i, lo, hi, r, dst) in self.pieces[b]:
                st[r, dst:dst + (hi - lo)].copy_(self.grads[i].reshape(-1)[lo:hi])
            out = self.grad_seg[b * self.chunk:(b + 1) * self.chunk]
            if self.has_reduce_scatter:
                works[k] = dist.reduce_scatter_tensor(out, st.view(-1), op=dist.ReduceOp.SUM,
                                                      group=self.group, async_op=True)
            else:
                dist.all_reduce(st, op=dist.ReduceOp.SUM, group=self.group)
                out.copy_(st[self.rank])
        for w in works:
            if w is not None:
                w.wait()

    # -- parameters out ----------------------------------------------------------------------
    def _gather_parameters(self) -> None:
        dist = self.dist
        for i in self.mine:
            n = self.params[i].numel()
            self.param_seg[self.offset[i]:self.offset[i] + n].copy_(self.params[i].reshape(-1))
        for b in range(self.n_buckets):
            st = self.stage_p[b % len(self.stage_p)]
            dist.all_gather_into_tensor(st.view(-1), self.param_seg[b * self.chunk:(b + 1) * self.chunk],
                                        group=self.group)
            for (i, lo, hi, r, dst) in self.pieces[b]:
                if r != self.rank:
                    self.params[i].view(-1)[lo:hi].copy_(st[r, dst:dst + (hi - lo)])

    def step(self, **hp) -> None:
        self._reduce_gradients()
        if self.local is not None:
            scale = float(hp.get("grad_scale", 1.0)) / self.world
            self.local.step(**dict(hp, grad_scale=scale))
        self._gather_parameters()

    def close(self) -> None:
        if self.local is not None and hasattr(self.local, "close"):
            self.local.close()
