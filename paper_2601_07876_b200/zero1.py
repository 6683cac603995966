"""ZeRO-1 style sharding of one parameter group over the ranks of a process group.

Every rank holds the whole flat parameter buffer (for forward / backward) but
only 1/world of the optimizer state.  One step:

    reduce-scatter(gradients, average)  ->  NOVAK step on the owned range
                                        ->  all-gather(parameters)

The NOVAK step has no cross-element term, so the owned range may cut tensors
anywhere; nothing is exchanged inside the step itself, and the ranks only have
to take the same number of steps for their lookahead synchronisations to
coincide.  Two options need a norm over the WHOLE group, gradient clipping and
the automatic learning-rate scaling: for them the step runs in two halves
(novak_step_begin / novak_step_finish) with one all-reduce of two doubles (the
ranks' sums of squares of gradients and parameters) in between.
Centralization and layer adaptation work on whole tensors, which an arbitrary
cut of the flat space does not keep together: this class refuses them.

Only argument marshalling and collectives live here: the local step is
whatever ``make_local`` returns (the CUDA optimizer on a GPU; the tests plug in
the CPU oracle to exercise the collectives under gloo).
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import sharding

ALIGN = 64      # elements: 256 bytes of fp32, so every rank's range starts 16-byte aligned


def padded_numel(total: int, world: int) -> int:
    """Length of the flat buffers: the next multiple of world x ALIGN elements."""
    unit = world * ALIGN
    return -(-total // unit) * unit


class ShardedNovak:
    """``flat_params``: one contiguous fp32 buffer of ``padded_numel(sum(numel), world)``
    elements holding the group's tensors back to back (tensor i at the sum of the
    earlier ``numel``); identical on every rank.  ``make_local(pieces)`` builds the
    local optimizer over this rank's pieces (views into ``flat_params``) and must
    return an object with ``step(list_of_gradient_views)``."""

    def __init__(self, flat_params: torch.Tensor, numel, make_local=None, group=None,
                 **hyper):
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.numel = [int(n) for n in numel]
        self.total = sum(self.numel)
        if flat_params.dim() != 1 or flat_params.numel() != padded_numel(self.total, self.world):
            raise ValueError("flat_params must be a 1-d buffer of padded_numel(total, world) elements")
        for key in ("centralize", "layer_adaptation"):
            if hyper.get(key):
                raise ValueError(f"{key} works on whole tensors: not available for a flat-range shard")
        self.two_halves = bool(hyper.get("clip_threshold") or hyper.get("auto_lr"))
        self.flat_params = flat_params
        self.shard = flat_params.numel() // self.world
        lo = self.rank * self.shard
        self.lo, self.hi = lo, min(lo + self.shard, self.total)   # owned elements (padding excluded)
        self.slices = self._owned_slices()
        self.param_shard = flat_params[lo:lo + self.shard]
        self.grad_shard = torch.zeros_like(self.param_shard)
        pieces = [self.param_shard[a - lo:b - lo] for a, b in self._flat_ranges()]
        if make_local is None:
            from .binding import NovakOptimizer
            make_local = lambda ps: NovakOptimizer(ps, **hyper) if ps else None
        self.local = make_local(pieces)
        self.totals = torch.zeros(2, dtype=torch.float64, device=flat_params.device)
        self.steps = 0

    def _flat_ranges(self):
        """Owned ranges of the flat space, one per tensor piece."""
        out, base = [], 0
        for n in self.numel:
            a, b = max(base, self.lo), min(base + n, self.hi)
            if a < b:
                out.append((a, b))
            base += n
        return out

    def _owned_slices(self):
        """(tensor, start, stop) of every owned piece, as sharding.partition_flat gives them."""
        out, base = [], 0
        for t, n in enumerate(self.numel):
            a, b = max(base, self.lo), min(base + n, self.hi)
            if a < b:
                out.append((t, a - base, b - base))
            base += n
        return out

    def step(self, flat_grads: torch.Tensor):
        """``flat_grads``: this rank's gradient of the whole group, laid out like
        ``flat_params`` (padding ignored).  After the call ``flat_params`` holds the
        updated parameters of the whole group on every rank."""
        if flat_grads.shape != self.flat_params.shape:
            raise ValueError("flat_grads must have the layout of flat_params")
        backend = dist.get_backend(self.group)
        if backend == "gloo":
            # gloo has no reduce-scatter: all-reduce, then keep the owned range
            dist.all_reduce(flat_grads, op=dist.ReduceOp.SUM, group=self.group)
            self.grad_shard.copy_(flat_grads[self.rank * self.shard:(self.rank + 1) * self.shard])
            self.grad_shard.div_(self.world)
        else:
            dist.reduce_scatter_tensor(self.grad_shard, flat_grads, op=dist.ReduceOp.AVG,
                                       group=self.group)
        lo = self.lo
        grads = [self.grad_shard[a - lo:b - lo] for a, b in self._flat_ranges()]
        if not self.two_halves:
            if self.local is not None:
                self.local.step(grads)
        else:
            # local sums of squares -> all-reduce of two doubles -> norm, factors, update
            self.totals.zero_()
            if self.local is not None:
                self.local.step_begin(grads)
                self.local.copy_local_sums(self.totals)
            dist.all_reduce(self.totals, op=dist.ReduceOp.SUM, group=self.group)
            if self.local is not None:
                self.local.step_finish(self.totals)
        self.steps += 1
        # every rank's updated range lands in every rank's own buffer
        dist.all_gather_into_tensor(self.flat_params, self.param_shard, group=self.group)
