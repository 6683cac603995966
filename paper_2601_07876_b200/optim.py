"""``torch.optim.Optimizer`` front end of the NOVAK step library.

The paper's method is used as a PyTorch optimizer (Algorithm 1: parameters,
hyperparameters, ``step`` with an optional closure for the true Nesterov
variant).  This class only collects pointers and forwards: every parameter
group is one handle of the C-ABI library (one fused multi-tensor step per
group), ``p.grad`` supplies the gradients, and a closure passed to ``step``
is evaluated at Eq. 10's look-ahead point while the group is in its first
N_taylor steps (Section 5.8: save, extrapolate, evaluate; the step then reads the
saved parameters, which is the restore).  No arithmetic of the method happens here.
"""
from __future__ import annotations

import torch

from . import binding as B

_GROUP_KEYS = ("lr", "betas", "eps", "weight_decay", "nesterov", "lookahead_k", "lookahead_alpha",
               "nesterov_beta", "lookahead_mode", "rectified", "clip_threshold", "centralize",
               "adaptive_beta", "layer_adaptation", "sparse_threshold", "auto_lr",
               "true_nesterov_steps", "moment_dtype", "graph_capturable")


class Novak(torch.optim.Optimizer):
    """NOVAK (arXiv 2601.07876) over fp32 CUDA parameters.

    Every parameter of a group must be a contiguous float32 CUDA tensor and must
    have a gradient (float32 or bfloat16, one dtype per group) when ``step`` is
    called.  ``lr`` and ``weight_decay`` of a group may be changed between steps
    (learning-rate schedulers); the other entries are fixed once the group has
    taken its first step.  With ``graph_capturable=True`` the step counter and the
    per-step scalars live on the device, so that ``step()`` may be captured into a
    CUDA graph (``torch.cuda.graph``) after one eager step and replayed.
    """

    def __init__(self, params, lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
                 nesterov="approximation", lookahead_k=5, lookahead_alpha=0.5, *,
                 nesterov_beta=None, lookahead_mode="last", rectified=True, clip_threshold=0.0,
                 centralize=False, adaptive_beta=False, layer_adaptation=False,
                 sparse_threshold=0.0, auto_lr=False, true_nesterov_steps=0, moment_dtype="f32",
                 graph_capturable=False):
        defaults = dict(lr=lr, betas=betas, eps=eps, weight_decay=weight_decay, nesterov=nesterov,
                        lookahead_k=lookahead_k, lookahead_alpha=lookahead_alpha,
                        nesterov_beta=nesterov_beta, lookahead_mode=lookahead_mode,
                        rectified=rectified, clip_threshold=clip_threshold, centralize=centralize,
                        adaptive_beta=adaptive_beta, layer_adaptation=layer_adaptation,
                        sparse_threshold=sparse_threshold, auto_lr=auto_lr,
                        true_nesterov_steps=true_nesterov_steps, moment_dtype=moment_dtype,
                        graph_capturable=graph_capturable)
        super().__init__(params, defaults)
        self._engines: list[B.NovakOptimizer | None] = [None] * len(self.param_groups)
        self._applied: list[tuple] = [()] * len(self.param_groups)
        self._grad_lists: list[tuple] = [(None, None)] * len(self.param_groups)

    # ---- one library handle per parameter group, made at the group's first step
    def _engine(self, gi: int) -> B.NovakOptimizer:
        eng = self._engines[gi]
        group = self.param_groups[gi]
        if eng is None:
            kw = {k: group[k] for k in _GROUP_KEYS}
            eng = B.NovakOptimizer(group["params"], **kw)
            self._engines[gi] = eng
            self._applied[gi] = (group["lr"], group["weight_decay"])
        elif self._applied[gi] != (group["lr"], group["weight_decay"]):
            eng.handle.set_option(B.NOVAK_OPT_LR, group["lr"])
            eng.handle.set_option(B.NOVAK_OPT_WEIGHT_DECAY, group["weight_decay"])
            self._applied[gi] = (group["lr"], group["weight_decay"])
        return eng

    def add_param_group(self, param_group):
        super().add_param_group(param_group)
        if hasattr(self, "_engines"):
            self._engines.append(None)
            self._applied.append(())
            self._grad_lists.append((None, None))

    def _grads(self, gi: int, eng: B.NovakOptimizer) -> B.GradList:
        """The group's gradients as a marshalled list, rebuilt only when a gradient
        tensor has moved (the caching allocator usually hands the same blocks back)."""
        grads = []
        for p in self.param_groups[gi]["params"]:
            if p.grad is None:
                raise RuntimeError("Novak.step: every parameter of a group needs a gradient "
                                   "(the group is updated by one fused multi-tensor kernel)")
            g = p.grad
            grads.append(g if g.is_contiguous() else g.contiguous())
        key = tuple((g.data_ptr(), g.dtype) for g in grads)
        cached_key, cached = self._grad_lists[gi]
        if cached_key != key:
            cached = eng.prepare(grads)
            self._grad_lists[gi] = (key, cached)
        else:
            cached.tensors = grads            # keeps THIS step's tensors alive
        return cached

    @torch.no_grad()
    def step(self, closure=None):
        """One step of every group.  With a closure: groups that are in their
        true-Nesterov steps are moved to theta + beta_N m first (Eq. 10), the
        closure is evaluated there (Eq. 11) and the parameters are put back
        before the update; otherwise the closure is evaluated where the
        parameters are.  Returns the closure's loss."""
        engines = [self._engine(gi) for gi in range(len(self.param_groups))]
        loss = None
        if closure is not None:
            ahead = [e for e in engines if e.wants_extrapolation()]
            for e in ahead:
                e.extrapolate()
            try:
                with torch.enable_grad():
                    loss = closure()
            except BaseException:
                for e in ahead:
                    e.restore()          # the step is abandoned: put theta_{t-1} back
                raise
        for gi, e in enumerate(engines):
            e.step(self._grads(gi, e))
        return loss

    # ---- checkpoints: the library's own records, one per group
    def state_dict(self):
        groups = [{k: v for k, v in g.items() if k != "params"} for g in self.param_groups]
        return {"param_groups": groups,
                "engines": [e.state_dict() if e is not None else None for e in self._engines]}

    def load_state_dict(self, state_dict):
        if len(state_dict["engines"]) != len(self.param_groups):
            raise ValueError("checkpoint has another number of parameter groups")
        for g, saved in zip(self.param_groups, state_dict["param_groups"]):
            g.update(saved)
        for gi, sd in enumerate(state_dict["engines"]):
            self._engines[gi] = None
            if sd is not None:
                self._engine(gi).load_state_dict(sd)
