"""Algorithm 1 around an optimizer, for callers that hold ``torch`` parameters.

A convenience layer over the binding: it owns the stored direction (one
snapshot of the previous aggregated gradient, App. A.2), counts Algorithm 1's
step t, and tells the caller whether to take the optimizer step.  All
arithmetic is in the CUDA library; nothing here touches gradient values.

    ctl = GradientAlignmentController(model.parameters())
    loss.backward()
    if ctl.step():            # False on a violation step: skip the update
        optimizer.step()

With ``exchange=True`` the snapshot is never copied: the tensors that hold the
gradient become the stored direction and each parameter's ``.grad`` is pointed
at the other tensor of its pair (which then holds the projected gradient, when
the step projected).  The loop must then ask the controller for the next
gradient tensors instead of the optimizer:

    ctl.zero_grad()           # not optimizer.zero_grad(): .grad moves to the free tensors
    loss.backward()
    if ctl.step():
        optimizer.step()      # reads .grad, must not modify it
"""
from __future__ import annotations

import dataclasses
from typing import Iterable, List, Optional

import torch

from . import binding as gb


class GradientAlignmentController:
    def __init__(self, params: Iterable[torch.nn.Parameter], hp: Optional[gb.HParams] = None,
                 snapshot_dtype: Optional[torch.dtype] = None, exchange: bool = False):
        """`params`: the trainable parameters whose ``.grad`` tensors form the flattened
        gradient.  `snapshot_dtype`: float32 (default) or bfloat16 when the gradients are
        bfloat16.  `exchange`: refresh the snapshot by swapping tensors instead of copying
        (the snapshot then has the gradients' element type).  Gradients must exist (one
        backward pass) before the first ``step``."""
        self.params: List[torch.nn.Parameter] = [p for p in params if p.requires_grad]
        if not self.params:
            raise ValueError("no trainable parameters")
        self.hp = hp or gb.HParams()
        self.exchange = bool(exchange)
        if self.exchange:
            self.hp = dataclasses.replace(self.hp, state_mode=gb.GAC_STATE_EXCHANGE)
        self.sets: List[List[torch.Tensor]] = []     # exchange mode: the two tensors of every parameter
        self.snapshot_dtype = snapshot_dtype or torch.float32
        self.t = 0
        self.ctx: Optional[gb.GacContext] = None
        self.snapshot: List[torch.Tensor] = []
        self._bound_ptrs: List[int] = []
        self.last: Optional[gb.gac_result] = None

    def _grads(self) -> List[torch.Tensor]:
        gs = []
        for p in self.params:
            if p.grad is None:
                raise RuntimeError("a parameter has no gradient: call backward() before step()")
            if not p.grad.is_contiguous():
                raise RuntimeError("gradients must be contiguous")
            gs.append(p.grad.view(-1))
        return gs

    def _bind(self, grads: List[torch.Tensor]) -> None:
        ptrs = [g.data_ptr() for g in grads]
        if self.exchange:
            if self.ctx is None:
                other = [torch.empty_like(g) for g in grads]
                self.sets = [grads, other]
                self.ctx = gb.gac_init(grads, other, self.hp)
            elif ptrs != [g.data_ptr() for g in self.sets[gb.gac_next_gradient_set(self.ctx)]]:
                raise RuntimeError("exchange mode: the gradient must be accumulated into the tensors the "
                                   "controller hands out -- call ctl.zero_grad() before backward()")
            return
        if self.ctx is None:
            self.snapshot = [torch.empty(g.numel(), dtype=self.snapshot_dtype, device=g.device) for g in grads]
            self.ctx = gb.gac_init(grads, self.snapshot, self.hp)
        elif ptrs != self._bound_ptrs:          # the framework re-allocated some .grad tensors
            gb.gac_rebind(self.ctx, grads, self.snapshot)
        self._bound_ptrs = ptrs

    def step(self, staleness: int = 0) -> bool:
        """Runs the two passes on the current gradients (in place) and returns True when
        the optimizer step should be taken (safe or projection), False on a violation
        or when a non-finite gradient was met."""
        grads = self._grads()
        self._bind(grads)
        self.t += 1
        self.last = gb.gac_stats(self.ctx, self.t, staleness=staleness)
        gb.gac_project(self.ctx)
        if self.exchange:
            # the tensors that held the gradient are the snapshot now; what the step sends on is
            # either still there (g unchanged: read it, do not modify it) or in the other tensors
            self.snapshot = self.sets[self.last.g_set]
            out = self.sets[self.last.out_set]
            for p, o in zip(self.params, out):
                p.grad = o.view_as(p)
        return self.last.regime != gb.GAC_REGIME_VIOLATION and not self.last.nonfinite

    def zero_grad(self) -> None:
        """Exchange mode: points every ``.grad`` at the tensor that is free for the next
        gradient and clears it.  Without exchange it clears the gradients in place."""
        if self.exchange and self.ctx is not None:
            nxt = self.sets[gb.gac_next_gradient_set(self.ctx)]
            for p, g in zip(self.params, nxt):
                p.grad = g.view_as(p)
        for p in self.params:
            if p.grad is not None:
                p.grad.zero_()

    def state_dict(self) -> dict:
        return {"t": self.t, "snapshot": [s.clone() for s in self.snapshot]}

    def load_state_dict(self, state: dict) -> None:
        """Resumes: the snapshot becomes the stored direction of the next step."""
        self.t = int(state["t"])
        grads = self._grads()
        self._bind(grads)
        if self.exchange:
            self.snapshot = self.sets[gb.gac_next_gradient_set(self.ctx) ^ 1]
        for dst, src in zip(self.snapshot, state["snapshot"]):
            dst.copy_(src)

    def close(self) -> None:
        if self.ctx is not None:
            gb.gac_free(self.ctx)
            self.ctx = None
