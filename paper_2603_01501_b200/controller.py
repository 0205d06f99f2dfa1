"""Algorithm 1 around an optimizer, for callers that hold ``torch`` parameters.

A convenience layer over the binding: it owns the stored direction (one
snapshot of the previous aggregated gradient, App. A.2), counts Algorithm 1's
step t, and tells the caller whether to take the optimizer step.  All
arithmetic is in the CUDA library; nothing here touches gradient values.

    ctl = GradientAlignmentController(model.parameters())
    loss.backward()
    if ctl.step():            # False on a violation step: skip the update
        optimizer.step()
"""
from __future__ import annotations

from typing import Iterable, List, Optional

import torch

from . import binding as gb


class GradientAlignmentController:
    def __init__(self, params: Iterable[torch.nn.Parameter], hp: Optional[gb.HParams] = None,
                 snapshot_dtype: Optional[torch.dtype] = None):
        """`params`: the trainable parameters whose ``.grad`` tensors form the flattened
        gradient.  `snapshot_dtype`: float32 (default) or bfloat16 when the gradients are
        bfloat16.  Gradients must exist (one backward pass) before the first ``step``."""
        self.params: List[torch.nn.Parameter] = [p for p in params if p.requires_grad]
        if not self.params:
            raise ValueError("no trainable parameters")
        self.hp = hp or gb.HParams()
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
        return self.last.regime != gb.GAC_REGIME_VIOLATION and not self.last.nonfinite

    def state_dict(self) -> dict:
        return {"t": self.t, "snapshot": [s.clone() for s in self.snapshot]}

    def load_state_dict(self, state: dict) -> None:
        """Resumes: the snapshot becomes the stored direction of the next step."""
        self.t = int(state["t"])
        grads = self._grads()
        self._bind(grads)
        for dst, src in zip(self.snapshot, state["snapshot"]):
            dst.copy_(src)

    def close(self) -> None:
        if self.ctx is not None:
            gb.gac_free(self.ctx)
            self.ctx = None
