"""torch.optim front end of the Muon step: argument marshalling only.

Every 2-D parameter handed to `Muon` is updated by one call of muon_step_batched per `step()`;
the arithmetic (momentum, Newton-Schulz, update) runs entirely in the CUDA library.  Parameters
that are not matrices belong to another optimizer (the paper delegates them to AdamW).
"""
from __future__ import annotations

from typing import Iterable, Sequence

import torch

from . import binding as mb
from .workloads import NS_STEPS, QUINTIC


class Muon(torch.optim.Optimizer):
    """Muon for 2-D fp32 CUDA parameters whose gradients are fp32 or bf16 (all of one kind).

    lr, momentum (mu), weight_decay (decoupled), ns_steps and coeffs have the meaning of
    muon_step_batched; `nesterov`, `eps` and `ns_precision` are fixed at construction because they
    are options of the library context.
    """

    def __init__(self, params: Iterable[torch.nn.Parameter], lr: float = 3e-5, momentum: float = 0.95,
                 weight_decay: float = 0.0, nesterov: bool = True, ns_steps: int = NS_STEPS,
                 coeffs: Sequence[float] = QUINTIC, eps: float = 1e-7, grad_dtype: torch.dtype = torch.float32,
                 ns_precision: str = "bf16"):
        params = list(params)
        for p in params:
            if p.dim() != 2 or p.dtype != torch.float32 or not p.is_cuda or not p.is_contiguous():
                raise ValueError("Muon takes contiguous 2-D fp32 CUDA parameters; give the others to another optimizer")
        if grad_dtype not in (torch.float32, torch.bfloat16):
            raise ValueError("gradients must be fp32 or bf16")
        super().__init__(params, dict(lr=lr, momentum=momentum, weight_decay=weight_decay))
        self._ns_steps, self._coeffs, self._grad_dtype = ns_steps, tuple(coeffs), grad_dtype
        opt = mb.muon_default_options(nesterov=1 if nesterov else 0, eps=eps,
                                      grad_dtype=mb.DTYPE_FP32 if grad_dtype == torch.float32 else mb.DTYPE_BF16,
                                      ns_precision=mb.NS_BF16 if ns_precision == "bf16" else mb.NS_FP32,
                                      coeffs_per_step=1 if len(self._coeffs) == 3 * ns_steps and ns_steps > 1 else 0)
        self._ctx = mb.Context(opt)

    @torch.no_grad()
    def step(self, closure=None):
        loss = None
        if closure is not None:
            with torch.enable_grad():
                loss = closure()
        for group in self.param_groups:
            ps = [p for p in group["params"] if p.grad is not None]
            if not ps:
                continue
            grads = []
            for p in ps:
                g = p.grad
                if g.dtype != self._grad_dtype or not g.is_contiguous():
                    g = g.to(self._grad_dtype).contiguous()     # a cast of the input, not part of the method
                grads.append(g)
            moms = []
            for p in ps:
                st = self.state[p]
                if "momentum_buffer" not in st:
                    st["momentum_buffer"] = torch.zeros_like(p)
                moms.append(st["momentum_buffer"])
            shapes = [tuple(p.shape) for p in ps]
            self._ctx.ensure_workspace(shapes)
            self._ctx.muon_step_batched([p.data for p in ps], grads, moms, shapes, group["lr"], group["momentum"],
                                        group["weight_decay"], self._ns_steps, self._coeffs)
        return loss
