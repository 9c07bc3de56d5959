"""torch.optim front end of the EFCP / Sparse M-FAC step (argument marshalling only).

Every arithmetic step - error feedback, Top-k, the window, the preconditioned direction
and the parameter update theta <- (1 - gamma eta) theta - eta s u (Algorithm 1 with the
decoupled weight decay of Section 2 and the optional norm clipping of the hyper-parameter
appendix) - runs in the CUDA library behind `binding`.  This class only lays the
parameters out as one flat fp32 vector (the optimizer treats the model as a single
vector in R^d), copies the gradients into a flat buffer and forwards the scalars.
"""
from typing import Optional

import torch

from . import binding


class SparseMFAC(torch.optim.Optimizer):
    """Sparse M-FAC with error feedback.

    lr, weight_decay : eta and gamma, per parameter group (a group is one contiguous range
                       of the flat vector; e.g. gamma = 0 for normalisation parameters).
    m, density, damp : window length, k / d and the dampening lambda (the paper's
                       "universal" setting is m = 1024, density = 0.01).
    clip_norm        : clip |u|_2 to this constant (0 = off).
    block            : block-wise Top-k with this block length (0 = global Top-k).
    flags            : binding.RHS_ACCUMULATOR / binding.VALUES_BF16.
    """

    def __init__(self, params, lr: float, m: int = 1024, density: float = 0.01,
                 damp: float = 1e-6, weight_decay: float = 0.0, clip_norm: float = 0.0,
                 k: Optional[int] = None, block: int = 0, flags: int = 0):
        if lr < 0 or weight_decay < 0 or clip_norm < 0:
            raise ValueError("lr, weight_decay and clip_norm must be non-negative")
        super().__init__(params, dict(lr=lr, weight_decay=weight_decay))
        plist = [p for g in self.param_groups for p in g["params"]]
        if not plist:
            raise ValueError("no parameters")
        dev = plist[0].device
        for p in plist:
            if p.device != dev or not p.is_cuda or p.dtype != torch.float32:
                raise ValueError("all parameters must be fp32 tensors on one CUDA device")
        self._d = sum(p.numel() for p in plist)
        self._clip = float(clip_norm)
        self._theta = torch.empty(self._d, dtype=torch.float32, device=dev)
        self._g = torch.zeros(self._d, dtype=torch.float32, device=dev)
        self._u = torch.empty(self._d, dtype=torch.float32, device=dev)
        # parameters become views of the flat vector, group after group
        self._ranges = []
        off = 0
        with torch.no_grad():
            for g in self.param_groups:
                start = off
                for p in g["params"]:
                    n = p.numel()
                    self._theta[off:off + n].copy_(p.reshape(-1))
                    p.data = self._theta[off:off + n].view(p.shape)
                    off += n
                self._ranges.append((start, off))
        kk = int(k) if k is not None else max(1, int(round(density * self._d)))
        with torch.cuda.device(dev):
            self._h = binding.Efcp(self._d, m, kk, damp, flags, block)

    @property
    def handle(self) -> "binding.Efcp":
        """The library handle (diagnostics: error_norm, status, state_export, ...)."""
        return self._h

    @property
    def last_update(self) -> torch.Tensor:
        """u_t of the last step (flat, device); not written when there is one parameter group
        and no clipping (the update is then applied without materialising u)."""
        return self._u

    @torch.no_grad()
    def step(self, closure=None):
        loss = None
        if closure is not None:
            with torch.enable_grad():
                loss = closure()
        off = 0
        for g in self.param_groups:
            for p in g["params"]:
                n = p.numel()
                if p.grad is None:
                    self._g[off:off + n].zero_()
                else:
                    self._g[off:off + n].copy_(p.grad.reshape(-1))
                off += n
        groups = self.param_groups
        if len(groups) == 1:
            # without clipping nobody needs u: the library applies it to theta as it forms
            self._h.step_apply(self._g, self._theta, self._u if self._clip > 0 else None,
                               float(groups[0]["lr"]), float(groups[0]["weight_decay"]),
                               self._clip)
        else:
            self._h.step(self._g, self._u)
            if self._clip > 0:
                self._h.update_norm(self._u, sync=False)
            for g, (a, b) in zip(groups, self._ranges):
                if b > a:
                    self._h.apply_update(self._theta[a:b], self._u[a:b], float(g["lr"]),
                                         float(g["weight_decay"]), self._clip)
        return loss
