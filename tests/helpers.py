"""Independent numpy restatements used to pin the CPU oracle (and nothing else).

Everything here is written from the formulas, in dense fp64 algebra, without
calling the oracle: a mistake in the oracle's sparse / Woodbury / Cholesky code
cannot hide behind a shared helper.
"""
import numpy as np


def mag_key(a: np.ndarray) -> np.ndarray:
    return a.astype(np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


def topk_by_sort(a: np.ndarray, k: int):
    """First k of a sort by (|a| bit pattern descending, index ascending), index-ascending."""
    key = mag_key(a).astype(np.int64)
    order = np.lexsort((np.arange(a.size), -key))  # last key is primary
    sel = np.sort(order[:k])
    return sel.astype(np.int32), a[sel].astype(np.float32)


class DenseSim:
    """EFCP with a dense m x d window and a brute-force d x d solve (tiny sizes only)."""

    def __init__(self, d, m, k, lam, rhs_accumulator=False, values_bf16=False):
        self.bf16 = values_bf16
        self.d, self.m, self.k = d, m, k
        self.lam = float(np.float32(lam))
        self.acc_mode = rhs_accumulator
        self.e = np.zeros(d, np.float32)
        self.G = np.zeros((m, d), np.float64)
        self.t = 0

    def step(self, g):
        g = g.astype(np.float32)
        a = (self.e + g).astype(np.float32)
        idx, val = topk_by_sort(a, self.k)
        if self.bf16:  # library conversion, not the oracle's bit manipulation
            import torch
            val = torch.from_numpy(val).to(torch.bfloat16).to(torch.float32).numpy()
        c = np.zeros(self.d, np.float32)
        c[idx] = val
        e_new = a.copy()
        e_new[idx] = a[idx] - val
        self.e = e_new
        self.G[self.t % self.m] = c.astype(np.float64)
        self.t += 1
        x = (a if self.acc_mode else c).astype(np.float64)
        F = self.lam * np.eye(self.d) + (self.G.T @ self.G) / self.m
        u = np.linalg.solve(F, x)
        self.last = dict(a=a, idx=idx, val=val, x=x, F=F)
        return u
