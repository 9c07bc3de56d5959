"""CPU oracle of Sparse GGT (test infrastructure only).

Follows the appendix "Sparse GGT", algorithm "Detailed Sparse GGT Implementation", step by
step in fp64 numpy: the compressed accumulator c_t = (V_t, I_t) of the error-feedback loop
(Algorithm 1; taken from the C++ oracle, whose error buffer, Top-k and ring buffer are the
same for every preconditioner) is written into row i of the window, delta = G x with
x = a_t[I_t] densified overwrites row and column i of the m x m matrix of scalar products,
that matrix is eigendecomposed, U_m = G^T V Sigma^+ is formed explicitly (d x rank, dense:
slow, small cases only) and

    u_t = x / eps + U_m [ (Sigma_m + eps I)^-1 - I / eps ] U_m^T x.

Readings.  The listing calls the eigenvalues of the scalar-product matrix Sigma_m^2 and
multiplies by "V sqrt(Sigma_m)^dagger": Sigma_m are the singular values of the window (square
roots of those eigenvalues) and the dagger is the pseudo-inverse, so that U_m has orthonormal
columns; components whose eigenvalue is at most m * 2^-48 times the largest are treated as
zero (empty rows of a window that is not full yet, linearly dependent rows).  Here G has one
gradient per row (m x d); the scalar-product matrix is G G^T.

Pinned in tests/test_oracle_pins.py by the definition u = ((sum_i c_i c_i^T)^(1/2) + eps I)^-1 x
evaluated with a dense d x d eigendecomposition, and by closed forms.
"""
import numpy as np

from . import ref


def rank_tolerance(m: int) -> float:
    """Eigenvalues of the scalar-product matrix below this fraction of the largest are zero."""
    return m * 2.0 ** -48


class RefSparseGGT:
    def __init__(self, d, m, k, eps, flags=0, block=0):
        # the dampening of the M-FAC oracle plays no part in the state that is used here
        self._ef = ref.RefEFCP(d, m, k, 1.0, flags, block)
        self.d, self.m, self.k, self.eps = int(d), int(m), self._ef.k, float(np.float32(eps))
        self.G = np.zeros((self.m, self.d))       # the window, one densified row per slot
        self.S = np.zeros((self.m, self.m))       # scalar products of the rows
        self.t = 0
        self.sigma = np.zeros(self.m)

    def close(self):
        self._ef.close()

    def error(self):
        return self._ef.error()

    def row(self, slot):
        return self._ef.row(slot)

    @property
    def step_count(self):
        return self.t

    def step(self, grad: np.ndarray) -> np.ndarray:
        self._ef.step(grad)                        # a = xi + g, c = Top-k(a), xi = a - c
        i = self.t % self.m
        self.t += 1
        idx, val = self._ef.row(i)
        x = np.zeros(self.d)
        x[idx] = val.astype(np.float64)            # a_t[I_t], densified
        self.G[i] = x                              # integrate values and indices
        delta = self.G @ x                         # scalar products with every row
        self.S[i, :] = delta
        self.S[:, i] = delta
        lam, V = np.linalg.eigh(self.S)            # S = V diag(lam) V^T
        lam = np.maximum(lam, 0.0)
        keep = lam > rank_tolerance(self.m) * lam.max() if lam.max() > 0 else np.zeros(self.m, bool)
        sig = np.sqrt(lam[keep])
        self.sigma = np.sqrt(lam)
        U = (self.G.T @ V[:, keep]) / sig          # U_m = G^T V Sigma^+, orthonormal columns
        coef = 1.0 / (sig + self.eps) - 1.0 / self.eps
        u = x / self.eps + U @ (coef * (U.T @ x))
        return u.astype(np.float32)
