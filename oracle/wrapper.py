"""CPU oracle of the parameter update around the preconditioner (test infrastructure only).

Plain numpy in fp64, written from the formulas:
  * Algorithm 1, last line of the loop:        theta_t = theta_{t-1} - eta_t u_t
  * Section 2 (interaction with regularisation): decoupled weight decay,
        theta_{t+1} = (1 - gamma eta_t) theta_t - eta_t u_t
  * hyper-parameter appendix: the norm of the preconditioned gradient u_t is clipped to a
    constant c, i.e. u_t is scaled by min(1, c / |u_t|_2)
  * Section 4 ("Error Feedback Evolution During Training"): |xi_t|_2 / (|g_1|_2 + ... + |g_t|_2)

Pinned by tests/test_oracle_pins.py (closed forms, an element-by-element loop, the
equivalence with gradient descent on the L2-regularised quadratic when the preconditioner
is the identity).  Nothing here is shared with the CUDA path.
"""
import numpy as np


def update_norm(u) -> float:
    """|u|_2 in fp64."""
    u = np.asarray(u, np.float64)
    return float(np.sqrt(np.sum(u * u)))


def clip_scale(u, clip_norm: float) -> float:
    """min(1, c / |u|_2); 1 when clipping is off (c = 0) or u = 0."""
    if clip_norm <= 0.0:
        return 1.0
    nrm = update_norm(u)
    if nrm == 0.0:
        return 1.0
    return min(1.0, float(clip_norm) / nrm)


def apply_update(theta, u, eta: float, gamma: float = 0.0, clip_norm: float = 0.0, scale=None):
    """theta <- (1 - gamma eta) theta - eta s u in fp64 (s = clip_scale(u) unless given, for
    a sub-range of a clipped update).  Returns fp64; the caller rounds."""
    theta = np.asarray(theta, np.float64)
    u64 = np.asarray(u, np.float64)
    s = clip_scale(u64, clip_norm) if scale is None else float(scale)
    eta = float(np.float32(eta))      # the interface takes fp32 scalars
    gamma = float(np.float32(gamma))
    return (1.0 - gamma * eta) * theta - eta * s * u64


def ef_evolution(error_norms, grad_norms):
    """|xi_t| / (|g_1| + ... + |g_t|) for t = 1..T."""
    e = np.asarray(error_norms, np.float64)
    g = np.cumsum(np.asarray(grad_norms, np.float64))
    return e / g
