"""Sparse GGT mode (EFCP_PRECOND_GGT) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ggt

pytestmark = pytest.mark.gpu

U_TOL = 1e-4  # relative L2 on the update, as for the M-FAC mode


def _binding():
    from paper_2306_06098_b200 import binding
    return binding


def bits(a):
    return np.ascontiguousarray(a).view(np.uint32)


def rel_l2(a, b):
    b = b.astype(np.float64)
    return np.linalg.norm(a.astype(np.float64) - b) / max(np.linalg.norm(b), 1e-300)


def run_ggt(d, m, k, eps, grads, flags=0, block=0):
    B = _binding()
    gpu = B.Efcp(d, m, k, eps, flags | B.PRECOND_GGT, block)
    cpu = ggt.RefSparseGGT(d, m, k, eps, flags, block)
    assert gpu.k == cpu.k
    g_dev = torch.empty(d, device="cuda")
    u_dev = torch.empty(d, device="cuda")
    worst = 0.0
    for t, g in enumerate(grads):
        g = np.ascontiguousarray(g, np.float32)
        g_dev.copy_(torch.from_numpy(g))
        u_dev.fill_(float("nan"))
        gpu.step(g_dev, u_dev)
        u_ref = cpu.step(g)
        assert gpu.status() == 0, (t, gpu.status())
        assert np.array_equal(bits(gpu.error()), bits(cpu.error())), t
        gi, gv = gpu.row(t % m)
        ci, cv = cpu.row(t % m)
        assert np.array_equal(gi, ci) and np.array_equal(bits(gv), bits(cv)), t
        u = u_dev.cpu().numpy()
        assert np.isfinite(u).all()
        err = rel_l2(u, u_ref)
        worst = max(worst, err)
        assert err <= U_TOL, f"update rel-L2 {err:.3e} at step {t}"
        assert gpu.last_residual() <= 1e-13  # off-diagonal norm the eigendecomposition reached
        # the scalar products are those of the oracle's window
        Sg = gpu.gram()
        assert np.allclose(Sg, cpu.S, rtol=1e-12, atol=1e-12 * np.abs(cpu.S).max())
    assert gpu.validate() == 0
    print(f"ggt parity d={d} m={m} k={k}: worst update rel-L2 {worst:.3e}")
    gpu.close()
    cpu.close()
    return worst


@pytest.mark.parametrize("d,m,k,eps,steps", [
    (5_000, 1, 50, 0.1, 3),          # one row: u = x / (|x| + eps)
    (20_000, 7, 200, 0.05, 20),      # odd m (padded pairing), the window wraps twice
    (100_003, 32, 1000, 0.01, 40),   # several slabs, ragged tail
    (272_474, 100, 2725, 0.01, 12),  # the paper's GGT setting: ResNet-20 size, m = 100, 1 %
    (50_000, 160, 500, 0.02, 6),     # the largest window the mode takes
    (30_000, 113, 300, 0.02, 4),     # odd m above 112
])
def test_ggt_parity(d, m, k, eps, steps):
    rng = np.random.default_rng(d + m)
    scale = np.exp(0.5 * rng.standard_normal(d))
    grads = ((scale * rng.standard_normal(d)).astype(np.float32) for _ in range(steps))
    run_ggt(d, m, k, eps, grads)


def test_ggt_with_blockwise_topk_and_bf16_values():
    B = _binding()
    d, m, k = 60_000, 16, 600
    rng = np.random.default_rng(9)
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(10)]
    run_ggt(d, m, k, 0.05, grads, block=2048)
    run_ggt(d, m, k, 0.05, grads, flags=B.VALUES_BF16)


def test_ggt_rank_deficient_window():
    # the same gradient pattern twice: the kept entries repeat, the rows are dependent
    d, m, k = 4_000, 6, 40
    rng = np.random.default_rng(10)
    g = np.zeros(d, np.float32)
    g[:k] = 1.0 + rng.random(k).astype(np.float32)
    grads = [g, g, (0.5 * g).astype(np.float32), rng.standard_normal(d).astype(np.float32), g]
    run_ggt(d, m, k, 0.1, grads)


def test_ggt_argument_errors():
    B = _binding()
    for args in ((1000, 161, 10, 0.1, B.PRECOND_GGT),
                 (1000, 8, 10, 0.1, B.PRECOND_GGT | B.RHS_ACCUMULATOR),
                 (1000, 8, 10, 0.0, B.PRECOND_GGT)):
        with pytest.raises(B.EfcpError) as ei:
            B.Efcp(*args)
        assert ei.value.code == B.EINVAL
