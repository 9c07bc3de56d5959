"""Pins for the CPU oracle: every check compares it with something that is not the
oracle (brute-force dense algebra, closed forms, a literal sort, invariants)."""
import numpy as np
import pytest

from oracle import ref
from tests.helpers import DenseSim, mag_key, topk_by_sort


def rel(a, b):
    return np.linalg.norm(np.asarray(a, np.float64) - b) / max(np.linalg.norm(b), 1e-300)


# ----------------------------------------------------------------- Top-k (Section 3.1)
def _check_topk(a, k):
    a = np.asarray(a, np.float32)
    want_i, want_v = topk_by_sort(a, k)
    for full in (False, True):
        got_i, got_v = ref.topk(a, k, fullsort=full)
        assert np.array_equal(got_i, want_i)
        assert np.array_equal(got_v.view(np.uint32), want_v.view(np.uint32))


def test_topk_random():
    rng = np.random.default_rng(1)
    for d, k in ((1, 1), (7, 3), (1000, 10), (4097, 4097), (50_000, 500)):
        _check_topk(rng.standard_normal(d), k)


def test_topk_ties_go_to_lower_index():
    a = np.full(100, 2.5, np.float32)
    idx, _ = ref.topk(a, 7)
    assert idx.tolist() == list(range(7))
    # +v and -v have the same magnitude: order decided by index alone
    a = np.array([1.0, -3.0, 3.0, -3.0, 0.5, 3.0], np.float32)
    idx, val = ref.topk(a, 2)
    assert idx.tolist() == [1, 2] and val.tolist() == [-3.0, 3.0]
    idx, _ = ref.topk(a, 3)
    assert idx.tolist() == [1, 2, 3]
    rng = np.random.default_rng(2)
    _check_topk(rng.integers(-3, 4, 5000).astype(np.float32), 1234)


def test_topk_zero_denormal_inf_nan_order():
    tiny = np.float32(1e-45)  # smallest denormal
    a = np.array([0.0, -0.0, tiny, -tiny, 1.0, np.inf, -np.inf, np.nan], np.float32)
    # magnitude order by bit pattern: nan > inf > 1 > denormal > zero
    assert ref.topk(a, 1)[0].tolist() == [7]
    assert ref.topk(a, 3)[0].tolist() == [5, 6, 7]
    assert ref.topk(a, 4)[0].tolist() == [4, 5, 6, 7]
    assert ref.topk(a, 6)[0].tolist() == [2, 3, 4, 5, 6, 7]
    assert ref.topk(a, 7)[0].tolist() == [0, 2, 3, 4, 5, 6, 7]  # +0 and -0 tie: lower index
    _check_topk(a, 5)


def test_topk_rejects_bad_arguments():
    a = np.zeros(4, np.float32)
    with pytest.raises(ValueError):
        ref.topk(a, 5)
    with pytest.raises(ValueError):
        ref.topk(a, 0)


# ------------------------------------------- error feedback (Algorithm 1)
def test_error_feedback_invariant_bitwise():
    rng = np.random.default_rng(3)
    d, m, k = 3001, 4, 37
    o = ref.RefEFCP(d, m, k, 1e-3)
    e_prev = np.zeros(d, np.float32)
    for t in range(9):
        g = (rng.standard_normal(d) * np.exp(rng.standard_normal(d))).astype(np.float32)
        o.step(g)
        a = (e_prev + g).astype(np.float32)  # independent fp32 add
        assert np.array_equal(o.accumulator().view(np.uint32), a.view(np.uint32))
        idx, val = o.row(t % m)
        want_i, want_v = topk_by_sort(a, k)
        assert np.array_equal(idx, want_i) and np.array_equal(val.view(np.uint32), want_v.view(np.uint32))
        e = o.error()
        assert np.all(e[idx].view(np.uint32) == 0)  # literally +0.0f at kept coordinates
        dens = np.zeros(d, np.float32)
        dens[idx] = val
        assert np.array_equal((e + dens).view(np.uint32) & 0x7FFFFFFF, mag_key(a))
        mask = np.ones(d, bool)
        mask[idx] = False
        assert np.array_equal(e[mask].view(np.uint32), a[mask].view(np.uint32))
        e_prev = e
    assert o.step_count == 9


def test_k_equals_d_is_dense_mfac():
    rng = np.random.default_rng(4)
    d, m = 24, 5
    o = ref.RefEFCP(d, m, d, 0.05)
    G = np.zeros((m, d))
    for t in range(8):
        g = rng.standard_normal(d).astype(np.float32)
        u = o.step(g)
        assert not o.error().any()
        G[t % m] = g
        F = np.float32(0.05).astype(np.float64) * np.eye(d) + G.T @ G / m
        assert rel(u, np.linalg.solve(F, g.astype(np.float64))) < 1e-6


# --------------------------- inverse-Fisher-vector product (Section 2.1, Eq. 2) by brute force
@pytest.mark.parametrize("acc_mode", [False, True])
@pytest.mark.parametrize("d,m,k,steps,lam", [
    (64, 1, 9, 3, 1e-2), (96, 2, 17, 5, 1e-3), (128, 4, 13, 11, 1e-4),
    (256, 8, 40, 6, 1e-3),  # fewer steps than rows: unwritten rows are zero gradients
    (200, 8, 21, 20, 1e-2),  # wraps twice
])
def test_update_matches_dense_solve(d, m, k, steps, lam, acc_mode):
    rng = np.random.default_rng(d + m)
    flags = ref.RHS_ACCUMULATOR if acc_mode else ref.RHS_COMPRESSED
    o = ref.RefEFCP(d, m, k, lam, flags)
    sim = DenseSim(d, m, k, lam, rhs_accumulator=acc_mode)
    scale = np.exp(rng.standard_normal(d))
    for t in range(steps):
        g = (scale * rng.standard_normal(d)).astype(np.float32)
        u = o.step(g)
        want = sim.step(g)
        assert np.array_equal(o.error().view(np.uint32), sim.e.view(np.uint32))
        assert rel(u, want) < 2e-6, (t, rel(u, want))
        # residual of the defining linear system, in dense fp64
        # (u is rounded to fp32, so the bound is the rounding of u pushed through F)
        F, x = sim.last["F"], sim.last["x"]
        r = F @ u.astype(np.float64) - x
        bound = 2.0 ** -23 * np.linalg.norm(np.abs(F) @ np.abs(u.astype(np.float64)))
        assert np.linalg.norm(r) <= bound + 1e-6 * np.linalg.norm(x)
        if not acc_mode:
            assert rel(o.update_rowform(), want) < 2e-6
    assert np.allclose(o.gram(), o.gram_full(), rtol=1e-13, atol=0)
    assert np.allclose(o.gram(), sim.G @ sim.G.T, rtol=1e-12, atol=1e-12)


# ------------------------------------------- bfloat16 window values (Section 3.1, "Format for V")
def test_bf16_rounding_matches_library_conversion_and_ties_to_even():
    import torch
    rng = np.random.default_rng(30)
    x = np.concatenate([
        (rng.standard_normal(200_000) * np.exp(8 * rng.standard_normal(200_000))).astype(np.float32),
        rng.integers(0, 2 ** 32, 200_000, dtype=np.uint64).astype(np.uint32).view(np.float32),
        np.array([0.0, -0.0, 1.0, np.inf, -np.inf, 3.3895314e38, 1e-45, 1.17549435e-38], np.float32)])
    x = x[~np.isnan(x)]
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = ref.round_bf16(x)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # exact ties: 1 + 2^-8 lies halfway between 1 and 1 + 2^-7 -> even mantissa (1.0);
    # 1 + 3 * 2^-8 lies halfway between 1 + 2^-7 and 1 + 2^-6 -> 1 + 2^-6
    ties = np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -(1 + 2.0 ** -8)], np.float32)
    assert ref.round_bf16(ties).tolist() == [1.0, 1 + 2.0 ** -6, -1.0]
    assert np.isnan(ref.round_bf16(np.array([np.nan], np.float32))[0])
    # near the largest finite value rounding goes to infinity, as the format demands
    assert np.isinf(ref.round_bf16(np.array([3.4e38], np.float32))[0])


def test_bf16_values_feed_the_rounding_residue_back():
    rng = np.random.default_rng(31)
    d, m, k = 2001, 4, 55
    o = ref.RefEFCP(d, m, k, 1e-3, ref.VALUES_BF16)
    e_prev = np.zeros(d, np.float32)
    for t in range(7):
        g = (rng.standard_normal(d) * np.exp(rng.standard_normal(d))).astype(np.float32)
        o.step(g)
        a = (e_prev + g).astype(np.float32)
        idx, val = o.row(t % m)
        want_i, want_v = topk_by_sort(a, k)       # selection is by the unrounded magnitude
        assert np.array_equal(idx, want_i)
        assert np.all((val.view(np.uint32) & 0xFFFF) == 0)          # representable in bfloat16
        assert np.all(np.abs(val - want_v) <= np.abs(want_v) * 2.0 ** -8)
        e = o.error()
        dens = np.zeros(d, np.float32)
        dens[idx] = val
        assert np.array_equal((e + dens).view(np.uint32), a.view(np.uint32))  # a = xi + c, exactly
        e_prev = e


@pytest.mark.parametrize("d,m,k,steps,lam", [(96, 2, 17, 5, 1e-3), (200, 8, 21, 20, 1e-2)])
def test_bf16_update_matches_dense_solve(d, m, k, steps, lam):
    rng = np.random.default_rng(d)
    o = ref.RefEFCP(d, m, k, lam, ref.VALUES_BF16)
    sim = DenseSim(d, m, k, lam, values_bf16=True)
    scale = np.exp(rng.standard_normal(d))
    for t in range(steps):
        g = (scale * rng.standard_normal(d)).astype(np.float32)
        u = o.step(g)
        want = sim.step(g)
        assert np.array_equal(o.error().view(np.uint32), sim.e.view(np.uint32))
        assert rel(u, want) < 2e-6, (t, rel(u, want))
        assert rel(o.update_rowform(), want) < 2e-6


# ------------------------------------------- block-wise Top-k (Section 3.1, "Sparsity Pattern")
def test_blockwise_topk_keeps_the_stated_count_in_every_block():
    rng = np.random.default_rng(33)
    d, m, k, block = 10_007, 3, 100, 1000      # 1 % -> ceil(1000/100) = 10 per full block
    o = ref.RefEFCP(d, m, k, 1e-3, block=block)
    assert o.k == 10 * 10 + 1                   # ten full blocks, ceil(7 * 100 / 10007) = 1
    e_prev = np.zeros(d, np.float32)
    for t in range(5):
        g = (rng.standard_normal(d) * np.exp(rng.standard_normal(d))).astype(np.float32)
        o.step(g)
        a = (e_prev + g).astype(np.float32)
        idx, val = o.row(t % m)
        assert np.all(np.diff(idx) > 0)
        want_i, want_v = [], []
        for b0 in range(0, d, block):
            blk = a[b0:b0 + block]
            c = -(-blk.size * k // d)
            bi, bv = topk_by_sort(blk, c)       # the definition, block by block
            want_i.append(bi + b0)
            want_v.append(bv)
        assert np.array_equal(idx, np.concatenate(want_i))
        assert np.array_equal(val.view(np.uint32), np.concatenate(want_v).view(np.uint32))
        e = o.error()
        assert not e[idx].any()
        e_prev = e


def test_blockwise_with_one_block_is_global_topk():
    rng = np.random.default_rng(34)
    d, m, k = 3000, 2, 77
    a = ref.RefEFCP(d, m, k, 1e-2)
    b = ref.RefEFCP(d, m, k, 1e-2, block=d)
    assert b.k == k
    for _ in range(4):
        g = rng.standard_normal(d).astype(np.float32)
        ua, ub = a.step(g), b.step(g)
        assert np.array_equal(ua.view(np.uint32), ub.view(np.uint32))


def test_m1_closed_form():
    # m = 1: F^-1 x = x/lam - g (g.x) / (lam (m lam + g.g))
    rng = np.random.default_rng(5)
    d, k, lam = 50, 6, np.float32(0.3)
    g = rng.standard_normal(d).astype(np.float32)
    o = ref.RefEFCP(d, 1, k, lam)
    u = o.step(g)
    idx, val = topk_by_sort(g, k)
    c = np.zeros(d)
    c[idx] = val
    L = float(lam)
    want = c / L - c * (c @ c) / (L * (L + c @ c))
    assert rel(u, want) < 1e-6


def test_disjoint_supports_closed_form():
    # rows with disjoint supports: S diagonal, coef_j = p_j / (lam (m lam + |g_j|^2))
    m, lam = 6, 1e-2
    n2 = np.array([3.0, 0.5, 7.0, 0.0, 2.0, 11.0])
    p = np.array([1.0, -2.0, 0.3, 0.0, 5.0, -1.0])
    want = p / (lam * (m * lam + n2))
    assert np.allclose(ref.woodbury_coef(np.diag(n2), p, lam), want, rtol=1e-13)
    assert np.allclose(ref.wsm_coef(np.diag(n2), p, lam), want, rtol=1e-12)


def test_large_lambda_limit_is_scaled_identity():
    rng = np.random.default_rng(6)
    d, m, k, lam = 300, 4, 30, np.float32(1e8)
    o = ref.RefEFCP(d, m, k, lam)
    for _ in range(6):
        g = rng.standard_normal(d).astype(np.float32)
        u = o.step(g)
    idx, val = o.row(5 % m)
    x = np.zeros(d)
    x[idx] = val
    assert rel(u, x / float(lam)) < 1e-6


def test_wsm_recursion_equals_woodbury_and_dense_recursion():
    rng = np.random.default_rng(7)
    for m, d, lam in ((1, 5, 0.1), (3, 10, 1e-2), (16, 40, 1e-3), (48, 64, 1e-4)):
        G = rng.standard_normal((m, d))
        x = rng.standard_normal(d)
        S, p = G @ G.T, G @ x
        c1 = ref.woodbury_coef(S, p, lam)
        c2 = ref.wsm_coef(S, p, lam)
        assert rel(c2, c1) < 1e-8
        # literal dense rank-one recursion, F_0 = lam I, F_j = F_{j-1} + g_j g_j^T / m
        Finv = np.eye(d) / lam
        for j in range(m):
            v = Finv @ G[j]
            Finv = Finv - np.outer(v, v) / (m + G[j] @ v)
        want = Finv @ x
        for c in (c1, c2):
            assert rel(x / lam - G.T @ c, want) < 1e-7


def test_planted_mistakes_are_caught():
    # dropping the 1/m factor, or using lam instead of m*lam on the diagonal, must
    # disagree with the dense definition by far more than the pin tolerance.
    rng = np.random.default_rng(8)
    m, d, lam = 4, 20, 1e-2
    G = rng.standard_normal((m, d))
    x = rng.standard_normal(d)
    S, p = G @ G.T, G @ x
    want = np.linalg.solve(lam * np.eye(d) + G.T @ G / m, x)
    good = x / lam - G.T @ ref.woodbury_coef(S, p, lam)
    assert rel(good, want) < 1e-9
    bad1 = x / lam - G.T @ (np.linalg.solve(lam * np.eye(m) + S, p) / lam)
    assert rel(bad1, want) > 1e-3


def test_oracle_rejects_bad_arguments():
    for args in ((0, 1, 1, 1e-3), (4, 0, 1, 1e-3), (4, 1, 0, 1e-3), (4, 1, 5, 1e-3),
                 (4, 1, 1, 0.0), (4, 1, 1, float("nan")), (2**31, 1, 1, 1e-3)):
        with pytest.raises(ValueError):
            ref.RefEFCP(*args)


def test_thread_count_does_not_change_results():
    import os
    import subprocess
    import sys
    code = (
        "import numpy as np, sys; sys.path.insert(0, %r)\n"
        "from oracle import ref\n"
        "rng=np.random.default_rng(0); o=ref.RefEFCP(5000,64,50,1e-4)\n"
        "for t in range(70): u=o.step(rng.standard_normal(5000).astype(np.float32))\n"
        "import hashlib; print(hashlib.sha1(u.tobytes()+o.gram().tobytes()).hexdigest())\n"
    ) % os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = set()
    for n in ("1", "3"):
        env = dict(os.environ, OMP_NUM_THREADS=n)
        outs.add(subprocess.run([sys.executable, "-c", code], env=env, check=True,
                                capture_output=True, text=True).stdout.strip())
    assert len(outs) == 1


# ------------------------------------------- parameter update (Algorithm 1, Section 2)
def test_update_plain_step_and_element_loop():
    from oracle import wrapper
    rng = np.random.default_rng(40)
    theta, u = rng.standard_normal(257), rng.standard_normal(257)
    eta, gamma = 0.125, 0.5  # exactly representable: no rounding in the scalars
    got = wrapper.apply_update(theta, u, eta, gamma)
    want = np.array([(1 - 0.0625) * theta[i] - 0.125 * u[i] for i in range(257)])
    assert np.allclose(got, want, rtol=0, atol=1e-15)
    # gamma = 0 is the last line of Algorithm 1's loop
    assert np.array_equal(wrapper.apply_update(theta, u, eta), theta - 0.125 * u)
    # eta = 0 leaves the parameters alone
    assert np.array_equal(wrapper.apply_update(theta, u, 0.0, 0.3, 5.0), theta)


def test_update_decoupled_decay_is_gradient_descent_on_the_l2_regularised_loss():
    # with the identity as preconditioner, u = grad L(theta) and the decoupled rule is
    # theta - eta (grad L + gamma theta): gradient descent on L + gamma/2 |theta|^2.  On the
    # quadratic L = 1/2 theta^T A theta - b^T theta it converges to (A + gamma I)^-1 b.
    from oracle import wrapper
    rng = np.random.default_rng(41)
    M = rng.standard_normal((6, 6))
    A = M @ M.T + np.eye(6)
    b = rng.standard_normal(6)
    gamma, eta = 0.25, 0.03125
    theta = np.zeros(6)
    for _ in range(4000):
        theta = wrapper.apply_update(theta, A @ theta - b, eta, gamma)
    assert np.allclose(theta, np.linalg.solve(A + gamma * np.eye(6), b), rtol=1e-9, atol=1e-12)


def test_update_clipping():
    from oracle import wrapper
    rng = np.random.default_rng(42)
    theta, u = rng.standard_normal(1000), 7.0 * rng.standard_normal(1000)
    nrm = np.linalg.norm(u)
    assert abs(wrapper.update_norm(u) - nrm) <= 1e-12 * nrm
    # active: the step has length eta * c exactly, in the direction of -u
    step = wrapper.apply_update(theta, u, 0.5, 0.0, clip_norm=10.0) - theta
    assert abs(np.linalg.norm(step) - 5.0) < 1e-12
    assert np.allclose(step / np.linalg.norm(step), -u / nrm, atol=1e-14)
    # inactive above the norm, off at 0, harmless for u = 0
    for c in (0.0, 2.0 * nrm):
        assert np.array_equal(wrapper.apply_update(theta, u, 0.5, 0.0, c), theta - 0.5 * u)
    assert wrapper.clip_scale(np.zeros(5), 1.0) == 1.0
    # a sub-range with the scale of the whole vector equals the slice of the whole update
    s = wrapper.clip_scale(u, 10.0)
    whole = wrapper.apply_update(theta, u, 0.5, 0.125, 10.0)
    part = wrapper.apply_update(theta[100:300], u[100:300], 0.5, 0.125, scale=s)
    assert np.array_equal(part, whole[100:300])


def test_ef_evolution_metric():
    from oracle import wrapper
    got = wrapper.ef_evolution([1.0, 1.0, 3.0], [2.0, 2.0, 2.0])
    assert np.allclose(got, [0.5, 0.25, 0.5])


# ------------------------------------------------------------- Sparse GGT (appendix)
def _ggt_definition(rows, x, eps):
    """((sum_i c_i c_i^T)^(1/2) + eps I)^-1 x with a dense d x d eigendecomposition."""
    C = np.asarray(rows, np.float64)
    lam, Q = np.linalg.eigh(C.T @ C)
    root = np.sqrt(np.maximum(lam, 0.0))
    return Q @ ((Q.T @ x) / (root + eps))


def test_ggt_matches_the_dense_definition():
    from oracle import ggt
    d, m, k, eps = 120, 5, 12, 0.05
    rng = np.random.default_rng(50)
    o = ggt.RefSparseGGT(d, m, k, eps)
    sim = DenseSim(d, m, k, 1.0)  # for the window only: its own solve is not used
    for t in range(13):  # the window fills and wraps twice
        g = rng.standard_normal(d).astype(np.float32)
        u = o.step(g)
        sim.step(g)
        rows = sim.G[:min(t + 1, m)]
        x = sim.G[t % m]
        want = _ggt_definition(rows, x, np.float64(np.float32(eps)))
        assert rel(u, want) < 1e-6, t
    o.close()


def test_ggt_closed_forms():
    from oracle import ggt
    d, eps = 64, 0.25
    rng = np.random.default_rng(51)
    # m = 1: the window is x alone and u = x / (|x| + eps)
    o = ggt.RefSparseGGT(d, 1, 8, eps)
    for _ in range(3):
        u = o.step(rng.standard_normal(d).astype(np.float32))
        idx, val = o.row(0)
        x = np.zeros(d)
        x[idx] = val
        assert rel(u, x / (np.linalg.norm(x) + eps)) < 1e-6
    o.close()
    # rows with disjoint supports are orthogonal: again u = x / (|x| + eps)
    o = ggt.RefSparseGGT(d, 4, 4, eps)
    for t in range(4):
        g = np.zeros(d, np.float32)
        g[8 * t:8 * t + 4] = 1.0 + rng.random(4)
        u = o.step(g)
        assert rel(u, g / (np.linalg.norm(g.astype(np.float64)) + eps)) < 1e-6
    o.close()
    # a repeated row (rank-deficient window): c c^T counted twice, u = x / (sqrt(2) |x| + eps)
    o = ggt.RefSparseGGT(d, 3, 4, eps)
    g = np.zeros(d, np.float32)
    g[:4] = (1.0, -2.0, 3.0, 0.5)
    o.step(g)
    u = o.step(g)  # the error buffer is zero on the kept entries, so the same row again
    assert rel(u, g / (np.sqrt(2.0) * np.linalg.norm(g.astype(np.float64)) + eps)) < 1e-6
    o.close()


def test_ggt_large_eps_limit_and_scaling():
    from oracle import ggt
    d, m, k = 80, 4, 8
    rng = np.random.default_rng(52)
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(6)]
    big = ggt.RefSparseGGT(d, m, k, 1e6)
    for g in grads:
        u = big.step(g)
    idx, val = big.row((len(grads) - 1) % m)
    x = np.zeros(d)
    x[idx] = val
    assert rel(u * 1e6, x) < 1e-4  # eps -> infinity: u -> x / eps
    big.close()
    # (G G^T)^(1/2) is homogeneous of degree 1: scaling gradients and eps by s leaves u unchanged
    a, b = ggt.RefSparseGGT(d, m, k, 0.125), ggt.RefSparseGGT(d, m, k, 0.5)
    for g in grads:
        ua, ub = a.step(g), b.step(4.0 * g)
        assert rel(ua, ub.astype(np.float64)) < 1e-6
    a.close()
    b.close()
