"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by
element on the same seeded inputs.  State (error buffer, ring rows) must be bit-exact at
every step; the update must agree within 1e-4 relative L2 (the bound the benchmark
definition states for fp32)."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2306_06098_b200 import gradgen

pytestmark = pytest.mark.gpu

U_TOL = 1e-4  # relative L2 on the update, fp32


def _binding():
    from paper_2306_06098_b200 import binding
    return binding


def bits(a):
    return np.ascontiguousarray(a).view(np.uint32)


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def lincomb_amplification(cpu, u_ref):
    """| |G|^T |w| | / |u| for the oracle's window and Eq. (2) weights: how much larger the
    terms of the linear combination are than its result.  fp32 accumulation of the
    combination (the precision the paper's LCG kernel uses) loses this factor times the
    fp32 unit roundoff; it is ~1 for the benchmark workloads and large only when window
    rows are nearly parallel (e.g. k = 1 with a repeated coordinate)."""
    assert not cpu.flags & ref.RHS_ACCUMULATOR
    w = -cpu.coef()
    w[(cpu.step_count - 1) % cpu.m] += 1.0 / np.float64(np.float32(cpu.lam))
    acc = np.zeros(cpu.d)
    for r in range(cpu.m):
        idx, val = cpu.row(r)
        np.add.at(acc, idx, np.abs(w[r]) * np.abs(val.astype(np.float64)))
    return np.linalg.norm(acc) / max(np.linalg.norm(u_ref.astype(np.float64)), 1e-300)


def run_parity(d, m, k, lam, grads, flags=0, check_rows="new", gram_every=0,
               allow_amplified=False, block=0, gpu_flags=0, gram_at=(), resid_from=None):
    """grads: iterable of fp32 numpy arrays.  Returns the worst update error seen.

    allow_amplified: for deliberately degenerate windows only - the bound becomes
    U_TOL + 8 * 2^-24 * amplification (see lincomb_amplification).
    gram_at: steps after which the whole scalar-product matrix is compared with the oracle's.
    resid_from: from this step on, the residual of the m x m solve (the drift monitor of the
    incrementally updated inverse) must stay below 1e-9 at every step."""
    B = _binding()
    gpu = B.Efcp(d, m, k, lam, flags | gpu_flags, block)  # gpu_flags: options the oracle has no part in
    cpu = ref.RefEFCP(d, m, k, lam, flags, block)
    assert gpu.k == cpu.k  # same row length (matters for block-wise Top-k)
    g_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    u_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    worst = worst_resid = 0.0
    for t, g in enumerate(grads):
        g = np.ascontiguousarray(g, np.float32)
        g_dev.copy_(torch.from_numpy(g))
        u_dev.fill_(float("nan"))  # every element must be overwritten
        gpu.step(g_dev, u_dev)
        u_ref = cpu.step(g)
        u = u_dev.cpu().numpy()
        assert gpu.status() == 0, (t, gpu.status())
        assert np.array_equal(bits(gpu.error()), bits(cpu.error())), f"error buffer differs at step {t}"
        slot = t % m
        gi, gv = gpu.row(slot)
        ci, cv = cpu.row(slot)
        assert np.array_equal(gi, ci), f"row indices differ at step {t}"
        assert np.array_equal(bits(gv), bits(cv)), f"row values differ at step {t}"
        assert np.isfinite(u).all(), f"update has unwritten / non-finite entries at step {t}"
        err = rel_l2(u, u_ref)
        worst = max(worst, err)
        tol = U_TOL
        if allow_amplified and err > U_TOL:
            tol = U_TOL + 8 * 2.0 ** -24 * lincomb_amplification(cpu, u_ref)
        assert err <= tol, f"update rel-L2 {err:.3e} (tol {tol:.3e}) at step {t}"
        if resid_from is not None and t >= resid_from:
            r = gpu.last_residual()
            worst_resid = max(worst_resid, r)
            assert r < 1e-9, f"m x m residual {r:.3e} at step {t}"
        if (gram_every and (t % gram_every == 0)) or t in gram_at:
            Sg, Sc = gpu.gram(), cpu.gram()
            assert np.array_equal(Sg, Sg.T)
            assert np.allclose(Sg, Sc, rtol=1e-12, atol=1e-12 * np.abs(Sc).max())
    if check_rows == "all":
        for s in range(m):
            gi, gv = gpu.row(s)
            ci, cv = cpu.row(s)
            assert np.array_equal(gi, ci) and np.array_equal(bits(gv), bits(cv))
    assert gpu.step_count == cpu.step_count
    assert gpu.validate() == 0  # offset table, 16-bit stream and slab weights are consistent
    print(f"parity d={d} m={m} k={k}: worst update rel-L2 {worst:.3e}" +
          (f", worst m x m residual {worst_resid:.3e}" if resid_from is not None else ""))
    gpu.close()
    cpu.close()
    return worst


def stream_grads(w, steps):
    s = gradgen.GradStream.for_workload(w)
    for _ in range(steps):
        yield s.next().numpy()


def test_c1_full_run():
    w = gradgen.C1
    run_parity(w.d, w.m, w.k, w.lam, stream_grads(w, w.steps), check_rows="all", gram_every=7)


def test_c2_shape_first_steps():
    w = gradgen.C2
    run_parity(w.d, w.m, w.k, w.lam, stream_grads(w, 24), gram_every=8)


def test_c2_full_run_ring_wraps_at_m1024():
    """The whole ResNet-20-shaped run: 2000 steps of an m = 1024 ring, so the window fills, wraps,
    and from step 1024 on every step removes a row from the explicitly kept inverse and borders
    it with the new one (976 replacements).  Error buffer, the new row and the update are
    compared with the oracle at every step, the scalar-product matrix around each wrap and at
    the end, and the residual of the m x m solve must not drift."""
    w = gradgen.C2
    assert w.steps == 2000 and w.m == 1024
    run_parity(w.d, w.m, w.k, w.lam, stream_grads(w, w.steps), check_rows="all",
               gram_at={w.m - 1, w.m, w.m + 1, 1500, w.steps - 1}, resid_from=w.m)


@pytest.mark.parametrize("d,m,k,steps", [
    (1, 1, 1, 3), (5, 2, 2, 6), (31, 3, 31, 7), (2049, 4, 100, 9), (4097, 8, 1, 20),
    (100_003, 16, 1000, 40), (1_000_001, 8, 33_333, 12),
])
def test_ragged_sizes(d, m, k, steps):
    rng = np.random.default_rng(d)
    scale = np.exp(rng.standard_normal(d))
    grads = ((scale * rng.standard_normal(d)).astype(np.float32) for _ in range(steps))
    run_parity(d, m, k, 1e-3, grads, check_rows="all", gram_every=3, allow_amplified=(k == 1))


# ---- right-hand side = the whole accumulator a_t (EFCP_RHS_ACCUMULATOR)
def test_accumulator_rhs_c1_full_run():
    w = gradgen.C1
    run_parity(w.d, w.m, w.k, w.lam, stream_grads(w, w.steps), flags=ref.RHS_ACCUMULATOR,
               check_rows="all", gram_every=7)


@pytest.mark.parametrize("d,m,k,steps,lam", [
    (5, 2, 2, 6, 1e-3), (2049, 4, 100, 9, 1e-3), (100_003, 16, 1000, 40, 1e-4),
    (1_000_001, 8, 33_333, 12, 1e-6), (3_000_017, 8, 30_000, 11, 1e-4),
])
def test_accumulator_rhs_ragged_sizes(d, m, k, steps, lam):
    rng = np.random.default_rng(d + 1)
    scale = np.exp(rng.standard_normal(d))
    grads = ((scale * rng.standard_normal(d)).astype(np.float32) for _ in range(steps))
    run_parity(d, m, k, lam, grads, flags=ref.RHS_ACCUMULATOR, check_rows="all", gram_every=3)


def test_accumulator_rhs_c2_shape_first_steps():
    w = gradgen.C2
    run_parity(w.d, w.m, w.k, w.lam, stream_grads(w, 12), flags=ref.RHS_ACCUMULATOR)


# ---- bfloat16 window values (EFCP_VALUES_BF16)
def test_bf16_values_c1_full_run():
    w = gradgen.C1
    run_parity(w.d, w.m, w.k, w.lam, stream_grads(w, w.steps), flags=ref.VALUES_BF16,
               check_rows="all", gram_every=7)


@pytest.mark.parametrize("d,m,k,steps,lam", [
    (5, 2, 2, 6, 1e-3), (2049, 4, 100, 9, 1e-3), (100_003, 16, 1000, 40, 1e-4),
    (1_000_001, 8, 33_333, 12, 1e-4), (3_000_017, 8, 30_000, 11, 1e-4),
])
def test_bf16_values_ragged_sizes(d, m, k, steps, lam):
    rng = np.random.default_rng(d + 2)
    scale = np.exp(rng.standard_normal(d))
    grads = ((scale * rng.standard_normal(d)).astype(np.float32) for _ in range(steps))
    run_parity(d, m, k, lam, grads, flags=ref.VALUES_BF16, check_rows="all", gram_every=3)


def test_bf16_values_cannot_be_combined_with_accumulator_rhs():
    B = _binding()
    with pytest.raises(B.EfcpError) as ei:
        B.Efcp(100, 2, 10, 1e-3, B.VALUES_BF16 | B.RHS_ACCUMULATOR)
    assert ei.value.code == B.EINVAL


# ---- block-wise Top-k (efcp_create_blockwise)
@pytest.mark.parametrize("d,m,k,block,steps,flags", [
    (65_536, 8, 655, 16_384, 20, 0),          # whole blocks, steady threshold
    (100_003, 4, 1000, 4096, 12, 0),          # ragged last block
    (1_000_001, 8, 10_000, 16_384, 10, 0),
    (50_000, 4, 500, 32, 6, 0),               # smallest block: one entry per block
    (300_007, 4, 3000, 8192, 8, 2),           # with bfloat16 values
    (300_007, 4, 3000, 8192, 8, 1),           # with x = a_t
    (20_000, 3, 20_000, 1024, 5, 0),          # k = d: every entry kept
])
def test_blockwise_topk(d, m, k, block, steps, flags):
    rng = np.random.default_rng(d + block)
    scale = np.exp(rng.standard_normal(d))
    grads = ((scale * rng.standard_normal(d)).astype(np.float32) for _ in range(steps))
    run_parity(d, m, k, 1e-3, grads, flags=flags, check_rows="all", block=block)


def test_blockwise_topk_ties_and_threshold_jumps():
    d, m, k, block = 40_000, 4, 400, 2048
    rng = np.random.default_rng(70)
    grads = [rng.integers(-2, 3, d).astype(np.float32) for _ in range(4)]
    grads += [(s * rng.standard_normal(d)).astype(np.float32) for s in (1.0, 0.01, 0.01, 50.0, 1.0)]
    grads += [np.zeros(d, np.float32), np.full(d, 2.5, np.float32)]
    run_parity(d, m, k, 1e-2, grads, check_rows="all", block=block)


def test_blockwise_dense_selection_beyond_one_key_per_thread():
    # 20 % density: a block keeps more entries than the kernel has threads, so every step
    # takes the bisection over all keys of the block
    d, m, k = 65_536, 4, 13_108
    rng = np.random.default_rng(71)
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(5)]
    run_parity(d, m, k, 1e-3, grads, check_rows="all", block=4096)
    run_parity(d, m, k, 1e-3, grads, check_rows="all", block=1024)


def test_blockwise_crowded_ranges_and_drifting_threshold():
    # every block has a hot segment of 300 coordinates of nearly equal magnitude (all the
    # candidates fall into one warp's range, more than its list holds), and the overall scale
    # decays and recovers so that the threshold leaves the margin in both directions
    d, m, k, block = 8192 * 6 + 1000, 4, 502, 8192
    rng = np.random.default_rng(72)
    hot = np.zeros(d, bool)
    for b0 in range(0, d, block):
        hot[b0 + 700:b0 + 1000] = True
    grads = []
    for s in (1.0, 1.0, 0.93, 0.6, 0.2, 0.2, 0.21, 3.0, 3.0, 2.9, 1e-3, 1e-3):
        g = rng.standard_normal(d)
        g[hot] = 5.0 + 0.01 * rng.standard_normal(int(hot.sum()))
        grads.append((s * g).astype(np.float32))
    run_parity(d, m, k, 1e-2, grads, check_rows="all", block=block)
    run_parity(d, m, k, 1e-2, grads, check_rows="all", block=16_384)


def test_blockwise_unaligned_gradient_and_side_stream():
    B = _binding()
    d, m, k, block = 70_001, 4, 700, 4096
    rng = np.random.default_rng(73)
    gpu = B.Efcp(d, m, k, 1e-3, 0, block)
    cpu = ref.RefEFCP(d, m, k, 1e-3, 0, block)
    gbuf = torch.empty(d + 3, dtype=torch.float32, device="cuda")
    ubuf = torch.empty(d + 3, dtype=torch.float32, device="cuda")
    side = torch.cuda.Stream()
    for t in range(6):
        g = rng.standard_normal(d).astype(np.float32)
        off = 1 if t % 2 == 0 else 0  # plain loads on even steps, bulk copies on odd ones
        gv, uv = gbuf[off:d + off], ubuf[3:d + 3]
        gv.copy_(torch.from_numpy(g))
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            gpu.step(gv, uv)
        side.synchronize()
        u_ref = cpu.step(g)
        assert gpu.status() == 0
        assert np.array_equal(bits(gpu.error()), bits(cpu.error())), t
        gi, gvals = gpu.row(t % m)
        ci, cvals = cpu.row(t % m)
        assert np.array_equal(gi, ci) and np.array_equal(bits(gvals), bits(cvals)), t
        assert rel_l2(uv.cpu().numpy(), u_ref) <= U_TOL
    assert gpu.validate() == 0
    gpu.close()
    cpu.close()


# ---- the two accumulators of the linear combination: int32 fixed point (default) and fp32
# (EFCP_LCG_FP32).  Every other parity case runs the default; these run both.
def _fp32():
    return _binding().LCG_FP32


def test_fp32_lcg_c1_full_run():
    w = gradgen.C1
    run_parity(w.d, w.m, w.k, w.lam, stream_grads(w, w.steps), check_rows="all",
               gpu_flags=_fp32())


@pytest.mark.parametrize("d,m,k,lam,steps,flags,block", [
    (300_007, 16, 3000, 1e-3, 24, 0, 0),         # ragged tail, several slabs
    (1_000_001, 8, 10_000, 1e-4, 10, 2, 0),      # bfloat16 values
    (300_007, 4, 3000, 1e-3, 8, 0, 8192),        # block-wise Top-k
    (3_000_017, 8, 30_000, 1e-4, 12, 0, 0),      # many slabs, the ring wraps
])
def test_both_lcg_accumulators_parity(d, m, k, lam, steps, flags, block):
    rng = np.random.default_rng(d + m)
    scale = np.exp(rng.standard_normal(d)).astype(np.float32)  # log-normal scales: heavy tail
    grads = [(scale * rng.standard_normal(d)).astype(np.float32) for _ in range(steps)]
    run_parity(d, m, k, lam, grads, flags=flags, block=block)
    run_parity(d, m, k, lam, grads, flags=flags, block=block, gpu_flags=_fp32())


def test_fixed_point_lcg_hard_inputs():
    """Ties, threshold jumps of 1e3, an all-zero gradient, outliers 300 times the rest: slabs
    whose grid is too coarse have to fall back to fp32, and the update stays in tolerance.
    (The same inputs run through the fp32 accumulator first: they are inside what the m x m
    solve can take, see the note on scale jumps in the tolerances.)"""
    B = _binding()
    d, m, k = 200_000, 8, 2000
    rng = np.random.default_rng(81)
    grads = [rng.integers(-2, 3, d).astype(np.float32) for _ in range(3)]
    grads += [(s * rng.standard_normal(d)).astype(np.float32) for s in (1.0, 1e-3, 1e-3, 30.0, 1.0)]
    g = rng.standard_normal(d).astype(np.float32)
    g[::5000] *= 300.0
    grads += [g, np.zeros(d, np.float32), rng.standard_normal(d).astype(np.float32)]
    run_parity(d, m, k, 1e-2, grads, check_rows="all", gpu_flags=_fp32())
    run_parity(d, m, k, 1e-2, grads, check_rows="all")


def test_fixed_point_lcg_fallback_path(monkeypatch):
    """With the acceptance bound at zero every slab is accumulated in integers, rejected and
    accumulated again in fp32: the second pass must start from a clean accumulator."""
    B = _binding()
    monkeypatch.setenv("EFCP_LCG_FIXED_TOL", "0")
    d, m, k = 300_007, 8, 3000
    rng = np.random.default_rng(83)
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(10)]
    run_parity(d, m, k, 1e-3, grads, check_rows="all")
    run_parity(d, m, k, 1e-3, grads, flags=B.VALUES_BF16, block=4096)
    h = B.Efcp(d, m, k, 1e-3)
    g_dev = torch.from_numpy(grads[0]).cuda()
    u_dev = torch.empty(d, device="cuda")
    h.step(g_dev, u_dev)
    assert h.fixed_point_fallbacks() > 0
    h.close()


def test_fixed_point_lcg_is_reproducible_and_survives_a_checkpoint():
    B = _binding()
    d, m, k, lam = 500_000, 8, 5000, 1e-3
    rng = np.random.default_rng(82)
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(12)]
    a, b = B.Efcp(d, m, k, lam), B.Efcp(d, m, k, lam)
    g_dev = torch.empty(d, device="cuda")
    ua, ub = torch.empty(d, device="cuda"), torch.empty(d, device="cuda")
    for t, g in enumerate(grads):
        g_dev.copy_(torch.from_numpy(g))
        a.step(g_dev, ua)
        b.step(g_dev, ub)
        if a.fixed_point_fallbacks() == 0 and b.fixed_point_fallbacks() == 0:
            assert torch.equal(ua, ub), t  # integer sums do not depend on the order of the adds
    assert a.fixed_point_fallbacks() == 0  # well-scaled data: every slab took the integer route
    blob = a.state_export()
    c = B.Efcp(d, m, k, lam)
    c.state_import(blob)
    g = rng.standard_normal(d).astype(np.float32)
    g_dev.copy_(torch.from_numpy(g))
    uc = torch.empty(d, device="cuda")
    a.step(g_dev, ua)
    c.step(g_dev, uc)
    assert torch.equal(ua, uc)
    assert c.validate() == 0 and c.status() == 0
    for h in (a, b, c):
        h.close()
    # the accumulator is not part of the state: an fp32 handle takes the same blob
    f = B.Efcp(d, m, k, lam, B.LCG_FP32)
    f.state_import(blob)
    assert f.fixed_point_fallbacks() == 0 and f.step_count == len(grads)
    f.close()


def test_blockwise_rejects_bad_block_sizes():
    B = _binding()
    for block in (16, 48, 20_000, -32):
        with pytest.raises(B.EfcpError) as ei:
            B.Efcp(10_000, 2, 100, 1e-3, 0, block)
        assert ei.value.code == B.EINVAL


def test_heavy_ties():
    # values from a small set: most of the selection is decided by the index rule
    d, m, k = 50_000, 4, 777
    rng = np.random.default_rng(11)
    grads = [rng.integers(-2, 3, d).astype(np.float32) for _ in range(6)]
    run_parity(d, m, k, 1e-2, grads, check_rows="all")


def test_all_equal_and_zero_gradients():
    d, m, k = 10_000, 3, 100
    grads = [np.full(d, 1.5, np.float32), np.zeros(d, np.float32), np.full(d, -1.5, np.float32),
             np.zeros(d, np.float32), np.zeros(d, np.float32)]
    run_parity(d, m, k, 1e-1, grads, check_rows="all")


def test_denormals_are_ordered_not_flushed():
    d, m, k = 4096, 2, 64
    rng = np.random.default_rng(12)
    g = (rng.integers(1, 1 << 20, d).astype(np.uint32)).view(np.float32)  # all denormal
    g = g * np.where(rng.random(d) < 0.5, -1, 1).astype(np.float32)
    big = g.copy()
    big[::97] = 1.0
    run_parity(d, m, k, 1.0, [g, big, g], check_rows="all")


def test_unaligned_pointers():
    B = _binding()
    d, m, k = 70_001, 4, 500
    rng = np.random.default_rng(13)
    gpu = B.Efcp(d, m, k, 1e-3)
    cpu = ref.RefEFCP(d, m, k, 1e-3)
    gbuf = torch.empty(d + 3, dtype=torch.float32, device="cuda")
    ubuf = torch.empty(d + 3, dtype=torch.float32, device="cuda")
    for t in range(5):
        g = rng.standard_normal(d).astype(np.float32)
        gv, uv = gbuf[1:d + 1], ubuf[3:d + 3]
        gv.copy_(torch.from_numpy(g))
        gpu.step(gv, uv)
        u_ref = cpu.step(g)
        assert np.array_equal(bits(gpu.error()), bits(cpu.error()))
        assert rel_l2(uv.cpu().numpy(), u_ref) <= U_TOL


def test_large_d_short_window_wraps():
    # large d with a short window so that the ring wraps at a size spanning many slabs
    d, m, k = 3_000_017, 8, 30_000
    rng = np.random.default_rng(14)
    scale = np.exp(rng.standard_normal(d)).astype(np.float32)
    grads = ((scale * rng.standard_normal(d).astype(np.float32)) for _ in range(19))
    run_parity(d, m, k, 1e-4, grads, check_rows="all", gram_every=6)


def test_nonfinite_gradient_sets_status():
    B = _binding()
    d = 1000
    gpu = B.Efcp(d, 2, 10, 1e-3)
    g = torch.randn(d, device="cuda")
    g[17] = float("inf")
    u = torch.empty_like(g)
    gpu.step(g, u)
    assert gpu.status() == B.ENUMERIC


def test_argument_errors():
    B = _binding()
    for args in ((0, 1, 1, 1e-3), (4, 0, 1, 1e-3), (4, 1, 0, 1e-3), (4, 1, 5, 1e-3),
                 (4, 1, 1, 0.0), (4, 1, 1, float("inf")), (2 ** 31, 1, 1, 1e-3), (4, 5000, 1, 1e-3)):
        with pytest.raises(B.EfcpError) as ei:
            B.Efcp(*args)
        assert ei.value.code == B.EINVAL
    gpu = B.Efcp(16, 2, 4, 1e-3)
    g = torch.zeros(16, device="cuda")
    with pytest.raises(B.EfcpError):
        gpu.step_ptr(0, g.data_ptr())
    with pytest.raises(B.EfcpError):
        gpu.step_ptr(g.data_ptr(), g.data_ptr())  # update must not alias grad
    assert B.state_bytes(0, 1, 1) == -1


def test_host_entry_point_matches_device_entry_point():
    B = _binding()
    d, m, k = 200_000, 8, 2000
    rng = np.random.default_rng(15)
    a, b = B.Efcp(d, m, k, 1e-3), B.Efcp(d, m, k, 1e-3)
    gh = torch.empty(d, dtype=torch.float32).pin_memory()
    uh = torch.empty(d, dtype=torch.float32).pin_memory()
    gd = torch.empty(d, dtype=torch.float32, device="cuda")
    ud = torch.empty(d, dtype=torch.float32, device="cuda")
    for t in range(10):
        gh.copy_(torch.from_numpy(rng.standard_normal(d).astype(np.float32)))
        gd.copy_(gh)
        a.step(gd, ud)
        b.step_host(gh, uh)
        assert np.array_equal(bits(a.error()), bits(b.error()))
        assert rel_l2(uh.numpy(), ud.cpu().numpy()) <= 1e-5


def test_inverse_does_not_drift_over_twenty_turns_of_the_ring():
    """The explicitly kept inverse is only ever updated, never rebuilt.  20,000 steps of the
    ResNet-20-shaped stream (about 19,000 row replacements in a full m = 1024 window, the order
    of a whole training run) must leave the residual of the m x m solve where it started, and
    the update must still solve the defining system at the end."""
    B = _binding()
    w = gradgen.C2
    gs = _device_stream(w)
    gpu = B.Efcp(w.d, w.m, w.k, w.lam)
    u = torch.empty(w.d, dtype=torch.float32, device="cuda")
    worst = 0.0
    for t in range(20_000):
        gpu.step(gs.next(), u)
        if t % 500 == 499:
            worst = max(worst, gpu.last_residual())
    assert gpu.status() == 0
    print(f"m x m residual over 20000 steps of {w.name}: worst {worst:.3e}")
    assert worst < 1e-9
    lam = float(np.float32(w.lam))
    I, V = gpu.window()
    slot = (gpu.step_count - 1) % w.m
    ud = u.double()
    x = torch.zeros(w.d, dtype=torch.float64, device="cuda")
    x.index_add_(0, I[slot].long(), V[slot].double())
    Fu = lam * ud
    bound = lam * ud.abs()
    for r in range(w.m):
        idx, val = I[r].long(), V[r].double()
        Fu.index_add_(0, idx, val * ((val * ud[idx]).sum() / w.m))
        bound.index_add_(0, idx, val.abs() * ((val.abs() * ud[idx].abs()).sum() / w.m))
    assert float((Fu - x).norm()) <= 4 * 2.0 ** -24 * float(bound.norm())
    gpu.close()


def test_host_entry_point_sends_finished_ranges_early_at_large_d():
    """Above about 600 slabs efcp_step_host runs the linear combination over four ranges of
    slabs and copies every finished range to the host while the next is accumulated: the
    result must be that of the device entry point."""
    B = _binding()
    d, m, k = 26_000_003, 2, 26_000
    rng = np.random.default_rng(16)
    a, b = B.Efcp(d, m, k, 1e-3), B.Efcp(d, m, k, 1e-3)
    gh = torch.empty(d, dtype=torch.float32).pin_memory()
    uh = torch.empty(d, dtype=torch.float32).pin_memory()
    gd = torch.empty(d, dtype=torch.float32, device="cuda")
    ud = torch.empty(d, dtype=torch.float32, device="cuda")
    for t in range(4):
        gh.copy_(torch.from_numpy(rng.standard_normal(d).astype(np.float32)))
        gd.copy_(gh)
        uh.fill_(float("nan"))
        a.step(gd, ud)
        b.step_host(gh, uh)
        assert np.array_equal(bits(a.error()), bits(b.error()))
        assert torch.isfinite(uh).all()
        assert torch.equal(uh, ud.cpu())  # integer accumulation: no dependence on the slab order
    assert a.fixed_point_fallbacks() == 0 and b.fixed_point_fallbacks() == 0
    a.close()
    b.close()


# ---- full size, in the launch configuration the benchmark times
def _device_stream(w, device="cuda"):
    return gradgen.GradStream.for_workload(w, device)


def _c5_corners():
    """The corners of the density x window sweep: densities 0.1 % and 10 %, windows 128 and 1024."""
    want = {"c5_dens0.001_m128", "c5_dens0.001_m1024", "c5_dens0.1_m128", "c5_dens0.1_m1024"}
    pts = [w for w in gradgen.sweep_points() if w.name in want]
    assert len(pts) == 4
    return pts


@pytest.mark.parametrize("w,steps", [(gradgen.C3, 20), (gradgen.C4, 3)] +
                         [(w, 3) for w in _c5_corners()], ids=lambda x: getattr(x, "name", None))
def test_full_size_first_steps_match_oracle(w, steps):
    """Element by element at the full dimension: every coordinate of the error buffer, the
    inserted rows and the update, for the first steps of the workload's own gradient stream
    (generated on the device, the same bytes copied to the oracle)."""
    B = _binding()
    gs = _device_stream(w)
    gpu = B.Efcp(w.d, w.m, w.k, w.lam)
    cpu = ref.RefEFCP(w.d, w.m, w.k, w.lam)
    u_dev = torch.empty(w.d, dtype=torch.float32, device="cuda")
    for t in range(steps):
        g_dev = gs.next()
        gpu.step(g_dev, u_dev)
        u_ref = cpu.step(g_dev.cpu().numpy())
        assert gpu.status() == 0
        assert np.array_equal(bits(gpu.error()), bits(cpu.error())), f"error buffer differs, step {t}"
        gi, gv = gpu.row(t)
        ci, cv = cpu.row(t)
        assert np.array_equal(gi, ci) and np.array_equal(bits(gv), bits(cv)), f"row differs, step {t}"
        assert rel_l2(u_dev.cpu().numpy(), u_ref) <= U_TOL
    gpu.close()
    cpu.close()


@pytest.mark.parametrize("w,flags", [(gradgen.C3, 0), (gradgen.C4, 0), (gradgen.C3, 1),
                                     (gradgen.C3, 8), (gradgen.C4, 8)] +
                         [(w, 0) for w in _c5_corners()],
                         ids=["c3", "c4", "c3_rhs_accumulator", "c3_fp32_lcg", "c4_fp32_lcg"] +
                         [w.name for w in _c5_corners()])
def test_full_size_steady_state_residual(w, flags):
    """With the window completely filled (the state the benchmark times) the update must
    solve the defining system (lambda I + (1/m) G^T G) u = x up to the rounding of u itself:
    | F u - x | <= 4 * 2^-24 * | lambda |u| + (1/m) |G|^T (|G| |u|) |, evaluated in fp64 on
    the device from the library's own window.  A wrong coefficient, a dropped row or a
    misplaced entry breaks this by orders of magnitude."""
    B = _binding()
    gs = _device_stream(w)
    gpu = B.Efcp(w.d, w.m, w.k, w.lam, flags)
    u = torch.empty(w.d, dtype=torch.float32, device="cuda")
    for t in range(w.m + 3):
        g = gs.next()
        gpu.step(g, u)
    assert gpu.status() == 0
    del gs
    lam = float(np.float32(w.lam))
    I, V = gpu.window()
    slot = (gpu.step_count - 1) % w.m
    ud = u.double()
    x = torch.zeros(w.d, dtype=torch.float64, device="cuda")
    if flags & 1:
        x += torch.from_numpy(gpu.error()).cuda().double()
    x.index_add_(0, I[slot].long(), V[slot].double())
    Gu = torch.empty(w.m, dtype=torch.float64, device="cuda")
    Gau = torch.empty(w.m, dtype=torch.float64, device="cuda")
    for r in range(w.m):
        idx, val = I[r].long(), V[r].double()
        ur = ud[idx]
        Gu[r] = (val * ur).sum()
        Gau[r] = (val.abs() * ur.abs()).sum()
    Fu = lam * ud
    bound = lam * ud.abs()
    for r in range(w.m):
        idx, val = I[r].long(), V[r].double()
        Fu.index_add_(0, idx, val * (Gu[r] / w.m))
        bound.index_add_(0, idx, val.abs() * (Gau[r] / w.m))
    res = float((Fu - x).norm())
    lim = 4 * 2.0 ** -24 * float(bound.norm())
    print(f"{w.name}: |Fu - x| = {res:.3e}, rounding bound {lim:.3e}, |x| = {float(x.norm()):.3e}")
    assert res <= lim
    assert gpu.last_residual() < 1e-9
    if not flags:
        print(f"{w.name}: slabs redone in fp32 over {gpu.step_count} steps: {gpu.fixed_point_fallbacks()}")
        assert gpu.fixed_point_fallbacks() == 0  # the benchmark workloads never need the fallback
    if not flags & 1:
        # The accumulation of the linear combination alone, range by range: u against the same
        # combination sum_r w_r row_r formed in fp64 from the library's window and weights.
        # With the fixed-point accumulator every range of coordinates must stay well inside
        # the update's tolerance even where a coordinate collects a hundred terms (10 %
        # density, m = 1024); the worst range is printed.
        wts = torch.from_numpy(gpu.weights()).cuda()
        exact = torch.zeros(w.d, dtype=torch.float64, device="cuda")
        for r in range(w.m):
            exact.index_add_(0, I[r].long(), V[r].double() * wts[r])
        span = 32_768
        pad = (-w.d) % span
        diff2 = torch.nn.functional.pad((ud - exact) ** 2, (0, pad)).view(-1, span).sum(1)
        ref2 = torch.nn.functional.pad(exact ** 2, (0, pad)).view(-1, span).sum(1)
        whole = float(diff2.sum().sqrt() / ref2.sum().sqrt())
        live = ref2 > 0
        per_range = (diff2[live] / ref2[live]).sqrt()
        print(f"{w.name}: linear combination vs fp64, whole vector {whole:.2e}, worst range of "
              f"{span} coordinates {float(per_range.max()):.2e} (of {int(live.sum())} ranges)")
        assert whole <= 2e-5
        assert float(per_range.max()) <= U_TOL
    gpu.close()


def test_threshold_jumps_between_steps():
    """The selection threshold of one step is the starting guess of the next; gradients whose
    scale jumps by factors of 30 to 1000 in both directions make that guess useless, and the
    result must not change (the exact two-pass route takes over)."""
    d, m, k = 400_003, 8, 4000
    rng = np.random.default_rng(21)
    scales = [1.0, 1.0, 0.03, 0.03, 30.0, 1.0, 0.01, 10.0, 10.0, 1.0, 1.0, 1.0]
    grads = ((s * rng.standard_normal(d)).astype(np.float32) for s in scales)
    run_parity(d, m, k, 1e-3, grads, check_rows="all")


def test_two_pass_route_alone(monkeypatch):
    """EFCP_NO_SPEC=1 switches the speculative candidate buckets off: same results."""
    monkeypatch.setenv("EFCP_NO_SPEC", "1")
    d, m, k = 300_007, 8, 3000
    rng = np.random.default_rng(22)
    scale = np.exp(rng.standard_normal(d))
    grads = ((scale * rng.standard_normal(d)).astype(np.float32) for _ in range(10))
    run_parity(d, m, k, 1e-4, grads, check_rows="all")


@pytest.mark.parametrize("flags", [0, 1, 2], ids=["fp32", "rhs_accumulator", "values_bf16"])
def test_checkpoint_resume_continues_bit_for_bit(flags):
    B = _binding()
    d, m, k = 250_003, 6, 2500
    rng = np.random.default_rng(40 + flags)
    scale = np.exp(rng.standard_normal(d))
    grads = [(scale * rng.standard_normal(d)).astype(np.float32) for _ in range(16)]
    a = B.Efcp(d, m, k, 1e-4, flags)
    g_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    ua = torch.empty(d, dtype=torch.float32, device="cuda")
    ub = torch.empty(d, dtype=torch.float32, device="cuda")
    for g in grads[:9]:  # past one turn of the ring
        g_dev.copy_(torch.from_numpy(g))
        a.step(g_dev, ua)
    blob = a.state_export()
    b = B.Efcp(d, m, k, 1e-4, flags)
    b.state_import(blob)
    assert b.step_count == a.step_count == 9
    for g in grads[9:]:
        g_dev.copy_(torch.from_numpy(g))
        a.step(g_dev, ua)
        b.step(g_dev, ub)
        # the update is a sum of fp32 shared-memory atomics whose order is not fixed: equal up
        # to fp32 rounding of the accumulation; the state below is bit for bit
        assert rel_l2(ub.cpu().numpy(), ua.cpu().numpy()) <= 1e-6
        assert np.array_equal(bits(a.error()), bits(b.error()))
    for s in range(m):
        ai, av = a.row(s)
        bi, bv = b.row(s)
        assert np.array_equal(ai, bi) and np.array_equal(bits(av), bits(bv))
    # a blob of another shape is refused
    c = B.Efcp(d, m + 1, k, 1e-4, flags)
    with pytest.raises(B.EfcpError) as ei:
        c.state_import(blob)
    assert ei.value.code == B.EINVAL


def test_error_norm_is_the_norm_of_the_error_buffer():
    B = _binding()
    d, m, k = 123_457, 4, 1000
    rng = np.random.default_rng(50)
    opt = B.Efcp(d, m, k, 1e-3)
    g_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    assert opt.error_norm() == 0.0
    for _ in range(5):
        g_dev.copy_(torch.from_numpy(rng.standard_normal(d).astype(np.float32)))
        opt.step(g_dev, u)
        want = np.linalg.norm(opt.error().astype(np.float64))
        assert abs(opt.error_norm() - want) <= 1e-12 * want


def test_large_window_m2048():
    # a window longer than the benchmark's: the shared-memory budget forces a narrower slab
    d, m, k = 600_011, 2048, 600
    rng = np.random.default_rng(60)
    scale = np.exp(rng.standard_normal(d))
    grads = ((scale * rng.standard_normal(d)).astype(np.float32) for _ in range(4))
    run_parity(d, m, k, 1e-3, grads, gram_every=2)


def test_steps_on_a_side_stream():
    B = _binding()
    d, m, k = 200_003, 4, 2000
    rng = np.random.default_rng(61)
    gpu = B.Efcp(d, m, k, 1e-3)
    cpu = ref.RefEFCP(d, m, k, 1e-3)
    side = torch.cuda.Stream()
    g_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    u_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    for t in range(6):
        g = rng.standard_normal(d).astype(np.float32)
        g_dev.copy_(torch.from_numpy(g))
        side.wait_stream(torch.cuda.current_stream())
        gpu.step(g_dev, u_dev, stream=side)
        side.synchronize()
        u_ref = cpu.step(g)
        assert np.array_equal(bits(gpu.error()), bits(cpu.error()))
        assert rel_l2(u_dev.cpu().numpy(), u_ref) <= U_TOL
