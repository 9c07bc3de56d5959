"""The coordinate-sharded step on one GPU: several shard handles in one process whose exchange
buffers are summed on the device must reproduce the unsharded state bit for bit and the
oracle's update within the usual tolerance."""
import numpy as np
import pytest
import torch

from oracle import ref

pytestmark = pytest.mark.gpu

U_TOL = 1e-4


def _mods():
    from paper_2306_06098_b200 import binding, sharded
    return binding, sharded


def bits(a):
    return np.ascontiguousarray(a).view(np.uint32)


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def run_sharded(d, m, k, lam, grads, ranges, flags=0):
    B, S = _mods()
    n = len(ranges)
    shards, ranges = S.create_local_shards(B, d, m, k, lam, n, flags, ranges)
    stepper = S.ShardedStep(shards, S.sum_in_process)
    whole = B.Efcp(d, m, k, lam, flags)
    cpu = ref.RefEFCP(d, m, k, lam, flags)
    g_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    u_dev = torch.empty(d, dtype=torch.float32, device="cuda")
    u_whole = torch.empty(d, dtype=torch.float32, device="cuda")
    worst = 0.0
    for t, g in enumerate(grads):
        g_dev.copy_(torch.from_numpy(np.ascontiguousarray(g, np.float32)))
        u_dev.fill_(float("nan"))
        stepper.step([g_dev[lo:hi] for lo, hi in ranges], [u_dev[lo:hi] for lo, hi in ranges])
        whole.step(g_dev, u_whole)
        u_ref = cpu.step(g)
        for s in shards:
            assert s.status() == 0, (t, s.status())
        # the error buffer and the new row, shard by shard, against the oracle
        e_ref = cpu.error()
        ci, cv = cpu.row(t % m)
        got_i, got_v = [], []
        for s, (lo, hi) in zip(shards, ranges):
            assert np.array_equal(bits(s.error()), bits(e_ref[lo:hi])), f"error buffer, step {t}"
            cnt = s.row_count(t % m)
            i, v = s.row(t % m)
            assert cnt == int(((ci >= lo) & (ci < hi)).sum()), f"row length, step {t}"
            got_i.append(i[:cnt] + lo)
            got_v.append(v[:cnt])
        got_i, got_v = np.concatenate(got_i), np.concatenate(got_v)
        assert np.array_equal(got_i, ci), f"row indices, step {t}"
        assert np.array_equal(bits(got_v), bits(cv)), f"row values, step {t}"
        assert np.array_equal(bits(whole.error()), bits(e_ref))
        u = u_dev.cpu().numpy()
        assert np.isfinite(u).all()
        err = rel_l2(u, u_ref)
        worst = max(worst, err)
        assert err <= U_TOL, f"update rel-L2 {err:.3e} at step {t}"
        assert rel_l2(u, u_whole.cpu().numpy()) <= 1e-5
    for s in shards:
        assert s.validate() == 0
        s.close()
    whole.close()
    cpu.close()
    print(f"sharded x{n} d={d} m={m} k={k}: worst update rel-L2 {worst:.3e}")


def test_two_shards_match_unsharded_and_oracle():
    d, m, k = 300_007, 8, 3000
    rng = np.random.default_rng(101)
    scale = np.exp(rng.standard_normal(d))
    grads = [(scale * rng.standard_normal(d)).astype(np.float32) for _ in range(20)]
    run_sharded(d, m, k, 1e-3, grads, [(0, 150_016), (150_016, d)])


def test_three_uneven_shards_and_bf16_values():
    B, _ = _mods()
    d, m, k = 500_000, 6, 5000
    rng = np.random.default_rng(102)
    scale = np.exp(rng.standard_normal(d))
    grads = [(scale * rng.standard_normal(d)).astype(np.float32) for _ in range(14)]
    run_sharded(d, m, k, 1e-3, grads, [(0, 100_000), (100_000, 420_001), (420_001, d)])
    run_sharded(d, m, k, 1e-3, grads, [(0, 250_000), (250_000, d)], flags=B.VALUES_BF16)


def test_ties_across_the_shard_boundary():
    """Values from a small set: the threshold key is shared by thousands of entries on both
    sides of the boundary, and the index rule must hand them out to the lower shard first."""
    d, m, k = 60_000, 4, 777
    rng = np.random.default_rng(103)
    grads = [rng.integers(-2, 3, d).astype(np.float32) for _ in range(6)]
    grads += [np.full(d, 1.5, np.float32), np.zeros(d, np.float32)]
    run_sharded(d, m, k, 1e-2, grads, [(0, 20_000), (20_000, 40_001), (40_001, d)])


def test_a_shard_that_keeps_nothing():
    """All large entries live in the first half: the second shard's rows are empty."""
    d, m, k = 80_000, 4, 400
    rng = np.random.default_rng(104)
    grads = []
    for _ in range(7):
        g = 1e-3 * rng.standard_normal(d)
        g[:40_000] += rng.standard_normal(40_000)
        grads.append(g.astype(np.float32))
    run_sharded(d, m, k, 1e-3, grads, [(0, 40_000), (40_000, d)])


def test_phases_must_be_called_in_order():
    B, S = _mods()
    shards, ranges = S.create_local_shards(B, 10_000, 2, 100, 1e-3, 2)
    n0 = ranges[0][1] - ranges[0][0]
    g = torch.zeros(n0, device="cuda")
    with pytest.raises(B.EfcpError) as ei:
        shards[0].shard_phase(1)
    assert ei.value.code == B.EINVAL
    with pytest.raises(B.EfcpError):
        shards[0].step(g, torch.empty(n0, device="cuda"))  # a shard has no one-call step
    with pytest.raises(B.EfcpError):
        B.Efcp(5000, 2, 0, 1e-3, B.RHS_ACCUMULATOR, shard=(10_000, 0, 5000, 100, 0, 2))
