"""Parameter update (Algorithm 1's last line, decoupled weight decay, norm clipping) and the
torch.optim front end against the CPU oracle.  All calls go through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ref, wrapper

pytestmark = pytest.mark.gpu

EPS = 2.0 ** -23


def _binding():
    from paper_2306_06098_b200 import binding
    return binding


def close_fp32(got, theta, u, eta, gamma, scale):
    """fp32 result against the fp64 formula: a few roundings of the two terms."""
    want = wrapper.apply_update(theta, u, eta, gamma, scale=scale)
    bound = 2 * EPS * (np.abs(theta.astype(np.float64)) + eta * scale * np.abs(u.astype(np.float64)))
    return np.all(np.abs(got.astype(np.float64) - want) <= bound + 1e-45)


@pytest.mark.parametrize("eta,gamma,clip", [
    (0.1, 0.0, 0.0), (0.01, 1e-4, 0.0), (0.5, 0.01, 10.0), (0.5, 0.0, 1e9), (0.0, 0.3, 1.0),
])
def test_apply_update_matches_the_formula(eta, gamma, clip):
    B = _binding()
    d = 1_000_003
    rng = np.random.default_rng(5)
    theta = rng.standard_normal(d).astype(np.float32)
    u = (3.0 * rng.standard_normal(d)).astype(np.float32)
    h = B.Efcp(d, 2, 100, 1e-3)
    t_dev, u_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(u).cuda()
    nrm = h.update_norm(u_dev)
    assert abs(nrm - wrapper.update_norm(u)) <= 1e-12 * nrm
    h.apply_update(t_dev, u_dev, eta, gamma, clip)
    s = wrapper.clip_scale(u, clip)
    assert (clip in (10.0, 1.0)) == (s < 1.0)
    assert close_fp32(t_dev.cpu().numpy(), theta, u, eta, gamma, s)
    assert np.array_equal(u_dev.cpu().numpy(), u)  # u is an input
    assert h.status() == 0
    h.close()


def test_apply_update_on_unaligned_subranges_with_group_scalars():
    B = _binding()
    d = 300_001
    rng = np.random.default_rng(6)
    theta = rng.standard_normal(d).astype(np.float32)
    u = (5.0 * rng.standard_normal(d)).astype(np.float32)
    h = B.Efcp(d, 2, 100, 1e-3)
    t_dev, u_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(u).cuda()
    h.update_norm(u_dev, sync=False)
    s = wrapper.clip_scale(u, 7.0)
    cuts = [0, 1, 1000, 100_003, d]
    scal = [(0.1, 0.0), (0.2, 0.01), (0.05, 0.1), (0.3, 0.0)]
    for (a, b), (eta, gamma) in zip(zip(cuts[:-1], cuts[1:]), scal):
        h.apply_update(t_dev[a:b], u_dev[a:b], eta, gamma, 7.0)
    got = t_dev.cpu().numpy()
    for (a, b), (eta, gamma) in zip(zip(cuts[:-1], cuts[1:]), scal):
        assert close_fp32(got[a:b], theta[a:b], u[a:b], eta, gamma, s)
    h.close()


def test_apply_update_argument_errors():
    B = _binding()
    d = 1000
    h = B.Efcp(d, 2, 10, 1e-3)
    t, u = torch.zeros(d, device="cuda"), torch.ones(d, device="cuda")
    with pytest.raises(B.EfcpError) as ei:  # clipping without a norm of this step's u
        h.apply_update(t, u, 0.1, 0.0, 1.0)
    assert ei.value.code == B.EINVAL
    for bad in ((-0.1, 0.0, 0.0), (0.1, -1.0, 0.0), (0.1, 0.0, -2.0), (float("nan"), 0.0, 0.0),
                (float("inf"), 0.0, 0.0)):
        with pytest.raises(B.EfcpError):
            h.apply_update(t, u, *bad)
    big = torch.zeros(d + 1, device="cuda")
    with pytest.raises(B.EfcpError):
        h.apply_update(big, big.clone(), 0.1)
    with pytest.raises(B.EfcpError):  # theta and update must be different buffers
        h.apply_update(t, t, 0.1)
    assert torch.count_nonzero(t).item() == 0
    h.close()


@pytest.mark.parametrize("clip,block", [(0.0, 0), (0.05, 0), (0.05, 2048)])
def test_step_apply_follows_the_oracle(clip, block):
    B = _binding()
    d, m, k, lam = 200_003, 8, 2000, 1e-3
    eta, gamma = 0.05, 0.01
    rng = np.random.default_rng(7)
    gpu = B.Efcp(d, m, k, lam, 0, block)
    cpu = ref.RefEFCP(d, m, k, lam, 0, block)
    theta = rng.standard_normal(d).astype(np.float32)
    t_dev = torch.from_numpy(theta).cuda()
    g_dev = torch.empty(d, device="cuda")
    u_dev = torch.empty(d, device="cuda")
    clipped = 0
    for t in range(12):
        g = rng.standard_normal(d).astype(np.float32)
        g_dev.copy_(torch.from_numpy(g))
        before = t_dev.cpu().numpy()
        gpu.step_apply(g_dev, t_dev, u_dev, eta, gamma, clip)
        u_ref = cpu.step(g)
        s = wrapper.clip_scale(u_ref, clip)
        clipped += s < 1.0
        want = wrapper.apply_update(before, u_ref, eta, gamma, scale=s)
        got = t_dev.cpu().numpy().astype(np.float64)
        step_len = np.linalg.norm(want - before)
        # the step differs by the update's tolerance (1e-4 of its length), theta by rounding
        assert np.linalg.norm(got - want) <= 1e-4 * step_len + 4 * EPS * np.linalg.norm(want)
        assert np.array_equal(gpu.error().view(np.uint32), cpu.error().view(np.uint32))
    assert (clipped > 0) == (clip > 0)
    assert gpu.status() == 0 and gpu.validate() == 0
    gpu.close()
    cpu.close()


def test_torch_optimizer_front_end():
    B = _binding()
    from paper_2306_06098_b200.optim import SparseMFAC
    torch.manual_seed(0)
    model = torch.nn.Sequential(torch.nn.Linear(64, 128), torch.nn.Tanh(),
                                torch.nn.LayerNorm(128), torch.nn.Linear(128, 10)).cuda()
    decay = [p for n, p in model.named_parameters() if p.ndim > 1]
    plain = [p for n, p in model.named_parameters() if p.ndim <= 1]
    groups = [dict(params=decay, weight_decay=0.01), dict(params=plain, weight_decay=0.0, lr=0.02)]
    m, lam, clip = 4, 1e-3, 0.5
    opt = SparseMFAC(groups, lr=0.05, m=m, density=0.05, damp=lam, clip_norm=clip)
    d = sum(p.numel() for p in model.parameters())
    k = max(1, int(round(0.05 * d)))
    cpu = ref.RefEFCP(d, m, k, lam)
    order = decay + plain
    n_decay = sum(p.numel() for p in decay)
    x = torch.randn(256, 64, device="cuda")
    y = torch.randint(0, 10, (256,), device="cuda")
    losses = []
    for t in range(6):
        opt.zero_grad()
        loss = torch.nn.functional.cross_entropy(model(x), y)
        loss.backward()
        losses.append(loss.item())
        g = torch.cat([p.grad.reshape(-1) for p in order]).cpu().numpy()
        before = torch.cat([p.detach().reshape(-1) for p in order]).cpu().numpy()
        opt.step()
        u_ref = cpu.step(g)
        s = wrapper.clip_scale(u_ref, clip)
        want = np.concatenate([
            wrapper.apply_update(before[:n_decay], u_ref[:n_decay], 0.05, 0.01, scale=s),
            wrapper.apply_update(before[n_decay:], u_ref[n_decay:], 0.02, 0.0, scale=s)])
        got = torch.cat([p.detach().reshape(-1) for p in order]).cpu().numpy().astype(np.float64)
        step_len = np.linalg.norm(want - before)
        assert np.linalg.norm(got - want) <= 1e-4 * step_len + 4 * EPS * np.linalg.norm(want)
    assert losses[-1] < losses[0]  # the preconditioned steps reduce the training loss
    assert opt.handle.status() == 0
    # parameters are views of one flat vector: the model sees the library's in-place update
    assert all(p.data_ptr() >= opt._theta.data_ptr() for p in order)
    cpu.close()


@pytest.mark.parametrize("flags_name,block,off", [("", 0, 0), ("", 0, 1), ("RHS_ACCUMULATOR", 0, 0),
                                                   ("VALUES_BF16", 4096, 0)])
def test_step_apply_without_materialising_u(flags_name, block, off):
    """update = NULL: the linear combination updates theta slab by slab."""
    B = _binding()
    flags = getattr(B, flags_name) if flags_name else 0
    d, m, k, lam = 150_001, 6, 1500, 1e-3
    eta, gamma = 0.03, 0.02
    rng = np.random.default_rng(8)
    gpu = B.Efcp(d, m, k, lam, flags, block)
    cpu = ref.RefEFCP(d, m, k, lam, flags, block)
    theta = rng.standard_normal(d).astype(np.float32)
    tbuf = torch.empty(d + 1, device="cuda")
    t_dev = tbuf[off:d + off]  # off = 1: a parameter vector that is not 16-byte aligned
    t_dev.copy_(torch.from_numpy(theta))
    g_dev = torch.empty(d, device="cuda")
    for t in range(9):
        g = rng.standard_normal(d).astype(np.float32)
        g_dev.copy_(torch.from_numpy(g))
        before = t_dev.cpu().numpy()
        gpu.step_apply(g_dev, t_dev, None, eta, gamma)
        u_ref = cpu.step(g)
        want = wrapper.apply_update(before, u_ref, eta, gamma)
        got = t_dev.cpu().numpy().astype(np.float64)
        step_len = np.linalg.norm(want - before)
        assert np.linalg.norm(got - want) <= 1e-4 * step_len + 4 * EPS * np.linalg.norm(want), t
        assert np.array_equal(gpu.error().view(np.uint32), cpu.error().view(np.uint32))
    assert gpu.status() == 0 and gpu.validate() == 0
    with pytest.raises(B.EfcpError) as ei:  # clipping needs u
        gpu.step_apply(g_dev, t_dev, None, eta, gamma, 1.0)
    assert ei.value.code == B.EINVAL
    assert gpu.step_count == 9  # the rejected call did not step
    gpu.close()
    cpu.close()
