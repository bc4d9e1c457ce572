"""GPU parity of the calls either side of the trellis pass (computed table, Adam, fused backward + update)."""
import numpy as np
import pytest

import oracle
from oracle import qat_oracle as qo

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2605_10655_b200 import Context
    c = Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("Lb", [1, 4, 8, 16])
def test_gaussian_table_matches_the_inverse_normal_cdf(ctx, Lb):
    got = ctx.bcjr_gaussian_codebook(Lb).cpu().numpy().astype(np.float64)
    ref = qo.gaussian_codebook(Lb)
    # single-precision inverse CDF: a few ulp of the value, plus the rounding of the argument
    # ((s + 1/2)/S to float32), which the slope 1/phi(c) magnifies in the tails
    tol = 4e-6 * np.maximum(1.0, np.abs(ref)) + 6e-8 / np.maximum(np.exp(-0.5 * ref ** 2) / np.sqrt(2 * np.pi), 1e-30) * ((np.arange(1 << Lb) + 0.5) / (1 << Lb)).clip(max=0.5)
    assert np.all(np.abs(got - ref) <= tol), float(np.abs(got - ref).max())
    np.testing.assert_array_equal(got, -got[::-1])                       # exactly antisymmetric
    assert np.all(np.diff(got) >= 0)


@pytest.mark.parametrize("numel", [1, 3, 4, 1023, 4096, 1 << 20 | 5])
def test_adam_update_matches_the_textbook_rule(ctx, numel):
    import torch
    rng = np.random.default_rng(numel)
    dev = torch.device("cuda", ctx.device)
    p0 = rng.standard_normal(numel).astype(np.float32)
    p = torch.from_numpy(p0.copy()).to(dev); m = torch.zeros(numel, device=dev); v = torch.zeros(numel, device=dev)
    rp, rm, rv = p0.astype(np.float64), np.zeros(numel), np.zeros(numel)
    gmax = np.zeros(numel)
    for t in range(1, 6):
        g = (rng.standard_normal(numel) * 10.0 ** rng.integers(-4, 2, numel)).astype(np.float32)
        ctx.bcjr_adam_update(p, torch.from_numpy(g).to(dev), m, v, t, lr=1e-2, beta1=0.9, beta2=0.99, eps=1e-8)
        rp, rm, rv = qo.adam_update(rp, g, rm, rv, t, 1e-2, 0.9, 0.99, 1e-8)
        gmax = np.maximum(gmax, np.abs(g))
    ctx.sync_status()
    np.testing.assert_allclose(p.cpu().numpy(), rp, rtol=2e-5, atol=2e-6)
    # the moments are sums of float32 terms of either sign: absolute error of a few ulp of the largest term
    assert np.all(np.abs(m.cpu().numpy() - rm) <= 1e-5 * np.abs(rm) + 3e-7 * gmax)
    assert np.all(np.abs(v.cpu().numpy() - rv) <= 1e-5 * np.abs(rv) + 3e-7 * gmax ** 2)


def test_adam_rejects_bad_arguments(ctx):
    import torch
    from paper_2605_10655_b200 import BcjrError
    dev = torch.device("cuda", ctx.device)
    x = torch.zeros(9, device=dev)
    with pytest.raises(BcjrError) as e:
        ctx.bcjr_adam_update(x, x, x, x, 0, 1e-3)                    # steps count from 1
    assert e.value.code == -1
    with pytest.raises(BcjrError) as e:
        ctx.bcjr_adam_update(x[1:], x[1:], x[1:], x[1:], 1, 1e-3)    # not 16-byte aligned
    assert e.value.code == -1


def test_annealed_qat_loop_follows_the_oracle_loop(ctx):
    # Algorithm 1 on one small matrix with a weight-space loss l = mean((soft - target)^2) standing in
    # for the layer-output loss: schedule -> soft codeword -> grad_soft -> backward -> Adam on the
    # latent weights and on the table, five steps; the oracle runs the same loop in float64
    import torch
    from paper_2605_10655_b200 import binding
    Lb, k, n, B, N = 8, 2, 32, 12, 5
    rng = np.random.default_rng(77)
    W0 = rng.standard_normal((B, n)).astype(np.float32)
    target = (W0 + 0.3 * rng.standard_normal((B, n))).astype(np.float32)
    dev = torch.device("cuda", ctx.device)
    c0 = qo.gaussian_codebook(Lb).astype(np.float32)          # both sides start from the oracle's table
    c_dev = torch.from_numpy(c0.copy()).to(dev)
    W = torch.from_numpy(W0.copy()).to(dev); tgt = torch.from_numpy(target).to(dev)
    mW = torch.zeros_like(W); vW = torch.zeros_like(W); mc = torch.zeros_like(c_dev); vc = torch.zeros_like(c_dev)
    rW, rc = W0.astype(np.float64), c0.astype(np.float64)
    rmW = np.zeros_like(rW); rvW = np.zeros_like(rW); rmc = np.zeros_like(rc); rvc = np.zeros_like(rc)
    losses, rlosses = [], []
    for t in range(1, N + 1):
        T = binding.temperature(1.0, 0.05, t, N)
        assert abs(T - qo.temperature(1.0, 0.05, t, N)) < 1e-15
        soft, _ = ctx.bcjr_soft_quantize(W, c_dev, Lb, k, n, T)
        g = 2.0 * (soft - tgt) / soft.numel()
        losses.append(float(((soft - tgt) ** 2).mean()))
        ctx.bcjr_backward_adam(g, mW, vW, t, lr_W=1e-2, m_c=mc, v_c=vc, lr_c=1e-3)
        rsoft = oracle.soft_quantize(rW, rc, Lb, k, T)["soft"]
        rg = 2.0 * (rsoft - target) / rsoft.size
        rlosses.append(float(((rsoft - target) ** 2).mean()))
        rb = oracle.backward(rW, rc, rg, Lb, k, T)
        rW, rmW, rvW = qo.adam_update(rW, rb["grad_W"], rmW, rvW, t, 1e-2)
        rc, rmc, rvc = qo.adam_update(rc, rb["grad_codebook"], rmc, rvc, t, 1e-3)
    assert ctx.sync_status().device_status == 0
    np.testing.assert_allclose(losses, rlosses, rtol=2e-3)
    # Adam's step is lr * sign-like where the gradient is tiny, so compare the trajectories in
    # units of the step size: five steps of 1e-2 (1e-3 for the table)
    assert np.abs(W.cpu().numpy() - rW).max() <= 0.2 * 1e-2 * N
    assert np.abs(c_dev.cpu().numpy() - rc).max() <= 0.2 * 1e-3 * N
    assert np.median(np.abs(W.cpu().numpy() - rW)) <= 1e-5
    # the saved state was consumed
    from paper_2605_10655_b200 import BcjrError
    with pytest.raises(BcjrError) as e:
        ctx.bcjr_backward(g)
    assert e.value.code == -4


@pytest.mark.parametrize("m,n", [(8, 8), (16, 64), (64, 16), (32, 512), (128, 2048), (8, 8192), (2048, 32)])
def test_hadamard_rotation_matches_the_matrix_product_and_inverts(ctx, m, n):
    import torch
    rng = np.random.default_rng(m * 31 + n)
    W = rng.standard_normal((m, n)).astype(np.float32)
    sL = rng.choice([-1.0, 1.0], m).astype(np.float32); sR = rng.choice([-1.0, 1.0], n).astype(np.float32)
    dev = torch.device("cuda", ctx.device)
    Wd, sLd, sRd = (torch.from_numpy(a).to(dev) for a in (W, sL, sR))
    Wt = ctx.bcjr_rht(Wd, sLd, sRd)
    ref = qo.rht_forward(W, sL, sR)                                  # dense matrix products in float64
    # log2(m n) butterfly stages of float32 additions on O(1) values
    assert np.abs(Wt.cpu().numpy() - ref).max() <= 2e-6 * np.abs(ref).max() * np.log2(m * n)
    back = ctx.bcjr_rht(Wt, sLd, sRd, inverse=True)
    assert np.abs(back.cpu().numpy() - W).max() <= 4e-6 * np.abs(W).max() * np.log2(m * n)
    ref_inv = qo.rht_inverse(ref, sL, sR)
    np.testing.assert_allclose(ref_inv, W, atol=1e-5)
    # in place
    Wc = Wd.clone()
    ctx.bcjr_rht(Wc, sLd, sRd, out=Wc)
    ctx.sync_status()
    assert torch.equal(Wc, Wt)


def test_rotation_rejects_sizes_that_are_not_powers_of_two(ctx):
    import torch
    from paper_2605_10655_b200 import BcjrError
    dev = torch.device("cuda", ctx.device)
    W = torch.zeros((24, 16), device=dev); s24 = torch.ones(24, device=dev); s16 = torch.ones(16, device=dev)
    with pytest.raises(BcjrError) as e:
        ctx.bcjr_rht(W, s24, s16)
    assert e.value.code == -1
    W = torch.zeros((8, 16384), device=dev)
    with pytest.raises(BcjrError) as e:
        ctx.bcjr_rht(W, torch.ones(8, device=dev), torch.ones(16384, device=dev))
    assert e.value.code == -5


def test_group_scales_and_their_inverse(ctx):
    import torch
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((37, 64)) * 10.0 ** rng.integers(-3, 3, (37, 1))).astype(np.float32)
    W[5, 16:32] = 0.0                                                # an all-zero group
    dev = torch.device("cuda", ctx.device)
    Wd = torch.from_numpy(W).to(dev)
    scales, Ws = ctx.bcjr_group_scale(Wd)
    rs, rWs = qo.group_scales(np.where(W == 0, 0, W))
    got_s = scales.cpu().numpy().reshape(37, 4)
    np.testing.assert_allclose(got_s, rs, rtol=2e-6)
    mask = np.repeat(rs > 0, 16, axis=1)
    np.testing.assert_allclose(Ws.cpu().numpy()[mask], rWs[mask], rtol=4e-6, atol=1e-7)
    assert torch.all(Ws[5, 16:32] == 0) and got_s[5, 1] == 0
    back = ctx.bcjr_group_unscale(Ws, scales)
    ctx.sync_status()
    np.testing.assert_allclose(back.cpu().numpy(), W, rtol=3e-7, atol=0)
