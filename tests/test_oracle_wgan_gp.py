"""Pins for the oracle's WGAN-GP step (Section 4.3.1): the critic's objective and its gradient (which needs the
derivative of an input gradient) against torch float64 double back-propagation, finite differences and the
closed form of a linear critic; the generator's gradient; the interpolation coefficients."""
import math

import numpy as np
import pytest
import torch

from oracle import pbt_oracle as O
from oracle import philox as px
from workloads import configs as C
from workloads.generate import Inputs


def _cfg(d=(2, 6, 4, 1), dtype=C.FP32, k=2):
    return C.PBTConfig(name="w", n_members=1, dtype=dtype, model=C.GAN, loss=C.LOSS_WGAN_GP,
                       optimizer=C.OPT_ADAM, widths=((3, 5, 2), tuple(d)), batch=8, eval_batch=8,
                       pool_rows=8, gan_d_steps=k, slots=("lr", "lr_d"),
                       priors=(("fixed", 0, 0),) * 2, perturb=(True, True),
                       clamp_lo=(-math.inf,) * 2, clamp_hi=(math.inf,) * 2, beta1=0.5, gp_lambda=10.0)


def _pop(cfg, seed, rng, lr=0.0):
    inp = Inputs(init_hparams=np.full((1, 2), lr),
                 x_pool=rng.standard_normal((8, 2)).astype(np.float32),
                 z_pool=rng.standard_normal((8, 3)).astype(np.float32),
                 x_eval=rng.standard_normal((8, 3)).astype(np.float32))
    pop = O.Population(cfg, inp, seed=seed)
    for t in range(len(pop.shapes)):
        pop.b[0][t] = (0.1 * rng.standard_normal(pop.b[0][t].shape)).astype(np.float32)
    return pop, inp


def _torch_critic_loss(Ws, bs, idx, real, fake, eps, lam):
    def D(a):
        for n, t in enumerate(idx):
            a = a @ Ws[t].T + bs[t]
            if n + 1 < len(idx):
                a = torch.relu(a)
        return a
    xhat = (eps[:, None] * real + (1 - eps[:, None]) * fake).detach().requires_grad_(True)
    gx, = torch.autograd.grad(D(xhat).sum(), xhat, create_graph=True)
    pen = ((gx.norm(dim=1) - 1.0) ** 2).mean()
    return D(fake).mean() - D(real).mean() + lam * pen


@pytest.mark.parametrize("d", [(2, 6, 4, 1), (2, 7, 1), (2, 5, 6, 3, 1)])
def test_critic_loss_and_gradient_match_torch_double_backward(d):
    rng = np.random.default_rng(21)
    cfg = _cfg(d)
    pop, _ = _pop(cfg, 4, rng)
    real = rng.standard_normal((8, 2))
    fake = rng.standard_normal((8, 2)) * 0.7 + 0.3
    eps = rng.random(8)
    loss, gW, gb, xhat = pop.wgan_gp_critic(0, real, fake, eps, 10.0)
    idx = pop._tensors_of_stack(1)
    Ws = {t: torch.tensor(pop.W[0][t].astype(np.float64), requires_grad=True) for t in idx}
    bs = {t: torch.tensor(pop.b[0][t].astype(np.float64), requires_grad=True) for t in idx}
    L = _torch_critic_loss(Ws, bs, idx, torch.tensor(real), torch.tensor(fake), torch.tensor(eps), 10.0)
    L.backward()
    assert abs(float(L.detach()) - loss) < 1e-12 * max(1.0, abs(loss))
    np.testing.assert_allclose(xhat, eps[:, None] * real + (1 - eps[:, None]) * fake, rtol=0, atol=1e-15)
    for t in idx:
        np.testing.assert_allclose(gW[t], Ws[t].grad.numpy(), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(gb[t], bs[t].grad.numpy(), rtol=1e-10, atol=1e-12)


def test_critic_gradient_by_finite_differences():
    rng = np.random.default_rng(22)
    pop, _ = _pop(_cfg(), 5, rng)
    real, fake, eps = rng.standard_normal((8, 2)), rng.standard_normal((8, 2)), rng.random(8)
    _, gW, gb, _ = pop.wgan_gp_critic(0, real, fake, eps, 10.0)
    idx = pop._tensors_of_stack(1)
    for t in idx:
        W0 = pop.W[0][t].astype(np.float64)
        for _ in range(3):
            o, i = rng.integers(0, W0.shape[0]), rng.integers(0, W0.shape[1])
            e = 1e-6
            Wp, Wm = W0.copy(), W0.copy()
            Wp[o, i] += e
            Wm[o, i] -= e
            pop.W[0][t] = Wp
            lp = pop.wgan_gp_critic(0, real, fake, eps, 10.0)[0]
            pop.W[0][t] = Wm
            lm = pop.wgan_gp_critic(0, real, fake, eps, 10.0)[0]
            pop.W[0][t] = W0
            assert abs((lp - lm) / (2 * e) - gW[t][o, i]) < 2e-6 * max(1.0, abs(gW[t][o, i]))


def test_linear_critic_closed_form():
    # D(x) = w.x + b: grad_x D = w everywhere, penalty = lam (||w|| - 1)^2, independent of the data
    rng = np.random.default_rng(23)
    pop, _ = _pop(_cfg(d=(2, 1)), 6, rng)
    t = pop._tensors_of_stack(1)[0]
    pop.W[0][t] = np.array([[0.6, -1.7]])
    real, fake, eps = rng.standard_normal((8, 2)), rng.standard_normal((8, 2)), rng.random(8)
    loss, gW, gb, _ = pop.wgan_gp_critic(0, real, fake, eps, 10.0)
    w = pop.W[0][t].astype(np.float64).reshape(-1)
    n = np.linalg.norm(w)
    want_loss = (fake @ w).mean() - (real @ w).mean() + 10.0 * (n - 1.0) ** 2
    want_g = fake.mean(axis=0) - real.mean(axis=0) + 2 * 10.0 * (n - 1.0) * w / n
    assert abs(loss - want_loss) < 1e-12
    np.testing.assert_allclose(gW[t].reshape(-1), want_g, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(gb[t], [0.0], atol=1e-15)          # +1/B per fake row, -1/B per real row
    # lam = 0 leaves the Wasserstein estimate alone
    l0, g0, _, _ = pop.wgan_gp_critic(0, real, fake, eps, 0.0)
    assert abs(l0 - ((fake @ w).mean() - (real @ w).mean())) < 1e-12
    np.testing.assert_allclose(g0[t].reshape(-1), fake.mean(axis=0) - real.mean(axis=0), rtol=1e-12, atol=1e-14)


def test_whole_step_critic_then_generator_against_torch():
    rng = np.random.default_rng(24)
    cfg = _cfg(k=1)
    pop, inp = _pop(cfg, 7, rng, lr=0.0)       # learning rates 0: the step only produces gradients and losses
    pop.step(1)
    Ws = {t: torch.tensor(pop.W[0][t].astype(np.float64), requires_grad=True) for t in range(len(pop.shapes))}
    bs = {t: torch.tensor(pop.b[0][t].astype(np.float64), requires_grad=True) for t in range(len(pop.shapes))}

    def net(a, idx):
        for n, t in enumerate(idx):
            a = a @ Ws[t].T + bs[t]
            if n + 1 < len(idx):
                a = torch.relu(a)
        return a

    z = torch.tensor(inp.z_pool.astype(np.float64))
    real = torch.tensor(inp.x_pool.astype(np.float64))
    gi, di = pop._tensors_of_stack(0), pop._tensors_of_stack(1)
    pop.step_count = 0                          # the coefficients of the step just taken
    eps = torch.tensor(pop._interp_eps(0, 0, 8))
    L = _torch_critic_loss(Ws, bs, di, real, net(z, gi).detach(), eps, cfg.gp_lambda)
    L.backward()
    assert abs(float(L.detach()) - pop.last_loss[0, 1]) < 1e-10
    for t in di:
        np.testing.assert_allclose(pop.gW[0][t], Ws[t].grad.numpy(), rtol=2e-6, atol=1e-8)
        np.testing.assert_allclose(pop.gb[0][t], bs[t].grad.numpy(), rtol=2e-6, atol=1e-8)
    for p in list(Ws.values()) + list(bs.values()):
        p.grad = None
    LG = -net(net(z, gi), di).mean()
    LG.backward()
    assert abs(float(LG.detach()) - pop.last_loss[0, 0]) < 1e-12
    for t in gi:
        np.testing.assert_allclose(pop.gW[0][t], Ws[t].grad.numpy(), rtol=2e-6, atol=1e-9)
        np.testing.assert_allclose(pop.gb[0][t], bs[t].grad.numpy(), rtol=2e-6, atol=1e-9)


def test_interpolation_coefficients():
    rng = np.random.default_rng(25)
    pop, _ = _pop(_cfg(), 8, rng)
    e0 = pop._interp_eps(0, 0, 4000)
    assert e0.min() > 0.0 and e0.max() < 1.0
    assert abs(e0.mean() - 0.5) < 0.02 and abs(e0.var() - 1.0 / 12.0) < 0.01
    assert np.array_equal(e0.astype(np.float32).astype(np.float64), e0)     # float32 holds them exactly
    assert not np.array_equal(e0[:8], pop._interp_eps(0, 1, 8))             # keyed by the critic update ...
    pop.step_count = 3
    assert not np.array_equal(e0[:8], pop._interp_eps(0, 0, 8))             # ... and by the step
    # row b uses word b mod 4 of block b div 4
    pop.step_count = 0
    w = px.draw(pop.seed, 0, 0, px.STREAM_INTERP, 1)[2]
    assert e0[6] == ((w >> 9) + 0.5) / 2 ** 23


def test_bf16_critic_stays_close_to_the_unrounded_one():
    rng = np.random.default_rng(26)
    real, fake, eps = rng.standard_normal((8, 2)), rng.standard_normal((8, 2)), rng.random(8)
    out = []
    for dt in (C.FP32, C.BF16):
        pop, _ = _pop(_cfg(dtype=dt), 9, np.random.default_rng(3))
        out.append(pop.wgan_gp_critic(0, O.round_bf16(real), O.round_bf16(fake), eps, 10.0))
    (l0, g0, b0, _), (l1, g1, b1, _) = out
    assert abs(l0 - l1) < 3e-2 * max(1.0, abs(l0))
    for t in g0:
        assert np.linalg.norm(g0[t] - g1[t]) < 5e-2 * np.linalg.norm(g0[t])


def test_training_reduces_the_critic_loss_and_moves_the_generator():
    rng = np.random.default_rng(27)
    pop, _ = _pop(_cfg(k=5), 10, rng, lr=2e-3)
    w_g = [w.copy() for w in pop.W[0]]
    losses = []
    for _ in range(40):
        pop.step(1)
        losses.append(pop.last_loss[0, 1])
    assert np.isfinite(losses).all()
    assert np.mean(losses[-5:]) < np.mean(losses[:5])                        # the critic learns
    assert any(not np.array_equal(a, b) for a, b in zip(w_g, pop.W[0]))
