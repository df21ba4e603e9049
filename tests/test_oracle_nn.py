"""Pins for the oracle's network step: gradients, losses, optimisers, eval.

Independent references used here: PyTorch CPU autograd in float64 (a library
routine), central finite differences, pure-Python triple loops, closed forms
of the optimiser recurrences, and closed-form energy distances.
"""
import math

import numpy as np
import pytest
import torch

from oracle import pbt_oracle as O
from workloads import configs as C
from workloads.generate import Inputs


def _mlp_cfg(loss, widths, dtype=C.FP32, opt=C.OPT_SGDM, n=2, batch=6, slots=None, **kw):
    if slots is None:
        slots = ("lr", "momentum") if opt == C.OPT_SGDM else ("lr", "beta1", "wd")
    nh = len(slots)
    return C.PBTConfig(name="t", n_members=n, dtype=dtype, model=C.MLP, loss=loss, optimizer=opt,
                       widths=(tuple(widths),), batch=batch, eval_batch=batch, pool_rows=batch,
                       slots=slots, priors=(("fixed", 0, 0),) * nh, perturb=(True,) * nh,
                       clamp_lo=(-math.inf,) * nh, clamp_hi=(math.inf,) * nh, **kw)


def _inputs(cfg, rng, h):
    w = cfg.widths[0]
    x = rng.standard_normal((cfg.pool_rows, w[0])).astype(np.float32)
    if cfg.loss == C.LOSS_MSE:
        y = rng.standard_normal((cfg.pool_rows, w[-1])).astype(np.float32)
    elif cfg.loss == C.LOSS_CE_HARD:
        y = rng.integers(0, w[-1], size=cfg.pool_rows).astype(np.int32)
    else:
        t = rng.random((cfg.pool_rows, w[-1]))
        y = (t / t.sum(axis=1, keepdims=True) * 0.97).astype(np.float32)   # deliberately not summing to 1
    hp = np.tile(np.asarray(h, dtype=np.float64), (cfg.n_members, 1))
    return Inputs(init_hparams=hp, x_pool=x, y_pool=y, x_eval=x, y_eval=y)


def _torch_loss(cfg, Ws, bs, x, y):
    a = torch.tensor(np.asarray(x, dtype=np.float64))
    for i, (w, b) in enumerate(zip(Ws, bs)):
        a = a @ w.T + b
        if i + 1 < len(Ws):
            a = torch.relu(a)
    if cfg.loss == C.LOSS_MSE:
        return ((a - torch.tensor(np.asarray(y, dtype=np.float64))) ** 2).sum(dim=1).mean()
    if cfg.loss == C.LOSS_CE_HARD:
        return torch.nn.functional.cross_entropy(a, torch.tensor(np.asarray(y, dtype=np.int64)))
    t = torch.tensor(np.asarray(y, dtype=np.float64))
    return -(t * torch.log_softmax(a, dim=1)).sum(dim=1).mean()


@pytest.mark.parametrize("loss", [C.LOSS_MSE, C.LOSS_CE_HARD, C.LOSS_CE_SOFT])
def test_mlp_gradient_matches_torch_autograd(loss):
    rng = np.random.default_rng(3)
    cfg = _mlp_cfg(loss, (5, 7, 6, 4))
    inp = _inputs(cfg, rng, [0.0, 0.0])          # lr = 0: the step only records the gradient
    pop = O.Population(cfg, inp, seed=5)
    for m in range(cfg.n_members):
        for t in range(len(pop.shapes)):
            pop.b[m][t] = rng.standard_normal(pop.b[m][t].shape).astype(np.float32)
    pop.step(1)
    for m in range(cfg.n_members):
        Ws = [torch.tensor(w.astype(np.float64), requires_grad=True) for w in pop.W[m]]
        bs = [torch.tensor(b.astype(np.float64), requires_grad=True) for b in pop.b[m]]
        L = _torch_loss(cfg, Ws, bs, inp.x_pool, inp.y_pool)
        L.backward()
        assert abs(float(L) - pop.last_loss[m, 0]) < 1e-12 * max(1.0, abs(float(L)))
        for t in range(len(Ws)):
            np.testing.assert_allclose(pop.gW[m][t], Ws[t].grad.numpy(), rtol=2e-6, atol=1e-9)
            np.testing.assert_allclose(pop.gb[m][t], bs[t].grad.numpy(), rtol=2e-6, atol=1e-9)
        # eval is minus the same loss on the held-out set (here the same rows)
        assert abs(pop.eval_member(m) + float(L)) < 1e-12 * max(1.0, abs(float(L)))


def test_forward_against_triple_loop():
    rng = np.random.default_rng(4)
    cfg = _mlp_cfg(C.LOSS_MSE, (3, 4, 2), batch=3)
    inp = _inputs(cfg, rng, [0.0, 0.0])
    pop = O.Population(cfg, inp, seed=1)
    acts, z = pop.forward(0, 0, inp.x_pool)
    W1, W2 = pop.W[0][0].astype(float), pop.W[0][1].astype(float)
    for r in range(3):
        hid = []
        for o in range(4):
            s = 0.0
            for i in range(3):
                s += float(inp.x_pool[r, i]) * W1[o, i]
            hid.append(max(s + float(pop.b[0][0][o]), 0.0))
        np.testing.assert_allclose(acts[1][r], hid, rtol=1e-14, atol=1e-300)
        for o in range(2):
            s = 0.0
            for i in range(4):
                s += hid[i] * W2[o, i]
            assert abs(z[r, o] - s - float(pop.b[0][1][o])) < 1e-13


def test_single_linear_layer_first_step_and_least_squares_limit():
    """One linear layer, mean-squared error, plain gradient descent on the full batch:
    from W = 0 the first step is W = lr (2/B) Y^T X exactly, and the iteration
    converges to the least-squares solution of the normal equations."""
    rng = np.random.default_rng(5)
    cfg = _mlp_cfg(C.LOSS_MSE, (4, 2), batch=32, n=1)
    inp = _inputs(cfg, rng, [0.05, 0.0])
    pop = O.Population(cfg, inp, seed=0)
    pop.W[0][0][:] = 0.0
    pop.step(1)
    X, Y = inp.x_pool.astype(np.float64), inp.y_pool.astype(np.float64)
    np.testing.assert_allclose(pop.W[0][0], 0.05 * 2.0 / 32 * Y.T @ X, rtol=1e-6)
    np.testing.assert_allclose(pop.b[0][0], 0.05 * 2.0 / 32 * Y.sum(axis=0), rtol=1e-6)
    pop.step(3000)
    A = np.concatenate([X, np.ones((32, 1))], axis=1)
    sol = np.linalg.lstsq(A, Y, rcond=None)[0]
    np.testing.assert_allclose(pop.W[0][0], sol[:4].T, atol=2e-4)
    np.testing.assert_allclose(pop.b[0][0], sol[4], atol=2e-4)


def test_sgdm_hand_trajectory():
    # g = 1, lr = 0.1, mu = 0.9: v = 1, 1.9, 2.71; theta = -0.1, -0.29, -0.561
    th, v = np.array([0.0]), np.array([0.0])
    seen = []
    for _ in range(3):
        th, v = O.sgdm_update(th, v, np.array([1.0]), 0.1, 0.9)
        seen.append((float(th[0]), float(v[0])))
    np.testing.assert_allclose(seen, [(-0.1, 1.0), (-0.29, 1.9), (-0.561, 2.71)], rtol=1e-14)


def test_adam_textbook_bias_correction_and_closed_forms():
    rng = np.random.default_rng(6)
    b1, b2, eps, lr = 0.9, 0.999, 1e-8, 1e-2
    g = rng.standard_normal((7, 5))
    th, m, v = rng.standard_normal(5), np.zeros(5), np.zeros(5)
    th_ref = th.copy()
    c1 = c2 = 1.0
    for t in range(1, 8):
        c1, c2 = c1 * b1, c2 * b2
        th, m, v = O.adam_update(th, m, v, g[t - 1], lr, b1, b2, eps, 0.0, c1, c2)
        # explicit sums: m_t = (1-b1) sum_i b1^(t-i) g_i, v_t likewise with g^2
        m_sum = (1 - b1) * sum(b1 ** (t - i) * g[i - 1] for i in range(1, t + 1))
        v_sum = (1 - b2) * sum(b2 ** (t - i) * g[i - 1] ** 2 for i in range(1, t + 1))
        th_ref = th_ref - lr * (m_sum / (1 - b1 ** t)) / (np.sqrt(v_sum / (1 - b2 ** t)) + eps)
        np.testing.assert_allclose(m, m_sum, rtol=1e-12)
        np.testing.assert_allclose(v, v_sum, rtol=1e-12)
        np.testing.assert_allclose(th, th_ref, rtol=1e-12)
    # constant gradient: every step moves by lr * sign(g)
    th, m, v, c1, c2 = np.array([0.0, 0.0]), np.zeros(2), np.zeros(2), 1.0, 1.0
    for t in range(1, 6):
        c1, c2 = c1 * b1, c2 * b2
        th, m, v = O.adam_update(th, m, v, np.array([3.0, -0.2]), lr, b1, b2, eps, 0.0, c1, c2)
        np.testing.assert_allclose(th, [-t * lr, t * lr], rtol=1e-6)
    # zero gradient: decoupled weight decay only, theta_t = theta_0 (1 - lr wd)^t
    th, m, v = np.array([2.0]), np.zeros(1), np.zeros(1)
    for t in range(1, 5):
        th, m, v = O.adam_update(th, m, v, np.zeros(1), lr, b1, b2, eps, 0.1, b1 ** t, b2 ** t)
        np.testing.assert_allclose(th, 2.0 * (1 - lr * 0.1) ** t, rtol=1e-14)


def test_population_adam_uses_running_products_of_a_changing_beta1():
    rng = np.random.default_rng(7)
    cfg = _mlp_cfg(C.LOSS_CE_HARD, (4, 3), opt=C.OPT_ADAM, n=1, batch=8)
    inp = _inputs(cfg, rng, [1e-2, 0.9, 0.0])
    pop = O.Population(cfg, inp, seed=2)
    pop.step(1)
    pop.H[0, 1] = np.float32(0.8)
    pop.step(1)
    c1 = np.float32(np.float32(0.9) * np.float32(0.8))
    c2 = np.float32(np.float32(0.999) * np.float32(0.999))
    assert pop.scalars[0, 0] == c1 and pop.scalars[0, 1] == c2
    assert list(pop.scalars[0, 2:]) == [1.0, 1.0]


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(8)
    a = np.concatenate([rng.standard_normal(4096) * 10 ** rng.uniform(-6, 6, 4096),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40]]).astype(np.float32)
    ref = torch.tensor(a).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.round_bf16(a), ref)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert O.round_bf16(np.array([1.00390625]))[0] == 1.0
    assert O.round_bf16(np.array([1.01171875]))[0] == 1.015625


def test_bf16_population_rounds_gemm_operands_only():
    rng = np.random.default_rng(9)
    cfg = _mlp_cfg(C.LOSS_CE_SOFT, (6, 5, 4), dtype=C.BF16, opt=C.OPT_ADAM, n=1, batch=8)
    inp = _inputs(cfg, rng, [1e-3, 0.9, 0.0])
    pop = O.Population(cfg, inp, seed=3)
    acts, z = pop.forward(0, 0, pop.q(inp.x_pool))
    for a in acts:
        np.testing.assert_array_equal(a, O.round_bf16(a))
    assert not np.array_equal(z, O.round_bf16(z))        # logits stay unrounded
    assert pop.W[0][0].dtype == np.float32               # masters stay float32
    assert not np.array_equal(pop.W[0][0].astype(np.float64), O.round_bf16(pop.W[0][0]))


def _ring(k):
    return np.array([math.cos(2 * math.pi * k / 8), math.sin(2 * math.pi * k / 8)])


def test_energy_distance_special_cases():
    on_modes = np.array([_ring(k) for k in range(8)] * 3)
    assert abs(O.energy_distance_to_ring(on_modes)) < 1e-14
    # all mass at the origin: E = 2 * 1 - 0 - (1/64) * 16 cot(pi/16)
    e0 = O.energy_distance_to_ring(np.zeros((5, 2)))
    assert abs(e0 - (2.0 - 0.25 / math.tan(math.pi / 16))) < 1e-13
    rng = np.random.default_rng(10)
    x = rng.standard_normal((17, 2))
    e = O.energy_distance_to_ring(x)
    assert e > 0
    c, s = math.cos(math.pi / 4), math.sin(math.pi / 4)
    rot = x @ np.array([[c, s], [-s, c]])
    assert abs(O.energy_distance_to_ring(rot) - e) < 1e-13      # the ring is invariant under 45 degrees
    mu = [_ring(k) for k in range(8)]
    cross = sum(math.dist(xi, m) for xi in x for m in mu) / (17 * 8)
    within = sum(math.dist(xi, xj) for xi in x for xj in x) / 17 ** 2
    modes = sum(math.dist(a, b) for a in mu for b in mu) / 64
    assert abs(e - (2 * cross - within - modes)) < 1e-13


def _gan_cfg():
    return C.PBTConfig(name="g", n_members=1, dtype=C.FP32, model=C.GAN, loss=C.LOSS_GAN,
                       optimizer=C.OPT_ADAM, widths=((3, 5, 2), (2, 6, 4, 1)), batch=8, eval_batch=8,
                       pool_rows=8, gan_d_steps=2, slots=("lr", "lr_d"),
                       priors=(("fixed", 0, 0),) * 2, perturb=(True, True),
                       clamp_lo=(-math.inf,) * 2, clamp_hi=(math.inf,) * 2, beta1=0.5)


def test_gan_gradients_match_torch_autograd():
    rng = np.random.default_rng(11)
    cfg = _gan_cfg()
    inp = Inputs(init_hparams=np.zeros((1, 2)),     # both learning rates 0: gradients only
                 x_pool=rng.standard_normal((8, 2)).astype(np.float32),
                 z_pool=rng.standard_normal((8, 3)).astype(np.float32),
                 x_eval=rng.standard_normal((8, 3)).astype(np.float32))
    pop = O.Population(cfg, inp, seed=4)
    for t in range(len(pop.shapes)):
        pop.b[0][t] = (0.1 * rng.standard_normal(pop.b[0][t].shape)).astype(np.float32)
    pop.step(1)
    Ws = [torch.tensor(w.astype(np.float64), requires_grad=True) for w in pop.W[0]]
    bs = [torch.tensor(b.astype(np.float64), requires_grad=True) for b in pop.b[0]]

    def net(a, idx):
        for n, t in enumerate(idx):
            a = a @ Ws[t].T + bs[t]
            if n + 1 < len(idx):
                a = torch.relu(a)
        return a

    z = torch.tensor(inp.z_pool.astype(np.float64))
    real = torch.tensor(inp.x_pool.astype(np.float64))
    sp = torch.nn.functional.softplus
    fake = net(z, [0, 1])
    LD = sp(-net(real, [2, 3, 4])).mean() + sp(net(fake.detach(), [2, 3, 4])).mean()
    LD.backward()
    assert abs(float(LD) - pop.last_loss[0, 1]) < 1e-12
    for t in (2, 3, 4):
        np.testing.assert_allclose(pop.gW[0][t], Ws[t].grad.numpy(), rtol=2e-6, atol=1e-9)
        np.testing.assert_allclose(pop.gb[0][t], bs[t].grad.numpy(), rtol=2e-6, atol=1e-9)
    for p in Ws + bs:
        p.grad = None
    LG = sp(-net(net(z, [0, 1]), [2, 3, 4])).mean()
    LG.backward()
    assert abs(float(LG) - pop.last_loss[0, 0]) < 1e-12
    for t in (0, 1):
        np.testing.assert_allclose(pop.gW[0][t], Ws[t].grad.numpy(), rtol=2e-6, atol=1e-9)
        np.testing.assert_allclose(pop.gb[0][t], bs[t].grad.numpy(), rtol=2e-6, atol=1e-9)
    # K discriminator updates and one generator update advanced the right products
    assert pop.scalars[0, 0] == np.float32(0.5) and pop.scalars[0, 2] == np.float32(0.25)


def test_gan_finite_difference_of_generator_loss():
    rng = np.random.default_rng(12)
    cfg = _gan_cfg()
    inp = Inputs(init_hparams=np.zeros((1, 2)),
                 x_pool=rng.standard_normal((8, 2)).astype(np.float32),
                 z_pool=rng.standard_normal((8, 3)).astype(np.float32),
                 x_eval=rng.standard_normal((8, 3)).astype(np.float32))
    pop = O.Population(cfg, inp, seed=5)
    pop.step(1)
    g = pop.gW[0][0].copy()

    def LG():
        _, out = pop.forward(0, 0, inp.z_pool)
        _, d = pop.forward(0, 1, out)
        return O.softplus(-d.reshape(-1)).mean()

    W0 = pop.W[0][0].astype(np.float64)
    for (o, i) in [(0, 0), (2, 1), (4, 2)]:
        e = 1e-6
        Wp, Wm = W0.copy(), W0.copy()
        Wp[o, i] += e
        Wm[o, i] -= e
        pop.W[0][0] = Wp
        lp = LG()
        pop.W[0][0] = Wm
        lm = LG()
        assert abs((lp - lm) / (2 * e) - g[o, i]) < 1e-6 * max(1.0, abs(g[o, i]))


def test_grouped_gemm_against_triple_loop():
    rng = np.random.default_rng(13)
    A, B = rng.standard_normal((2, 3, 5)), rng.standard_normal((2, 4, 5))
    bias, mask = rng.standard_normal((2, 4)), rng.standard_normal((2, 3, 4))
    mask[0, 1, 2] = 0.0
    got = O.grouped_gemm(A, B, bias, True, mask)
    for b in range(2):
        for m in range(3):
            for n in range(4):
                s = sum(A[b, m, k] * B[b, n, k] for k in range(5)) + bias[b, n]
                s = max(s, 0.0) if mask[b, m, n] > 0 else 0.0
                assert abs(got[b, m, n] - s) < 1e-13
    plain = O.grouped_gemm(A, B)
    assert abs(plain[1, 2, 3] - float(A[1, 2] @ B[1, 3])) < 1e-13


def test_rmsprop_hand_trajectory_and_torch_optimizer():
    # g = 1, rho = 0.9, lr = 0.1, eps = 0: ms = 0.1, 0.19; theta = -0.1/sqrt(0.1), then - 0.1/sqrt(0.19) more
    th, ms = np.array([0.0]), np.array([0.0])
    th, ms = O.rmsprop_update(th, ms, np.array([1.0]), 0.1, 0.9, 0.0)
    assert abs(ms[0] - 0.1) < 1e-15 and abs(th[0] + 0.1 / math.sqrt(0.1)) < 1e-15
    th, ms = O.rmsprop_update(th, ms, np.array([1.0]), 0.1, 0.9, 0.0)
    assert abs(ms[0] - 0.19) < 1e-15 and abs(th[0] + 0.1 / math.sqrt(0.1) + 0.1 / math.sqrt(0.19)) < 1e-15
    # against torch.optim.RMSprop (no momentum, not centred) on a random gradient sequence
    rng = np.random.default_rng(21)
    g = rng.standard_normal((6, 5))
    w = torch.zeros(5, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.RMSprop([w], lr=3e-3, alpha=0.99, eps=1e-8)
    th, ms = np.zeros(5), np.zeros(5)
    for t in range(6):
        w.grad = torch.tensor(g[t])
        opt.step()
        th, ms = O.rmsprop_update(th, ms, g[t], 3e-3, 0.99, 1e-8)
        np.testing.assert_allclose(th, w.detach().numpy(), rtol=1e-12, atol=1e-15)


def test_rmsprop_population_step_uses_the_gradient_of_the_loss():
    rng = np.random.default_rng(22)
    cfg = _mlp_cfg(C.LOSS_MSE, (4, 3, 2), n=1, batch=8).replace(optimizer=C.OPT_RMSPROP, slots=("lr",),
                                                                priors=(("fixed", 0, 0),), perturb=(True,),
                                                                clamp_lo=(-math.inf,), clamp_hi=(math.inf,), beta2=0.9)
    inp = _inputs(cfg, rng, [1e-2])
    pop = O.Population(cfg, inp, seed=3)
    w0 = pop.W[0][0].astype(np.float64).copy()
    pop.step(1)
    g = pop.gW[0][0].astype(np.float64)
    expect = w0 - 1e-2 * g / (np.sqrt(0.1 * g * g) + float(np.float32(1e-8)))
    np.testing.assert_allclose(pop.W[0][0], expect, rtol=2e-6, atol=1e-9)
    np.testing.assert_allclose(pop.o1W[0][0], np.float32(1.0 - np.float32(0.9)) * g * g, rtol=2e-6)


def test_plain_sgd_is_gradient_descent_and_the_zero_momentum_limit():
    """Section 3's example of `step`: theta <- theta - lr * gradient.  Pinned three ways: the update function on a
    hand trajectory; one population step against torch.optim.SGD on the same network and batch; and SGD with
    momentum 0, which takes the same steps."""
    th = np.array([1.0, -2.0])
    for _ in range(3):                       # gradient of (1/2)|theta|^2 is theta: theta shrinks by (1 - lr) per step
        th = O.sgd_update(th, th, 0.25)
    np.testing.assert_allclose(th, np.array([1.0, -2.0]) * 0.75 ** 3, rtol=1e-15)

    rng = np.random.default_rng(8)
    cfg = _mlp_cfg(C.LOSS_MSE, (5, 7, 3), batch=16, n=1, opt=C.OPT_SGD, slots=("lr",))
    inp = _inputs(cfg, rng, [0.05])
    pop = O.Population(cfg, inp, seed=0)
    for b in pop.b[0]:
        b[:] = rng.standard_normal(b.shape).astype(np.float32) * 0.1
    Ws = [torch.tensor(w.astype(np.float64), requires_grad=True) for w in pop.W[0]]
    bs = [torch.tensor(b.astype(np.float64), requires_grad=True) for b in pop.b[0]]
    opt = torch.optim.SGD(Ws + bs, lr=0.05)
    for _ in range(3):
        opt.zero_grad()
        _torch_loss(cfg, Ws, bs, inp.x_pool, inp.y_pool).backward()
        opt.step()
        pop.step(1)
    for w, tw in zip(pop.W[0] + pop.b[0], Ws + bs):
        np.testing.assert_allclose(w, tw.detach().numpy(), rtol=2e-6, atol=1e-7)
    assert not any(o.any() for o in pop.o1W[0] + pop.o1b[0])          # no optimiser state is kept

    mom = O.Population(_mlp_cfg(C.LOSS_MSE, (5, 7, 3), batch=16, n=1, opt=C.OPT_SGDM, slots=("lr", "momentum")),
                       _inputs(cfg, np.random.default_rng(8), [0.05, 0.0]), seed=0)
    ref = O.Population(cfg, _inputs(cfg, np.random.default_rng(8), [0.05]), seed=0)
    mom.step(3)
    ref.step(3)
    for a, b in zip(mom.W[0] + mom.b[0], ref.W[0] + ref.b[0]):
        np.testing.assert_array_equal(a, b)
