"""Seeded synthetic inputs for a `PBTConfig` (data only; none of the method).

Everything a run consumes from outside is drawn here, once, from NumPy's
PCG64 generator keyed by (seed, tag): training pools, held-out sets, a fixed
random "teacher" network that labels them, and the initial per-member
hyperparameters sampled from the config's priors.  The arrays are handed
unchanged to the CPU oracle and (after a dtype conversion that is exact) to
the GPU library, so both sides see bit-identical inputs.

Pools of bf16 populations are float32 arrays whose values are exactly
representable in bfloat16.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

from . import configs as C


@dataclass
class Inputs:
    init_hparams: np.ndarray                 # [N, nh] float64 (float32-representable for NN configs)
    x_pool: Optional[np.ndarray] = None      # [pool, in] float32  (GAN: real samples [pool, 2])
    y_pool: Optional[np.ndarray] = None      # mse: [pool, out] f32; ce_hard: [pool] i32; ce_soft: [pool, out] f32
    z_pool: Optional[np.ndarray] = None      # GAN only: generator noise [pool, zdim] float32
    x_eval: Optional[np.ndarray] = None      # [eval, in] float32   (GAN: fixed eval noise [eval, zdim])
    y_eval: Optional[np.ndarray] = None


def _to_bf16_grid(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16-representable float32 (ties to even)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def _rng(seed: int, tag: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tag)])


def _teacher(widths, rng) -> list:
    ws = []
    for i in range(len(widths) - 1):
        fan_in, fan_out = widths[i], widths[i + 1]
        a = np.sqrt(6.0 / fan_in)
        w = rng.uniform(-a, a, size=(fan_out, fan_in)).astype(np.float32)
        b = rng.uniform(-0.1, 0.1, size=(fan_out,)).astype(np.float32)
        ws.append((w, b))
    return ws


def _teacher_forward(ws, x: np.ndarray, chunk: int = 8192) -> np.ndarray:
    outs = []
    for s in range(0, x.shape[0], chunk):
        a = x[s:s + chunk]
        for i, (w, b) in enumerate(ws):
            a = a @ w.T + b
            if i + 1 < len(ws):
                a = np.maximum(a, 0.0)
        outs.append(a.astype(np.float32))
    return np.concatenate(outs, axis=0)


def _softmax(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.float64)
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z)
    return (e / e.sum(axis=1, keepdims=True)).astype(np.float32)


def _init_hparams(cfg: C.PBTConfig, rng) -> np.ndarray:
    n, nh = cfg.n_members, cfg.nh
    h = np.zeros((n, nh), dtype=np.float64)
    for k, (kind, lo, hi) in enumerate(cfg.priors):
        if kind == "logu":
            h[:, k] = np.exp(rng.uniform(np.log(lo), np.log(hi), size=n))
        elif kind == "u":
            h[:, k] = rng.uniform(lo, hi, size=n)
        elif kind == "fixed":
            h[:, k] = lo
        else:
            raise ValueError(kind)
    if cfg.model == C.TOY:
        # Figure 2: worker i optimises along axis i only
        h[:] = 0.0
        for m in range(n):
            h[m, m % nh] = 1.0
        return h
    return h.astype(np.float32).astype(np.float64)


def make_inputs(cfg: C.PBTConfig, seed: Optional[int] = None) -> Inputs:
    seed = cfg.seed if seed is None else seed
    h = _init_hparams(cfg, _rng(seed, 1))
    if cfg.model == C.TOY:
        return Inputs(init_hparams=h)

    bf16 = cfg.dtype == C.BF16
    grid = _to_bf16_grid if bf16 else (lambda a: np.ascontiguousarray(a, dtype=np.float32))

    if cfg.model == C.GAN:
        zdim = cfg.widths[0][0]
        xdim = cfg.widths[0][-1]
        assert xdim == 2, "the mixture-of-Gaussians ring is two-dimensional"

        def ring(rng, rows):
            k = rng.integers(0, 8, size=rows)
            mu = np.stack([np.cos(2 * np.pi * k / 8), np.sin(2 * np.pi * k / 8)], axis=1)
            return (mu + 0.02 * rng.standard_normal((rows, 2))).astype(np.float32)

        x_pool = grid(ring(_rng(seed, 2), cfg.pool_rows))
        z_pool = grid(_rng(seed, 3).standard_normal((cfg.pool_rows, zdim)).astype(np.float32))
        z_eval = grid(_rng(seed, 4).standard_normal((cfg.eval_batch, zdim)).astype(np.float32))
        return Inputs(init_hparams=h, x_pool=x_pool, z_pool=z_pool, x_eval=z_eval)

    widths = cfg.widths[0]
    teacher = _teacher(widths, _rng(seed, 5))

    def draw_x(rng, rows):
        if cfg.loss == C.LOSS_CE_HARD:
            return grid(rng.random((rows, widths[0]), dtype=np.float32))
        return grid(rng.standard_normal((rows, widths[0]), dtype=np.float32))

    def label(x, rng):
        t = _teacher_forward(teacher, x)
        if cfg.loss == C.LOSS_MSE:
            return (t + 0.1 * rng.standard_normal(t.shape)).astype(np.float32)
        if cfg.loss == C.LOSS_CE_HARD:
            return np.argmax(t, axis=1).astype(np.int32)
        if cfg.loss == C.LOSS_CE_SOFT:
            return grid(_softmax(t))
        raise ValueError(cfg.loss)

    x_pool = draw_x(_rng(seed, 6), cfg.pool_rows)
    y_pool = label(x_pool, _rng(seed, 7))
    x_eval = draw_x(_rng(seed, 8), cfg.eval_batch)
    y_eval = label(x_eval, _rng(seed, 9))
    return Inputs(init_hparams=h, x_pool=x_pool, y_pool=y_pool, x_eval=x_eval, y_eval=y_eval)
