"""Helpers shared by the parity tests (no method arithmetic here)."""
import numpy as np

# Tolerances, per tensor, as ||gpu - oracle||_2 / ||oracle||_2.
#   fp32 populations: weights 1e-5 (the stated bar); gradients and optimiser state 1e-4
#     (fp32 accumulation over K <= 2048 terms against float64: ~sqrt(K) * 6e-8).
#   bf16 populations: 2e-2 for weights (the stated bar) and the same for gradients / state:
#     both sides multiply identical bf16 operands; differences come from fp32 vs float64
#     accumulation and from the rare activation whose bf16 rounding flips (one ulp = 2^-8).
TOL = {"fp32": {"w": 1e-5, "g": 1e-4}, "bf16_fp32master": {"w": 2e-2, "g": 2e-2}}


def tensor_slices(cfg):
    """(name, slice) of every tensor in the interface's flat order: per stack, per layer, W then b."""
    out, o = [], 0
    for s, ws in enumerate(cfg.widths):
        for l in range(len(ws) - 1):
            n = ws[l] * ws[l + 1]
            out.append((f"s{s}.W{l}", slice(o, o + n)))
            o += n
            out.append((f"s{s}.b{l}", slice(o, o + ws[l + 1])))
            o += ws[l + 1]
    return out


def rel_err(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    nb = np.linalg.norm(b)
    na = np.linalg.norm(a - b)
    if nb == 0.0:
        return 0.0 if na == 0.0 else float("inf")
    return na / nb


def adam_well_conditioned(cfg, cpu_state, tol_g):
    """Adam's normalised update lr * m / (sqrt(v) + eps) behaves like lr * sign(g) while the
    moments are young: an element whose gradient could change sign under a perturbation that
    the gradient tolerance itself allows (|g| < tol_g * rms(g) of its tensor) can move by a
    full 2 lr, which swamps tensors whose norm is itself O(lr) (biases start at zero).  Such
    elements are left out of the direct weight comparison only; they stay in the gradient,
    moment and optimiser-arithmetic comparisons.  Decided from oracle values alone."""
    keep = np.ones(cpu_state["grad"].shape, dtype=bool)
    for _, sl in tensor_slices(cfg):
        g = cpu_state["grad"][sl].astype(np.float64)
        rms = np.sqrt(np.mean(g * g)) if g.size else 0.0
        keep[sl] = np.abs(g) >= tol_g * rms if rms > 0 else False
    return keep


def identically_zero_gradient_tensors(cfg):
    """Tensors whose gradient is zero by construction.  The Wasserstein critic's objective is unchanged when a
    constant is added to D, so its output bias has gradient sum_b (-1/B) + sum_b (+1/B) = 0: what either side
    holds there is the rounding noise of that sum (partial sums of size one), and Adam turns noise into steps
    of order lr.  Such a tensor is compared absolutely (gradient and moments stay at noise level), not
    relatively to the oracle's own noise."""
    if cfg.model == "gan_pair" and cfg.loss == "wgan_gp":
        return {f"s1.b{len(cfg.widths[1]) - 2}"}
    return set()


def critic_offset(cfg, state):
    """The Wasserstein critic is defined up to an additive constant (its output bias, which only rounding noise
    moves: see identically_zero_gradient_tensors).  The generator's loss -mean D(G(z)) contains that constant;
    adding the bias back gives the part of the loss that is determined."""
    names = identically_zero_gradient_tensors(cfg)
    off = 0.0
    for name, sl in tensor_slices(cfg):
        if name in names:
            off += float(np.asarray(state["w"][sl], dtype=np.float64).sum())
    return off


def assert_state_close(cfg, gpu_state, cpu_state, keys, tol, what=""):
    keep = None
    if cfg.optimizer in ("adam", "rmsprop") and "w" in keys and "grad" in cpu_state:
        keep = adam_well_conditioned(cfg, cpu_state, tol.get("grad", 2e-2))
    zero_grad = identically_zero_gradient_tensors(cfg)
    noise = {"grad": 1e-6, "opt1": 1e-6, "opt2": 1e-12}
    for key in keys:
        for name, sl in tensor_slices(cfg):
            a, b = gpu_state[key][sl], cpu_state[key][sl]
            if name in zero_grad:
                if key in noise:
                    assert np.abs(a).max() <= noise[key] and np.abs(b).max() <= noise[key], f"{what} {key} {name}"
                continue
            if key == "w" and keep is not None:
                a = np.where(keep[sl], a, b)
            e = rel_err(a, b)
            assert e <= tol[key], f"{what} {key} {name}: rel err {e:.3e} > {tol[key]:.1e}"


def push_oracle_state(gpu, cpu):
    """Overwrite the GPU population with the oracle's state (all members)."""
    for m in range(cpu.N):
        if cpu.toy:
            gpu.set_state(m, w=cpu.theta[m], hparams=cpu.H[m].astype(np.float64),
                          fitness=float(cpu.fitness[m]), step=cpu.step_count, round=cpu.round)
        else:
            f = cpu.get_flat(m)
            gpu.set_state(m, w=f["w"], opt1=f["opt1"], opt2=f["opt2"], scalars=f["scalars"],
                          hparams=cpu.H[m].astype(np.float64), fitness=float(cpu.fitness[m]),
                          step=cpu.step_count, round=cpu.round)


def oracle_history_arrays(cpu, depth=10):
    """The oracle's score histories as the dense (scores [N][depth], counts [N]) pair of the interface."""
    h = np.zeros((cpu.N, depth), dtype=np.float64)
    c = np.zeros(cpu.N, dtype=np.int32)
    for m in range(cpu.N):
        c[m] = len(cpu.history[m])
        h[m, :c[m]] = [float(x) for x in cpu.history[m]]
    return h, c
