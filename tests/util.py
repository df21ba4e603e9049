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


# Sign-like optimisers (Adam, RMSProp) and zero-initialised tensors.
#
# While the moments are young the normalised update lr * m / (sqrt(v) + eps) is lr * sign(g) whatever |g| is, and for
# |g| of the order of eps it is lr * g / (|g| + eps), whose slope is 1 / eps.  An element whose gradient the two
# sides do not agree on (a near-zero sum whose sign or size differs by rounding) then moves by up to 2 lr on one
# side relative to the other.  For a weight matrix that is part of the measured error (its norm is set by the
# initialisation, and weight matrices are ALWAYS compared whole).  A bias vector starts at zero, so for the first
# steps its whole norm is O(lr) and a single such element is worth more than the relative bar.  For bias vectors
# whose norm is still of order lr, and only for them, an element is taken out of the relative comparison when the
# two gradients of that element disagree by more than a quarter of the oracle's value, |g_gpu - g_oracle| >
# 0.25 |g_oracle| (the bias gradient is always stored by the library).  Such an element must be a near-zero one
# (|g_oracle| at most NEAR_ZERO times the tensor's rms: asserted), and it is checked against the
# absolute bound |w_gpu - w_oracle| <= 2 lr (Adam; 2 lr / sqrt(1 - rho) for RMSProp, whose first update is
# g / sqrt((1 - rho) g^2)) instead.  An element whose gradient is exactly zero on both sides (a dead ReLU unit) is
# never masked.  The ledger below records how many elements each tensor kept; tests assert the kept fraction and
# the session prints the table.
DISAGREE = 0.25
NEAR_ZERO = {"fp32": 1e-3, "bf16_fp32master": 5e-2}   # a masked element's |g_oracle| is at most this times the tensor's rms
O_LR_NORM = 64.0        # a tensor counts as "norm of order lr" while rms(w_oracle) <= O_LR_NORM * lr
LEDGER = {}             # (case, tensor name) -> [elements compared relatively, elements masked, worst rel err]
DRIFT = {}              # (case, steps without re-seeding, "W" | "b" | "fitness") -> worst relative error seen


def _lr_of(cfg, name, hparams):
    slot = cfg.slot("lr_d") if (name.startswith("s1.") and cfg.slot("lr_d") >= 0) else cfg.slot("lr")
    return float(hparams[slot]) if slot >= 0 else 0.0


def sign_like_mask(cfg, name, w_ref, g_ref, g_gpu, lr):
    """Boolean array: True where the element is compared absolutely (see above), or None if the tensor is
    compared whole."""
    if cfg.optimizer not in ("adam", "rmsprop") or ".b" not in name or lr <= 0.0 or g_gpu is None:
        return None
    w = np.asarray(w_ref, dtype=np.float64)
    if w.size and np.sqrt(np.mean(w * w)) > O_LR_NORM * lr:
        return None
    go = np.asarray(g_ref, dtype=np.float64)
    gg = np.asarray(g_gpu, dtype=np.float64)
    masked = np.abs(gg - go) > DISAGREE * np.abs(go)
    # The near-zero requirement does not apply where the stored gradient is not the whole story: tensors updated
    # several times per step (a GAN's critic: the gradient kept is that of the last of K updates, by which time the
    # two sides have drifted apart by K - 1 updates) and tensors whose elements cancel exactly (a unit that is active
    # on one more row on one side changes its element by a whole term).  The absolute bound still holds them.
    several = cfg.model == "gan_pair" and name.startswith("s1.") and cfg.gan_d_steps > 1
    if masked.any() and not several and name not in exactly_cancelling_gradient_tensors(cfg):
        rms = np.sqrt(np.mean(go * go))
        worst = np.abs(go[masked]).max()
        assert worst <= NEAR_ZERO[cfg.dtype] * max(rms, 1e-30) or rms == 0.0, \
            f"{name}: gradients disagree on an element that is not near zero ({worst:.3e} vs rms {rms:.3e})"
    return masked


def ledger_rows(prefix=""):
    return sorted((k, v) for k, v in LEDGER.items() if k[0].startswith(prefix))


def assert_kept_fractions(case, floor=0.98, cfg=None):
    """Per tensor of `case`, over every member and step compared so far: at least `floor` of the elements went
    through the relative comparison."""
    exempt = exactly_cancelling_gradient_tensors(cfg) if cfg is not None else set()
    for (c, name), (kept, masked, _) in ledger_rows(case):
        if c == case and kept + masked > 0 and name not in exempt:
            frac = kept / (kept + masked)
            assert frac >= floor, f"{case} {name}: only {frac:.4f} of the elements compared relatively"


def exactly_cancelling_gradient_tensors(cfg):
    """Tensors many of whose gradient elements cancel EXACTLY in exact arithmetic, so that no floor on the kept
    fraction applies to them.  The Wasserstein critic's last-layer deltas are exactly -1/B (real rows) and +1/B
    (generated rows), so the bias gradient of a hidden critic unit is (1/B) w_u (#generated rows on which it is
    active - #real rows on which it is active): zero whenever the two counts agree, and then each side holds 0.0 or
    the rounding noise of its own summation order, which a sign-like optimiser turns into a step of size lr."""
    if cfg.model == "gan_pair" and cfg.loss == "wgan_gp":
        return {f"s1.b{l}" for l in range(len(cfg.widths[1]) - 2)}
    return set()


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


def assert_state_close(cfg, gpu_state, cpu_state, keys, tol, what="", case=None):
    """Tensor by tensor, ||gpu - oracle|| / ||oracle|| <= tol[key].  `case` names the ledger entry (default: the
    first word of `what`)."""
    zero_grad = identically_zero_gradient_tensors(cfg)
    noise = {"grad": 1e-6, "opt1": 1e-6, "opt2": 1e-12}
    case = case if case is not None else (what.split()[0] if what else cfg.name)
    hp = gpu_state.get("hparams") if isinstance(gpu_state, dict) else None
    for key in keys:
        for name, sl in tensor_slices(cfg):
            a, b = gpu_state[key][sl], cpu_state[key][sl]
            if name in zero_grad:
                if key in noise:
                    assert np.abs(a).max() <= noise[key] and np.abs(b).max() <= noise[key], f"{what} {key} {name}"
                continue
            masked = None
            if key == "w" and "grad" in cpu_state and hp is not None:
                lr = _lr_of(cfg, name, hp)
                g_gpu = gpu_state["grad"][sl] if "grad" in gpu_state else None
                masked = sign_like_mask(cfg, name, b, cpu_state["grad"][sl], g_gpu, lr)
            if masked is not None and masked.any():
                bound = 2.0 * lr * (1.0 + 1e-3)
                if cfg.model == "gan_pair" and name.startswith("s1."):
                    bound *= max(1, cfg.gan_d_steps)          # that many critic updates per step
                if cfg.optimizer == "rmsprop":
                    bound /= np.sqrt(1.0 - float(np.float32(cfg.beta2)))
                d = np.abs(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64))[masked]
                assert d.max() <= bound, f"{what} {key} {name}: masked element off by {d.max():.3e} > 2 lr = {bound:.3e}"
                a, b = a[~masked], b[~masked]
            e = rel_err(a, b)
            if key == "w":
                rec = LEDGER.setdefault((case, name), [0, 0, 0.0])
                rec[0] += int(np.size(a))
                rec[1] += int(masked.sum()) if masked is not None else 0
                rec[2] = max(rec[2], e)
            assert e <= tol[key], f"{what} {key} {name}: rel err {e:.3e} > {tol[key]:.1e}"


def push_oracle_state(gpu, cpu):
    """Overwrite the GPU population with the oracle's state (all members)."""
    for m in range(cpu.N):
        if cpu.toy:
            gpu.set_state(m, w=cpu.theta[m], hparams=cpu.H[m].astype(np.float64),
                          fitness=float(cpu.fitness[m]), step=int(cpu.t[m]), round=cpu.round)
        else:
            f = cpu.get_flat(m)
            gpu.set_state(m, w=f["w"], opt1=f["opt1"], opt2=f["opt2"], scalars=f["scalars"],
                          hparams=cpu.H[m].astype(np.float64), fitness=float(cpu.fitness[m]),
                          step=int(cpu.t[m]), round=cpu.round)


def oracle_history_arrays(cpu, depth=10):
    """The oracle's score histories as the dense (scores [N][depth], counts [N]) pair of the interface."""
    h = np.zeros((cpu.N, depth), dtype=np.float64)
    c = np.zeros(cpu.N, dtype=np.int32)
    for m in range(cpu.N):
        c[m] = len(cpu.history[m])
        h[m, :c[m]] = [float(x) for x in cpu.history[m]]
    return h, c
