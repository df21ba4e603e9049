"""Plain CPU oracle for lockstep Population Based Training -- TEST INFRASTRUCTURE.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may use
this module; the GPU library never imports, links or calls it, and it shares
no code with the GPU path.  It is slow on purpose: one member at a time,
float64 arithmetic, NumPy matmul as the only library primitive, no blocking
or fusion, so each function can be read against the passage it cites.

What it follows
---------------
* Algorithm 1 (Section 3) in the partial-synchrony form of Appendix A.1: all
  members take the same number of `step`s, then `eval`, then exploit/explore.
* `step` (Eq. 2): one gradient update of the member's weights conditioned on
  its own hyperparameters h (SGD, SGD with momentum, or Adam; Sections 4.1.1,
  4.2.1, 4.3.1 name the optimisers, Appendix A.4 gives Adam's constants).
* `eval` (Eq. 1): a function of the weights only -- held-out loss (negated so
  that larger is better), the toy's true objective Q (Figure 2), or the
  negative energy distance of generated samples to the target mixture.
* `exploit`: truncation selection (Section 4.1.1 (b)): rank all members; each
  member in the bottom 20 % copies a member drawn uniformly from the top 20 %.
* `explore`: perturb (Section 4.1.1 (a)): every hyperparameter of a member
  that copied is multiplied by 0.8 or 1.2 independently (0.5 / 2.0 in Section
  4.3.1 are the same operator with other factors).
* The other operators the paper lists: binary tournament (Section 4.3.1 (b)),
  t-test selection on the last 10 scores (Section 4.1.1, exploit (a)), and
  resampling from the prior (Section 4.1.1, explore (b)).
* The guard of Algorithm 1 (explore and re-evaluate only when the weights
  changed) and the population update.

Readings taken where the paper is silent (each one is listed in the design
notes of the repository): total order (fitness descending, member index
ascending; NaN ranks last; -0 equals +0); n_cut = max(1, floor(N * 1/5));
donor index by multiply-shift of one Philox word; one Philox bit per
perturbed slot with probability 1/2; clamp after perturbation; optimiser state
travels with the weights; Adam's bias correction uses running products of the
betas actually used; bf16 populations round GEMM operands (weights shadow,
activations, back-propagated deltas) to bfloat16 and keep masters in float32.

Pins (tests/test_oracle_*.py): toy closed form and the paper's printed Q ~ 0.4
(Figure 2 caption); brute-force enumeration of truncation selection for
N = 2..5; donor uniformity; copy / explore / lineage invariants; member
isolation with exploit off; finite-difference gradients; least-squares special
case; hand-computed optimiser trajectories; energy-distance special cases;
Philox known-answer vectors; Welch's test against printed critical values, the
closed-form t distributions with 1 and 2 degrees of freedom and an independent
library routine; resampling against the prior's range, rate and quantiles.
Members at their own pace (`run_schedule`): every
schedule over small populations against each member run alone, the lockstep
schedule against `run`, own-clock `ready` against its definition.
`Population.run` over a whole neural-network
config has no external truth to compare with: parity unpinned beyond the pins
of its parts.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional

import numpy as np

from . import philox as px

# flag bits and tags are re-declared here on purpose (no shared constants with
# the GPU library)
COPY_WEIGHTS, COPY_HPARAMS, EXPLORE = 1, 2, 4
N_SCALARS = 4  # c1, c2 of stack 0; c1, c2 of stack 1 (Adam bias-correction products)
MAX_LAYERS = 8
WINDOW_ALIGN = 128


# --------------------------------------------------------------------------
# rounding helpers
# --------------------------------------------------------------------------
def round_bf16(a: np.ndarray) -> np.ndarray:
    """float -> nearest bfloat16 (ties to even), returned as float64 values."""
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(f.shape)


def _f32(a):
    return np.asarray(a, dtype=np.float64).astype(np.float32)


# --------------------------------------------------------------------------
# exploit / explore: pure functions on small arrays (Section 4.1.1)
# --------------------------------------------------------------------------
def n_cut_of(n: int, num: int = 1, den: int = 5) -> int:
    """Size of the bottom and of the top set: 20 % of N, at least one, never overlapping."""
    if n < 2:
        return 0
    c = max(1, (n * num) // den)
    return min(c, n // 2)


def rank_members(fitness) -> List[int]:
    """Members from best to worst: fitness descending, index ascending on ties; NaN last."""
    keyed = []
    for i, f in enumerate(fitness):
        f = float(f)
        if math.isnan(f):
            f = -math.inf
        keyed.append((-f if f != 0.0 else 0.0, i))
    keyed.sort()
    return [i for _, i in keyed]


def donor_index(word: int, n_cut: int) -> int:
    """Uniform index in [0, n_cut) from a 32-bit word by multiply-shift."""
    return (int(word) * int(n_cut)) >> 32


def ready_members(step: int, interval: int, offsets=None, n: int = 0) -> np.ndarray:
    """`ready` of Algorithm 1 for every member at optimisation step `step` (Section 3: enough steps have gone by
    since the member was last ready).  Member m is ready when step - offsets[m] is a positive multiple of
    `interval`; with no offsets all members are ready together (the lockstep schedule), with offsets the ready
    points are staggered as they are when workers run at their own pace."""
    if offsets is None or len(offsets) == 0:
        return np.full(n, step > 0 and step % interval == 0, dtype=bool)
    return np.array([(step - int(o)) > 0 and (step - int(o)) % interval == 0 for o in offsets], dtype=bool)


def ready_members_own(t, interval: int, offsets=None) -> np.ndarray:
    """`ready(p, t, P)` of Algorithm 1 with every member on its own clock (Section 3: workers run asynchronously, each
    counting its own steps): member m is ready when its OWN step count t[m], minus its offset, is a positive
    multiple of `interval`.  With equal counts this is ready_members."""
    t = np.asarray(t, dtype=np.int64)
    o = np.zeros_like(t) if offsets is None or len(offsets) == 0 else np.asarray(offsets, dtype=np.int64)
    d = t - o
    return (d > 0) & (d % interval == 0)


def _is_ready(ready, i) -> bool:
    return True if ready is None else bool(ready[i])


def truncation_select(fitness, seed: int, rnd: int, num: int = 1, den: int = 5, ready=None) -> np.ndarray:
    """Copy map src[N]: src[i] == i for members that keep their state; a bottom
    member b gets src[b] = a top member drawn uniformly (Section 4.1.1 (b)).
    Only members that are `ready` (Algorithm 1; None = all) exploit; the ranking is over the whole population."""
    n = len(fitness)
    src = np.arange(n, dtype=np.int32)
    c = n_cut_of(n, num, den)
    if c == 0:
        return src
    order = rank_members(fitness)
    top, bottom = order[:c], order[n - c:]
    for b in bottom:
        if not _is_ready(ready, b):
            continue
        word = px.draw(seed, b, rnd, px.STREAM_EXPLOIT, 0)[0]
        src[b] = top[donor_index(word, c)]
    return src


def tournament_select(fitness, seed: int, rnd: int, ready=None) -> np.ndarray:
    """Binary tournament (Section 4.3.1 (b)): every member draws one OTHER member uniformly and copies it if that
    member's score is strictly better (NaN counts as the worst score).  src[i] == i where nothing is copied.
    All decisions use the fitness vector as it stands before any copy."""
    n = len(fitness)
    src = np.arange(n, dtype=np.int32)
    if n < 2:
        return src
    f = [(-math.inf if math.isnan(float(x)) else float(x)) for x in fitness]
    for i in range(n):
        if not _is_ready(ready, i):
            continue
        word = px.draw(seed, i, rnd, px.STREAM_EXPLOIT, 1)[0]
        j = donor_index(word, n - 1)
        if j >= i:
            j += 1
        if f[j] > f[i]:
            src[i] = j
    return src


HISTORY = 10  # evaluations kept per member for the t-test (Section 4.1.1, exploit (a): the last 10 scores)


def welch_t_test(a, b):
    """Welch's unequal-variance t-test of sample b against sample a.  Returns (t, df, p): the statistic
    (mean_b - mean_a) / sqrt(s_a^2/n_a + s_b^2/n_b) with unbiased variances, the Welch-Satterthwaite degrees
    of freedom, and the two-sided p-value P(|T_df| >= |t|) = I_{df/(df+t^2)}(df/2, 1/2) (the regularised
    incomplete beta function is the library primitive of this step)."""
    from scipy.special import betainc
    a = [float(x) for x in a]
    b = [float(x) for x in b]
    na, nb = len(a), len(b)
    ma = sum(a) / na
    mb = sum(b) / nb
    va = sum((x - ma) ** 2 for x in a) / (na - 1)
    vb = sum((x - mb) ** 2 for x in b) / (nb - 1)
    qa, qb = va / na, vb / nb
    se2 = qa + qb
    t = (mb - ma) / math.sqrt(se2)
    df = se2 * se2 / (qa * qa / (na - 1) + qb * qb / (nb - 1))
    p = float(betainc(df / 2.0, 0.5, df / (df + t * t)))
    return t, df, p


def ttest_better(hist_self, hist_other, alpha: float) -> bool:
    """Section 4.1.1, exploit (a): the other member replaces this one if its mean score over its recorded
    evaluations is higher and Welch's t-test rejects equal means at level alpha (two-sided).  Readings: NaN
    scores count as -inf; fewer than two recorded scores on either side -> no test, no copy; a member whose own
    mean is -inf is replaced by any member with a larger mean; if both samples have zero variance the larger mean
    wins outright (the statistic is unbounded); any other non-finite statistic -> no copy."""
    clean = lambda h: [(-math.inf if math.isnan(float(x)) else float(x)) for x in h]
    a, b = clean(hist_self), clean(hist_other)
    if len(a) < 2 or len(b) < 2:
        return False
    ma, mb = sum(a) / len(a), sum(b) / len(b)
    if not (mb > ma):
        return False
    if ma == -math.inf:
        return True
    if not math.isfinite(mb):
        return False
    va = sum((x - ma) ** 2 for x in a) / (len(a) - 1)
    vb = sum((x - mb) ** 2 for x in b) / (len(b) - 1)
    if va / len(a) + vb / len(b) == 0.0:
        return True
    _, _, p = welch_t_test(a, b)
    return bool(p < alpha)


def ttest_select(histories, seed: int, rnd: int, alpha: float, ready=None) -> np.ndarray:
    """T-test selection (Section 4.1.1, exploit (a)): every member draws one OTHER member uniformly and copies it
    if `ttest_better` holds for the two score histories (oldest first, at most HISTORY entries each).
    src[i] == i where nothing is copied.  All decisions use the histories as they stand before any copy."""
    n = len(histories)
    src = np.arange(n, dtype=np.int32)
    if n < 2:
        return src
    for i in range(n):
        if not _is_ready(ready, i):
            continue
        word = px.draw(seed, i, rnd, px.STREAM_EXPLOIT, 2)[0]
        j = donor_index(word, n - 1)
        if j >= i:
            j += 1
        if ttest_better(histories[i], histories[j], alpha):
            src[i] = j
    return src


def explore_bits(seed: int, member: int, rnd: int, nh: int) -> List[int]:
    """One bit per hyperparameter slot: 1 -> multiply by the high factor, 0 -> low."""
    bits = []
    for k in range(nh):
        words = px.draw(seed, member, rnd, px.STREAM_EXPLORE, k >> 2)
        bits.append((words[k & 3] >> 31) & 1)
    return bits


def perturb(h_row: np.ndarray, bits, mask, factor_lo, factor_hi, lo, hi) -> np.ndarray:
    """Section 4.1.1 (a): each perturbable slot times factor_lo or factor_hi (one
    rounding, in h's own dtype), then clamped to [lo, hi]."""
    dt = h_row.dtype.type
    out = h_row.copy()
    for k in range(len(out)):
        if not mask[k]:
            continue
        f = dt(factor_hi) if bits[k] else dt(factor_lo)
        v = dt(out[k] * f)
        v = max(v, dt(lo[k]))
        v = min(v, dt(hi[k]))
        out[k] = v
    return out


def resample_threshold(q: float) -> int:
    """Probability q as a 32-bit threshold: a slot is resampled when its Philox word is below it."""
    return min(max(int(q * 4294967296.0), 0), 0xFFFFFFFF)


def resample(h_row: np.ndarray, seed: int, member: int, rnd: int, mask, priors, q: float, lo, hi) -> np.ndarray:
    """Section 4.1.1, explore (b): each hyperparameter of a member that copied is, with probability q, drawn
    afresh from its prior; otherwise the copied value is kept.  Slot k uses Philox block 16 + k of the explore
    stream: word 0 decides (word < q * 2^32), word 1 gives u = (word + 1/2) / 2^32, and the value is
    lo + u (hi - lo) for a uniform prior, exp(log lo + u (log hi - log lo)) for a log-uniform one -- computed in
    float64, rounded once to h's dtype, then clamped like a perturbed value."""
    dt = h_row.dtype.type
    out = h_row.copy()
    thr = resample_threshold(q)
    for k in range(len(out)):
        kind, plo, phi = priors[k]
        if not mask[k] or kind == "fixed":
            continue
        words = px.draw(seed, member, rnd, px.STREAM_EXPLORE, 16 + k)
        if not (words[0] < thr):
            continue
        u = (float(words[1]) + 0.5) / 4294967296.0
        if kind == "logu":
            la, lb = math.log(plo), math.log(phi)
            v = math.exp(la + u * (lb - la))
        else:
            v = plo + u * (phi - plo)
        v = dt(v)
        v = max(v, dt(lo[k]))
        v = min(v, dt(hi[k]))
        out[k] = v
    return out


# --------------------------------------------------------------------------
# losses (batch means) and their derivative with respect to the logits
# --------------------------------------------------------------------------
def softplus(x):
    return np.maximum(x, 0.0) + np.log1p(np.exp(-np.abs(x)))


def sigmoid(x):
    return np.where(x >= 0, 1.0 / (1.0 + np.exp(-np.abs(x))), np.exp(-np.abs(x)) / (1.0 + np.exp(-np.abs(x))))


def loss_mse(z, y):
    """mean over the batch of sum_j (z_j - y_j)^2;  dL/dz = 2 (z - y) / B."""
    b = z.shape[0]
    d = z - y.reshape(z.shape)
    return float((d * d).sum() / b), 2.0 * d / b


def loss_ce_hard(z, labels):
    """mean_i [ logsumexp(z_i) - z_i[label_i] ];  dL/dz = (softmax(z) - onehot) / B."""
    b = z.shape[0]
    zm = z - z.max(axis=1, keepdims=True)
    e = np.exp(zm)
    s = e.sum(axis=1, keepdims=True)
    logp = zm - np.log(s)
    idx = np.arange(b)
    loss = float(-logp[idx, labels].sum() / b)
    d = e / s
    d[idx, labels] -= 1.0
    return loss, d / b


def loss_ce_soft(z, t):
    """mean_i [ -sum_j t_ij log softmax(z_i)_j ];  dL/dz = (softmax(z) * sum_j t_ij - t) / B."""
    b = z.shape[0]
    zm = z - z.max(axis=1, keepdims=True)
    e = np.exp(zm)
    s = e.sum(axis=1, keepdims=True)
    logp = zm - np.log(s)
    loss = float(-(t * logp).sum() / b)
    d = (e / s) * t.sum(axis=1, keepdims=True) - t
    return loss, d / b


def energy_distance_to_ring(x: np.ndarray, n_modes: int = 8) -> float:
    """V-statistic energy distance between the sample x[n,2] and the equally
    weighted modes mu_k = (cos 2 pi k/8, sin 2 pi k/8):
        E = 2/(n K) sum_i sum_k |x_i - mu_k| - 1/n^2 sum_i sum_j |x_i - x_j|
            - 1/K^2 sum_k sum_l |mu_k - mu_l|."""
    x = np.asarray(x, dtype=np.float64)
    n = x.shape[0]
    k = np.arange(n_modes)
    mu = np.stack([np.cos(2 * np.pi * k / n_modes), np.sin(2 * np.pi * k / n_modes)], axis=1)
    cross = 0.0
    for i in range(n):
        cross += np.sqrt(((x[i] - mu) ** 2).sum(axis=1)).sum()
    within = 0.0
    for i in range(n):
        within += np.sqrt(((x[i] - x) ** 2).sum(axis=1)).sum()
    modes = 0.0
    for a in range(n_modes):
        modes += np.sqrt(((mu[a] - mu) ** 2).sum(axis=1)).sum()
    return 2.0 * cross / (n * n_modes) - within / (n * n) - modes / (n_modes * n_modes)


# --------------------------------------------------------------------------
# optimiser updates on one tensor (float64 arithmetic; caller stores in master precision)
# --------------------------------------------------------------------------
def sgd_update(theta, g, lr):
    """Plain stochastic gradient descent, the `step` Section 3 takes as its example: theta <- theta - lr g."""
    return theta - lr * g


def sgdm_update(theta, vel, g, lr, mu):
    """v <- mu v + g;  theta <- theta - lr v  (no dampening, no Nesterov)."""
    vel = mu * vel + g
    return theta - lr * vel, vel


def rmsprop_update(theta, ms, g, lr, rho, eps):
    """RMSProp (Tieleman & Hinton, 2012), the optimiser of the paper's RL experiments (Section 4.1.1):
    ms <- rho ms + (1 - rho) g^2;  theta <- theta - lr g / (sqrt(ms) + eps)."""
    ms = rho * ms + (1.0 - rho) * g * g
    return theta - lr * g / (np.sqrt(ms) + eps), ms


def adam_update(theta, m, v, g, lr, b1, b2, eps, wd, c1, c2):
    """m <- b1 m + (1-b1) g; v <- b2 v + (1-b2) g^2;
    theta <- theta - lr (m/(1-c1)) / (sqrt(v/(1-c2)) + eps) - lr wd theta,
    where c1, c2 are the running products of the betas used so far (including
    this step); with constant betas c1 = b1^t, the textbook bias correction."""
    m = b1 * m + (1.0 - b1) * g
    v = b2 * v + (1.0 - b2) * g * g
    mhat = m / (1.0 - c1)
    vhat = v / (1.0 - c2)
    theta = theta - lr * mhat / (np.sqrt(vhat) + eps) - lr * wd * theta
    return theta, m, v


# --------------------------------------------------------------------------
# the population
# --------------------------------------------------------------------------
class Population:
    """State (theta, h, p, t) of every member (Algorithm 1) plus optimiser state."""

    def __init__(self, cfg, inputs, seed: Optional[int] = None, only_members=None):
        """only_members: build (and later step / evaluate) just these members of the population; the
        others stay empty.  For checking a sample of a large population member by member."""
        self.cfg = cfg
        self.inp = inputs
        self.seed = int(cfg.seed if seed is None else seed)
        self.N = cfg.n_members
        self.members = list(range(self.N)) if only_members is None else [int(m) for m in only_members]
        self.toy = cfg.model == "toy_quadratic"
        self.gan = cfg.model == "gan_pair"
        self.bf16 = cfg.dtype == "bf16_fp32master"
        self.master = np.float64 if self.toy else np.float32
        self.q = round_bf16 if self.bf16 else (lambda a: np.asarray(a, dtype=np.float64))
        self.t = np.zeros(self.N, dtype=np.int64)    # every member's own step count (Algorithm 1's t)
        self.round = 0
        self.H = np.array(inputs.init_hparams, dtype=np.float64).astype(self.master)
        self.fitness = np.zeros(self.N, dtype=self.master)
        self.history = [[] for _ in range(self.N)]   # scores of the last HISTORY evaluations, oldest first
        self.src = np.arange(self.N, dtype=np.int32)
        self.last_loss = np.zeros((self.N, 2), dtype=np.float64)
        self.scalars = np.ones((self.N, N_SCALARS), dtype=np.float32)
        # tensors[m] = list over (stack, layer) of dicts W, b
        self.shapes = []  # (stack, layer, out, in)
        if self.toy:
            d = cfg.nh
            self.theta = np.tile(np.asarray(cfg.toy_theta0, dtype=np.float64), (self.N, 1))
            assert self.theta.shape == (self.N, d)
        else:
            for s, ws in enumerate(cfg.widths):
                for l in range(len(ws) - 1):
                    self.shapes.append((s, l, ws[l + 1], ws[l]))
            self.W = [[None] * len(self.shapes) for _ in range(self.N)]
            self.b = [[None] * len(self.shapes) for _ in range(self.N)]
            for m in self.members:
                for t, (s, l, fo, fi) in enumerate(self.shapes):
                    self.W[m][t] = self._init_weight(m, s, l, fo, fi)
                    self.b[m][t] = np.zeros(fo, dtype=np.float32)
            z = lambda: [[None if x is None else np.zeros_like(x) for x in row] for row in self.W]
            zb = lambda: [[None if x is None else np.zeros_like(x) for x in row] for row in self.b]
            self.o1W, self.o1b = z(), zb()      # momentum / Adam m
            self.o2W, self.o2b = z(), zb()      # Adam v
            self.gW, self.gb = z(), zb()        # last gradient (for inspection)

    @property
    def step_count(self) -> int:
        """Steps taken by the members this population holds; in lockstep they all agree."""
        return int(self.t[self.members].max()) if len(self.members) else 0

    @step_count.setter
    def step_count(self, value: int):
        self.t[:] = int(value)

    # ----- initial weights: U(-a, a), a = sqrt(6 / fan_in), biases zero ------
    def _init_weight(self, m, s, l, fo, fi):
        n = fo * fi
        blocks = np.arange((n + 3) // 4, dtype=np.uint64)
        words = px.philox4x32_10_np(np.uint64(m), blocks, np.uint64(px.STREAM_INIT),
                                    np.uint64(s * MAX_LAYERS + l), self.seed)
        x = np.stack(words, axis=1).reshape(-1)[:n]
        u = (x >> np.uint32(8)).astype(np.float32) * np.float32(2.0 ** -23) - np.float32(1.0)
        a = np.float32(math.sqrt(6.0 / fi))
        return (u * a).astype(np.float32).reshape(fo, fi)

    # ----- helpers -----------------------------------------------------------
    def _tensors_of_stack(self, s):
        return [t for t, sh in enumerate(self.shapes) if sh[0] == s]

    def _hp(self, m, name, default):
        k = self.cfg.slot(name)
        return float(self.H[m, k]) if k >= 0 else float(default)

    def _window(self, m, block, word_index, pool_rows, batch):
        """Start row of this (member, step) window: a multiple of 128 drawn from
        the batch stream, so both sides read identical rows of the pool."""
        n_win = (pool_rows - batch) // WINDOW_ALIGN + 1
        w = px.draw(self.seed, m, int(self.t[m]), px.STREAM_BATCH, block)[word_index]
        return WINDOW_ALIGN * ((int(w) * n_win) >> 32)

    # ----- network forward / backward for one member -------------------------
    def forward(self, m, s, a0):
        """z_l = a_{l-1} W_l^T + b_l, a_l = ReLU(z_l) on hidden layers, last layer
        linear.  Returns (activations a_0..a_{L-1} as fed to the next GEMM, z_L)."""
        ts = self._tensors_of_stack(s)
        acts = [np.asarray(a0, dtype=np.float64)]
        z = None
        for i, t in enumerate(ts):
            w = self.q(self.W[m][t])
            z = acts[-1] @ w.T + self.b[m][t].astype(np.float64)
            if i + 1 < len(ts):
                acts.append(self.q(np.maximum(z, 0.0)))
        return acts, z

    def backward(self, m, s, acts, dz_last, need_wgrad=True, need_input_grad=False):
        """dW_l = dZ_l^T a_{l-1};  db_l = column sums of dZ_l;
        dZ_{l-1} = (dZ_l W_l) * [a_{l-1} > 0].  dz_last is already rounded."""
        ts = self._tensors_of_stack(s)
        dz = dz_last
        gW, gb = {}, {}
        dinput = None
        for i in range(len(ts) - 1, -1, -1):
            t = ts[i]
            if need_wgrad:
                gW[t] = dz.T @ acts[i]
                gb[t] = dz.sum(axis=0)
            if i > 0:
                da = dz @ self.q(self.W[m][t])
                dz = self.q(da * (acts[i] > 0.0))
            elif need_input_grad:
                dinput = self.q(dz @ self.q(self.W[m][t]))
        return gW, gb, dinput

    # ----- optimiser over the tensors of one stack ---------------------------
    def _apply(self, m, s, gW, gb, lr):
        cfg = self.cfg
        ts = self._tensors_of_stack(s)
        for t in ts:
            self.gW[m][t] = _f32(gW[t])
            self.gb[m][t] = _f32(gb[t])
        if cfg.optimizer == "sgd_plain":
            for t in ts:
                for P, g in ((self.W, gW[t]), (self.b, gb[t])):
                    P[m][t] = _f32(sgd_update(P[m][t].astype(np.float64), _f32(g).astype(np.float64), lr))
        elif cfg.optimizer == "sgdm":
            mu = self._hp(m, "momentum", cfg.momentum)
            for t in ts:
                for P, O, g in ((self.W, self.o1W, gW[t]), (self.b, self.o1b, gb[t])):
                    # the gradient is consumed at master precision (it is stored as float32)
                    th, vel = sgdm_update(P[m][t].astype(np.float64), O[m][t].astype(np.float64),
                                          _f32(g).astype(np.float64), lr, mu)
                    P[m][t], O[m][t] = _f32(th), _f32(vel)
        elif cfg.optimizer == "rmsprop":
            rho, eps = float(np.float32(cfg.beta2)), float(np.float32(cfg.eps))
            for t in ts:
                for P, O, g in ((self.W, self.o1W, gW[t]), (self.b, self.o1b, gb[t])):
                    th, ms = rmsprop_update(P[m][t].astype(np.float64), O[m][t].astype(np.float64),
                                            _f32(g).astype(np.float64), lr, rho, eps)
                    P[m][t], O[m][t] = _f32(th), _f32(ms)
        elif cfg.optimizer == "adam":
            b1 = self._hp(m, "beta1", cfg.beta1)
            b2 = float(np.float32(cfg.beta2))
            wd = float(np.float32(self._hp(m, "wd", cfg.weight_decay)))
            eps = float(np.float32(cfg.eps))
            # running products kept in float32 (they are part of the copied state)
            c1 = np.float32(self.scalars[m, 2 * s] * np.float32(b1))
            c2 = np.float32(self.scalars[m, 2 * s + 1] * np.float32(cfg.beta2))
            self.scalars[m, 2 * s], self.scalars[m, 2 * s + 1] = c1, c2
            b1 = float(np.float32(b1))
            for t in ts:
                for P, O1, O2, g in ((self.W, self.o1W, self.o2W, gW[t]),
                                     (self.b, self.o1b, self.o2b, gb[t])):
                    th, mm, vv = adam_update(P[m][t].astype(np.float64), O1[m][t].astype(np.float64),
                                             O2[m][t].astype(np.float64), _f32(g).astype(np.float64),
                                             lr, b1, b2, eps, wd, float(c1), float(c2))
                    P[m][t], O1[m][t], O2[m][t] = _f32(th), _f32(mm), _f32(vv)
        else:
            raise ValueError(cfg.optimizer)

    # ----- one `step` (Eq. 2) for one member ----------------------------------
    def _loss_and_dz(self, z, y):
        cfg = self.cfg
        if cfg.loss == "mse":
            return loss_mse(z, y.astype(np.float64))
        if cfg.loss == "ce_hard":
            return loss_ce_hard(z, y)
        if cfg.loss == "ce_soft":
            return loss_ce_soft(z, y.astype(np.float64))
        raise ValueError(cfg.loss)

    def _step_toy(self, m):
        # ascend the surrogate 1.2 - sum_i h_i theta_i^2 (Figure 2):
        # theta_i <- theta_i + eta * (-2 h_i theta_i), three roundings per element
        eta = np.float64(self.cfg.toy_eta)
        g = (np.float64(-2.0) * self.H[m]) * self.theta[m]
        self.theta[m] = self.theta[m] + eta * g

    def _step_mlp(self, m, batch=None):
        cfg = self.cfg
        if batch is None:
            off = self._window(m, 0, 0, cfg.pool_rows, cfg.batch)
            x = self.inp.x_pool[off:off + cfg.batch]
            y = self.inp.y_pool[off:off + cfg.batch]
        else:
            x, y = batch
        acts, z = self.forward(m, 0, self.q(x))
        loss, dz = self._loss_and_dz(z, y)
        self.last_loss[m, 0] = loss
        gW, gb, _ = self.backward(m, 0, acts, self.q(dz))
        self._apply(m, 0, gW, gb, self._hp(m, "lr", 0.0))

    def _interp_eps(self, m, j, B):
        """Interpolation coefficient of row b in discriminator update j of this step: word b mod 4 of Philox
        block j * 65536 + b div 4 of the interpolation stream; eps = ((word >> 9) + 1/2) / 2^23, which float32
        holds exactly."""
        eps = np.empty(B, dtype=np.float64)
        for b in range(B):
            w = px.draw(self.seed, m, int(self.t[m]), px.STREAM_INTERP, j * 65536 + (b >> 2))[b & 3]
            eps[b] = ((int(w) >> 9) + 0.5) / 8388608.0
        return eps

    def wgan_gp_critic(self, m, real, fake, eps, lam):
        """The critic's WGAN-GP objective (Section 4.3.1) and its gradient for member m:
            L_D = mean D(fake) - mean D(real) + lam * mean_b (||grad_x D(xhat_b)||_2 - 1)^2,
            xhat_b = eps_b real_b + (1 - eps_b) fake_b.
        The critic is a ReLU MLP, so its input gradient is a chain of matrix products gated by the activation
        masks of the forward pass on xhat (u_L = 1; u_{l-1} = (u_l W_l) * [a_l > 0]; grad_x D = u_0 W_0), and the
        penalty's gradient with respect to W_l follows by differentiating that chain (the masks are piecewise
        constant): with r_b = (2 lam / B)(n_b - 1) / n_b * grad_x D(xhat_b), n_b the norm (r_b = 0 where n_b = 0),
            dv_0 = r,  dv_{l+1} = (dv_l W_l^T) * [a_{l+1} > 0],  dL/dW_l += u_l^T dv_l.
        Biases get no gradient from the penalty.  Operands of every product are rounded like all GEMM operands
        (`self.q`); the input gradient itself is not rounded.  Returns (L_D, gW, gb, xhat)."""
        B = real.shape[0]
        ts = self._tensors_of_stack(1)
        nl = len(ts)
        xhat = self.q(eps[:, None] * real + (1.0 - eps[:, None]) * fake)
        acts, d = self.forward(m, 1, np.concatenate([real, fake, xhat], axis=0))
        d = d.reshape(-1)
        W = [self.q(self.W[m][t]) for t in ts]
        u = [None] * nl
        u[nl - 1] = np.ones((B, 1), dtype=np.float64)
        for l in range(nl - 1, 0, -1):
            u[l - 1] = self.q((u[l] @ W[l]) * (acts[l][2 * B:] > 0.0))
        gx = u[0] @ W[0]
        nrm = np.sqrt((gx * gx).sum(axis=1))
        pen = lam * np.mean((nrm - 1.0) ** 2)
        loss = d[B:2 * B].mean() - d[:B].mean() + pen
        scale = np.where(nrm > 0.0, (2.0 * lam / B) * (nrm - 1.0) / np.where(nrm > 0.0, nrm, 1.0), 0.0)
        dv = [None] * nl
        dv[0] = self.q(scale[:, None] * gx)
        for l in range(nl - 1):
            dv[l + 1] = self.q((dv[l] @ W[l].T) * (acts[l + 1][2 * B:] > 0.0))
        dl = np.concatenate([np.full(B, -1.0 / B), np.full(B, 1.0 / B)]).reshape(-1, 1)
        gW, gb, _ = self.backward(m, 1, [a[:2 * B] for a in acts], self.q(dl))
        for l, t in enumerate(ts):
            gW[t] = gW[t] + u[l].T @ dv[l]
        return loss, gW, gb, xhat

    def _step_wgan_gp(self, m):
        """Section 4.3.1: K critic updates on the WGAN-GP objective, then one generator update on
        L_G = -mean D(G(z))."""
        cfg = self.cfg
        B = cfg.batch
        for j in range(cfg.gan_d_steps):
            offr = self._window(m, j, 0, cfg.pool_rows, B)
            offz = self._window(m, j, 1, cfg.pool_rows, B)
            real = self.q(self.inp.x_pool[offr:offr + B])
            zz = self.q(self.inp.z_pool[offz:offz + B])
            _, gout = self.forward(m, 0, zz)
            fake = self.q(gout)
            loss, gW, gb, _ = self.wgan_gp_critic(m, real, fake, self._interp_eps(m, j, B), cfg.gp_lambda)
            self.last_loss[m, 1] = loss
            self._apply(m, 1, gW, gb, self._hp(m, "lr_d", 0.0))
        offz = self._window(m, cfg.gan_d_steps, 1, cfg.pool_rows, B)
        zz = self.q(self.inp.z_pool[offz:offz + B])
        gacts, gout = self.forward(m, 0, zz)
        fake = self.q(gout)
        dacts, d = self.forward(m, 1, fake)
        self.last_loss[m, 0] = -d.reshape(-1).mean()
        dl = np.full((B, 1), -1.0 / B)
        _, _, dfake = self.backward(m, 1, dacts, self.q(dl), need_wgrad=False, need_input_grad=True)
        gW, gb, _ = self.backward(m, 0, gacts, dfake)
        self._apply(m, 0, gW, gb, self._hp(m, "lr", 0.0))

    def _step_gan(self, m):
        """Section 4.3.1: K discriminator updates, then one generator update.
        Non-saturating logistic losses: L_D = mean softplus(-D(x)) + mean
        softplus(D(G(z))), L_G = mean softplus(-D(G(z)))."""
        cfg = self.cfg
        B = cfg.batch
        for j in range(cfg.gan_d_steps):
            offr = self._window(m, j, 0, cfg.pool_rows, B)
            offz = self._window(m, j, 1, cfg.pool_rows, B)
            real = self.q(self.inp.x_pool[offr:offr + B])
            zz = self.q(self.inp.z_pool[offz:offz + B])
            _, gout = self.forward(m, 0, zz)
            fake = self.q(gout)
            acts, d = self.forward(m, 1, np.concatenate([real, fake], axis=0))
            d = d.reshape(-1)
            self.last_loss[m, 1] = softplus(-d[:B]).mean() + softplus(d[B:]).mean()
            dl = np.concatenate([-sigmoid(-d[:B]), sigmoid(d[B:])]) / B
            gW, gb, _ = self.backward(m, 1, acts, self.q(dl.reshape(-1, 1)))
            self._apply(m, 1, gW, gb, self._hp(m, "lr_d", 0.0))
        offz = self._window(m, cfg.gan_d_steps, 1, cfg.pool_rows, B)
        zz = self.q(self.inp.z_pool[offz:offz + B])
        gacts, gout = self.forward(m, 0, zz)
        fake = self.q(gout)
        dacts, d = self.forward(m, 1, fake)
        d = d.reshape(-1)
        self.last_loss[m, 0] = softplus(-d).mean()
        dl = -sigmoid(-d) / B
        _, _, dfake = self.backward(m, 1, dacts, self.q(dl.reshape(-1, 1)),
                                    need_wgrad=False, need_input_grad=True)
        gW, gb, _ = self.backward(m, 0, gacts, dfake)
        self._apply(m, 0, gW, gb, self._hp(m, "lr", 0.0))

    def step(self, k: int = 1, members=None, batch=None):
        """k steps for all (or the given) members (Algorithm 1, line `step`).  Each member counts its own steps:
        what a member does at a step (which rows it trains on, its interpolation draws) is keyed by its own count
        t[m], so a member that is held back and resumed later continues exactly where it stopped."""
        members = self.members if members is None else [int(m) for m in members]
        for _ in range(k):
            for m in members:
                if self.toy:
                    self._step_toy(m)
                elif self.gan and self.cfg.loss == "wgan_gp":
                    self._step_wgan_gp(m)
                elif self.gan:
                    self._step_gan(m)
                else:
                    self._step_mlp(m, batch)
                self.t[m] += 1

    # ----- `eval` (Eq. 1): a function of the weights only ---------------------
    def eval_member(self, m) -> float:
        cfg = self.cfg
        if self.toy:
            s = np.float64(0.0)
            for i in range(self.theta.shape[1]):
                s = s + self.theta[m, i] * self.theta[m, i]
            return float(np.float64(1.2) - s)
        if self.gan:
            _, x = self.forward(m, 0, self.q(self.inp.x_eval))
            return -energy_distance_to_ring(_f32(x))
        _, z = self.forward(m, 0, self.q(self.inp.x_eval))
        loss, _ = self._loss_and_dz(z, self.inp.y_eval)
        return -loss

    def eval(self, members=None):
        members = self.members if members is None else members
        for m in members:
            self.fitness[m] = self.master(self.eval_member(m))
            self.history[m] = (self.history[m] + [self.fitness[m]])[-HISTORY:]
        return self.fitness.copy()

    # ----- exploit + explore at a ready point ---------------------------------
    def exploit_explore(self, ready=None):
        """One ready point.  `ready[m]` (Algorithm 1: `if ready(p, t, P)`; None = everybody) says which members
        exploit and explore now; the others keep their record but are ranked and can be copied from."""
        cfg = self.cfg
        rule = getattr(cfg, "exploit", "truncation")
        if rule == "tournament":
            src = tournament_select(self.fitness, self.seed, self.round, ready)
        elif rule == "ttest":
            src = ttest_select(self.history, self.seed, self.round, cfg.ttest_alpha, ready)
        else:
            src = truncation_select(self.fitness, self.seed, self.round, cfg.trunc_num, cfg.trunc_den, ready)
        copied = [b for b in range(self.N) if src[b] != b]
        # every copy reads the donor's record as it was BEFORE this ready point (under the tournament rule a
        # donor may itself be a recipient), so the donors are snapshotted first
        old_H, old_fit = self.H.copy(), self.fitness.copy()
        old_hist = [list(h) for h in self.history]
        snap = {int(src[b]): self._snapshot_member(int(src[b])) for b in copied} if cfg.flags & COPY_WEIGHTS else {}
        for b in copied:
            d = int(src[b])
            if cfg.flags & COPY_WEIGHTS:
                self._restore_member(b, snap[d])
            if cfg.flags & COPY_HPARAMS:
                self.H[b] = old_H[d]
        if cfg.flags & EXPLORE:
            for b in copied:
                if getattr(cfg, "explore", "perturb") == "resample":
                    self.H[b] = resample(self.H[b], self.seed, b, self.round, cfg.perturb, cfg.priors,
                                         cfg.resample_prob, cfg.clamp_lo, cfg.clamp_hi)
                    continue
                bits = explore_bits(self.seed, b, self.round, cfg.nh)
                self.H[b] = perturb(self.H[b], bits, cfg.perturb, cfg.factor_lo, cfg.factor_hi,
                                    cfg.clamp_lo, cfg.clamp_hi)
        if cfg.flags & COPY_WEIGHTS:
            for b in copied:
                # eval depends on the weights only, so the copy's performance is the donor's
                self.fitness[b] = old_fit[int(src[b])]
                # ... and so are the scores recorded for it (the t-test compares like with like)
                self.history[b] = list(old_hist[int(src[b])])
        self.src = src
        self.round += 1
        return src

    def _snapshot_member(self, m):
        if self.toy:
            return self.theta[m].copy()
        return ([[x.copy() for x in A[m]] for A in (self.W, self.b, self.o1W, self.o1b, self.o2W, self.o2b)],
                self.scalars[m].copy())

    def _restore_member(self, dst, snap):
        if self.toy:
            self.theta[dst] = snap
            return
        arrays, scalars = snap
        for A, rows in zip((self.W, self.b, self.o1W, self.o1b, self.o2W, self.o2b), arrays):
            A[dst] = [x.copy() for x in rows]
        self.scalars[dst] = scalars

    def best(self) -> int:
        """Member with the highest p; the lowest index wins ties (Algorithm 1, return)."""
        return rank_members(self.fitness)[0]

    # ----- whole run in partial synchrony (Appendix A.1) ----------------------
    def run(self, total_steps=None, on_ready=None):
        cfg = self.cfg
        total = cfg.total_steps if total_steps is None else total_steps
        offsets = getattr(cfg, "ready_offsets", ())
        for _ in range(total):
            self.step(1)
            ready = ready_members(self.step_count, cfg.ready_interval, offsets, self.N)
            if ready.any():
                self.eval()
                if on_ready is not None:
                    on_ready(self, "pre")
                self.exploit_explore(None if ready.all() else ready)
                if on_ready is not None:
                    on_ready(self, "post")
        return self.best()

    # ----- members at their own pace (Section 3: asynchronous workers) ----------
    def run_schedule(self, schedule, on_ready=None):
        """Algorithm 1 with members advancing at different rates.  `schedule` is a sequence of boolean masks, one per
        tick: the members that take one step in that tick (a worker that is pre-empted or slow simply sits out).
        After a tick, a member that stepped and whose OWN count satisfies `ready` exploits and explores; the others
        keep their record but are ranked and can be copied from.  Evaluating everybody at such a point equals
        Algorithm 1's per-step eval, because a member that did not step has not changed."""
        cfg = self.cfg
        offsets = getattr(cfg, "ready_offsets", ())
        for mask in schedule:
            mask = np.asarray(mask, dtype=bool)
            active = [m for m in self.members if mask[m]]
            if not active:
                continue
            self.step(1, members=active)
            ready = ready_members_own(self.t, cfg.ready_interval, offsets) & mask
            if ready.any():
                self.eval()
                if on_ready is not None:
                    on_ready(self, "pre")
                self.exploit_explore(None if ready.all() else ready)
                if on_ready is not None:
                    on_ready(self, "post")
        return self.best()

    # ----- flat views in the interface order ----------------------------------
    # Per stack, per layer: W[out][in] row-major, then b[out]; stacks in order.
    def _flat(self, Ws, bs, m):
        parts = []
        for t in range(len(self.shapes)):
            parts.append(np.asarray(Ws[m][t]).reshape(-1))
            parts.append(np.asarray(bs[m][t]).reshape(-1))
        return np.concatenate(parts)

    def get_flat(self, m) -> Dict[str, np.ndarray]:
        if self.toy:
            return {"w": self.theta[m].copy()}
        return {"w": self._flat(self.W, self.b, m), "opt1": self._flat(self.o1W, self.o1b, m),
                "opt2": self._flat(self.o2W, self.o2b, m), "grad": self._flat(self.gW, self.gb, m),
                "scalars": self.scalars[m].astype(np.float64)}

    def set_flat(self, m, w=None, opt1=None, opt2=None, scalars=None):
        if self.toy:
            if w is not None:
                self.theta[m] = np.asarray(w, dtype=np.float64)
            return
        for vec, Ws, bs in ((w, self.W, self.b), (opt1, self.o1W, self.o1b), (opt2, self.o2W, self.o2b)):
            if vec is None:
                continue
            vec = np.asarray(vec, dtype=np.float32)
            o = 0
            for t, (s, l, fo, fi) in enumerate(self.shapes):
                Ws[m][t] = vec[o:o + fo * fi].reshape(fo, fi).copy()
                o += fo * fi
                bs[m][t] = vec[o:o + fo].copy()
                o += fo
        if scalars is not None:
            self.scalars[m] = np.asarray(scalars, dtype=np.float32)

    @property
    def n_params(self) -> int:
        if self.toy:
            return self.theta.shape[1]
        return sum(fo * fi + fo for (_, _, fo, fi) in self.shapes)


# --------------------------------------------------------------------------
# the member-batched contraction on its own (forward / data-gradient / weight-gradient form)
# --------------------------------------------------------------------------
def grouped_gemm(A, B, bias=None, relu=False, mask=None):
    """C_b[m][n] = sum_k A_b[m][k] B_b[n][k] in float64, then + bias_b[n], max(., 0), and zero
    where mask_b[m][n] <= 0 -- the three epilogues of the layer equations in `forward` / `backward`."""
    out = []
    for b in range(A.shape[0]):
        c = np.asarray(A[b], dtype=np.float64) @ np.asarray(B[b], dtype=np.float64).T
        if bias is not None:
            c = c + np.asarray(bias[b], dtype=np.float64)[None, :]
        if relu:
            c = np.maximum(c, 0.0)
        if mask is not None:
            c = c * (np.asarray(mask[b], dtype=np.float64) > 0.0)
        out.append(c)
    return np.stack(out)
