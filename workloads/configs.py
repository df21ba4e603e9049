"""Population descriptions (purely declarative; no arithmetic of the method).

Each `PBTConfig` names one population: how many members, what each member is
(toy quadratic, MLP, or generator/discriminator pair), which optimiser it runs,
which optimiser settings are per-member hyperparameters and which are fixed,
and how exploit/explore is parameterised (Section 4.1.1: truncation selection
with a 20 % cut, perturbation by 0.8 / 1.2; Section 4.3.1: 0.5 / 2.0).

The named entries of `CONFIGS` are the five benchmark populations plus small
"mini" versions of each that a CPU finishes in seconds.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

# dtype / model / loss / optimiser tags (strings here; each consumer maps them
# to its own enumeration)
FP64_TOY = "fp64_toy"
FP32 = "fp32"
BF16 = "bf16_fp32master"

TOY = "toy_quadratic"
MLP = "mlp"
GAN = "gan_pair"

LOSS_TOY = "toy"
LOSS_MSE = "mse"
LOSS_CE_HARD = "ce_hard"
LOSS_CE_SOFT = "ce_soft"
LOSS_GAN = "gan_logistic"
LOSS_WGAN_GP = "wgan_gp"   # Section 4.3.1: Wasserstein critic with gradient penalty

OPT_SGD = "sgd_plain"
OPT_SGDM = "sgdm"
OPT_ADAM = "adam"
OPT_RMSPROP = "rmsprop"   # beta2 is the decay of the mean square

COPY_WEIGHTS = 1
COPY_HPARAMS = 2
EXPLORE = 4


@dataclass(frozen=True)
class PBTConfig:
    name: str
    n_members: int
    dtype: str
    model: str
    loss: str
    optimizer: str
    # layer widths: stack 0 = the MLP (or the generator), stack 1 = discriminator
    widths: Tuple[Tuple[int, ...], ...]
    batch: int = 0
    eval_batch: int = 0
    pool_rows: int = 0
    gan_d_steps: int = 0
    # hyperparameter slots: name -> column of the per-member vector h
    slots: Tuple[str, ...] = ()            # e.g. ("lr", "momentum")
    # priors used only to draw the initial h (kind, lo, hi); kind in {"logu", "u", "fixed"}
    priors: Tuple[Tuple[str, float, float], ...] = ()
    perturb: Tuple[bool, ...] = ()         # which slots explore may perturb
    clamp_lo: Tuple[float, ...] = ()
    clamp_hi: Tuple[float, ...] = ()
    # fixed optimiser constants (used when the quantity is not a slot)
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    momentum: float = 0.0
    weight_decay: float = 0.0
    toy_eta: float = 0.0
    toy_theta0: Tuple[float, ...] = ()
    # exploit / explore
    trunc_num: int = 1
    trunc_den: int = 5
    factor_lo: float = 0.8
    factor_hi: float = 1.2
    flags: int = COPY_WEIGHTS | COPY_HPARAMS | EXPLORE
    exploit: str = "truncation"   # or "tournament" (Section 4.3.1 (b)), "ttest" (Section 4.1.1, exploit (a))
    ttest_alpha: float = 0.05     # significance level of the t-test (not stated in the paper)
    explore: str = "perturb"      # or "resample" (Section 4.1.1, explore (b))
    resample_prob: float = 0.25   # probability that a slot is redrawn from its prior (not stated in the paper)
    gp_lambda: float = 10.0       # weight of the gradient penalty (the value of the paper that introduced WGAN-GP)
    ready_interval: int = 1
    ready_offsets: Tuple[int, ...] = ()   # per member: ready when step - offset is a positive multiple of the interval
                                          # (empty: everybody together); staggered ready points as under asynchrony
    total_steps: int = 0
    seed: int = 0

    @property
    def nh(self) -> int:
        return len(self.slots)

    def slot(self, name: str) -> int:
        return self.slots.index(name) if name in self.slots else -1

    def replace(self, **kw) -> "PBTConfig":
        return dataclasses.replace(self, **kw)


INF = math.inf


def _toy() -> PBTConfig:
    # Figure 2: two workers, theta0 = (0.9, 0.9), h = (1,0) and (0,1), exploit
    # every 4 iterations.  Exploit copies theta only; explore perturbs the
    # member's own h.
    return PBTConfig(
        name="c1_toy", n_members=2, dtype=FP64_TOY, model=TOY, loss=LOSS_TOY,
        optimizer=OPT_SGD, widths=((2,),), slots=("h0", "h1"),
        priors=(("fixed", 0.0, 0.0), ("fixed", 0.0, 0.0)),
        perturb=(True, True), clamp_lo=(-INF, -INF), clamp_hi=(INF, INF),
        toy_eta=0.01, toy_theta0=(0.9, 0.9),
        flags=COPY_WEIGHTS | EXPLORE, ready_interval=4, total_steps=40, seed=0)


def _c2(n=16, widths=(256, 512, 512, 1), batch=128, eval_batch=2048, pool=65536,
        interval=100, steps=2000, name="c2_mlp_fp32") -> PBTConfig:
    return PBTConfig(
        name=name, n_members=n, dtype=FP32, model=MLP, loss=LOSS_MSE,
        optimizer=OPT_SGDM, widths=(tuple(widths),), batch=batch,
        eval_batch=eval_batch, pool_rows=pool, slots=("lr", "momentum"),
        priors=(("logu", 1e-4, 1e-1), ("u", 0.5, 0.99)),
        perturb=(True, True), clamp_lo=(-INF, -INF), clamp_hi=(INF, 0.999),
        ready_interval=interval, total_steps=steps, seed=0)


def _c3(n=32, widths=(784, 1024, 1024, 10), batch=256, eval_batch=2048, pool=65536,
        interval=50, steps=5000, name="c3_mlp_bf16") -> PBTConfig:
    return PBTConfig(
        name=name, n_members=n, dtype=BF16, model=MLP, loss=LOSS_CE_HARD,
        optimizer=OPT_ADAM, widths=(tuple(widths),), batch=batch,
        eval_batch=eval_batch, pool_rows=pool, slots=("lr", "beta1", "wd"),
        priors=(("logu", 1e-5, 1e-2), ("u", 0.8, 0.95), ("logu", 1e-6, 1e-3)),
        perturb=(True, True, True), clamp_lo=(-INF, -INF, -INF),
        clamp_hi=(INF, 0.999, INF), beta2=0.999, eps=1e-8,
        ready_interval=interval, total_steps=steps, seed=0)


def _c4(n=24, g=(64, 512, 512, 2), d=(2, 512, 512, 1), batch=512, eval_batch=4096,
        pool=65536, interval=200, steps=2000, name="c4_gan_bf16") -> PBTConfig:
    # Section 4.3.1: K = 5 discriminator updates then one generator update;
    # Appendix A.4: Adam with beta1 = 0.5, beta2 = 0.999, eps = 1e-8.
    return PBTConfig(
        name=name, n_members=n, dtype=BF16, model=GAN, loss=LOSS_GAN,
        optimizer=OPT_ADAM, widths=(tuple(g), tuple(d)), batch=batch,
        eval_batch=eval_batch, pool_rows=pool, gan_d_steps=5,
        slots=("lr", "lr_d"),
        priors=(("logu", 1e-5, 1e-3), ("logu", 1e-5, 1e-3)),
        perturb=(True, True), clamp_lo=(-INF, -INF), clamp_hi=(INF, INF),
        beta1=0.5, beta2=0.999, eps=1e-8,
        ready_interval=interval, total_steps=steps, seed=0)


def _c5(n=80, widths=(2048, 2048, 2048, 2048, 1024), batch=512, eval_batch=2048,
        pool=65536, interval=25, steps=500, name="c5_large_bf16") -> PBTConfig:
    return PBTConfig(
        name=name, n_members=n, dtype=BF16, model=MLP, loss=LOSS_CE_SOFT,
        optimizer=OPT_ADAM, widths=(tuple(widths),), batch=batch,
        eval_batch=eval_batch, pool_rows=pool, slots=("lr", "wd"),
        priors=(("logu", 1e-5, 1e-2), ("logu", 1e-6, 1e-3)),
        perturb=(True, True), clamp_lo=(-INF, -INF), clamp_hi=(INF, INF),
        beta1=0.9, beta2=0.999, eps=1e-8,
        ready_interval=interval, total_steps=steps, seed=0)


CONFIGS: Dict[str, PBTConfig] = {
    "c1": _toy(),
    "c2": _c2(),
    "c3": _c3(),
    "c4": _c4(),
    "c5": _c5(),
    # small versions with the same structure: several tiles plus ragged tails,
    # finished by the CPU oracle in seconds
    "c2_mini": _c2(n=5, widths=(40, 72, 56, 1), batch=24, eval_batch=40, pool=512,
                   interval=3, steps=9, name="c2_mini"),
    "c3_mini": _c3(n=6, widths=(72, 136, 200, 10), batch=40, eval_batch=96, pool=640,
                   interval=3, steps=9, name="c3_mini"),
    "c4_mini": _c4(n=5, g=(16, 72, 136, 2), d=(2, 136, 72, 1), batch=48, eval_batch=160,
                   pool=512, interval=2, steps=6, name="c4_mini"),
    "c5_mini": _c5(n=10, widths=(128, 192, 256, 136, 72), batch=136, eval_batch=200,
                   pool=768, interval=2, steps=6, name="c5_mini"),
    # plain SGD (Section 3's example of `step`): learning rate is the only slot
    "c2_mini_sgd": _c2(n=5, widths=(40, 72, 56, 1), batch=24, eval_batch=40, pool=512, interval=3, steps=6,
                       name="c2_mini_sgd").replace(optimizer=OPT_SGD, slots=("lr",), priors=(("logu", 1e-4, 1e-1),),
                                                   perturb=(True,), clamp_lo=(-INF,), clamp_hi=(INF,)),
    "c3_mini_sgd": _c3(n=6, widths=(72, 136, 200, 10), batch=40, eval_batch=96, pool=640, interval=3, steps=6,
                       name="c3_mini_sgd").replace(optimizer=OPT_SGD, slots=("lr",), priors=(("logu", 1e-4, 1e-1),),
                                                   perturb=(True,), clamp_lo=(-INF,), clamp_hi=(INF,)),
    # RMSProp (the optimiser of the paper's RL experiments) on the same small shapes; learning rate is the only slot
    "c2_mini_rms": _c2(n=5, widths=(40, 72, 56, 1), batch=24, eval_batch=40, pool=512, interval=3, steps=6,
                       name="c2_mini_rms").replace(optimizer=OPT_RMSPROP, slots=("lr",), priors=(("logu", 1e-4, 1e-2),),
                                                   perturb=(True,), clamp_lo=(-INF,), clamp_hi=(INF,), beta2=0.99),
    "c3_mini_rms": _c3(n=6, widths=(72, 136, 200, 10), batch=40, eval_batch=96, pool=640, interval=3, steps=6,
                       name="c3_mini_rms").replace(optimizer=OPT_RMSPROP, slots=("lr",), priors=(("logu", 1e-5, 1e-3),),
                                                   perturb=(True,), clamp_lo=(-INF,), clamp_hi=(INF,), beta2=0.99),
    # the paper's own GAN objective (WGAN-GP) on the GAN shapes
    "c4_mini_wgan": _c4(n=5, g=(16, 72, 136, 2), d=(2, 136, 72, 1), batch=48, eval_batch=160,
                        pool=512, interval=2, steps=4, name="c4_mini_wgan").replace(loss=LOSS_WGAN_GP),
    "c4_mid_wgan": _c4(n=3, g=(64, 512, 512, 2), d=(2, 512, 512, 1), batch=512, eval_batch=512,
                       pool=2048, interval=1, steps=2, name="c4_mid_wgan").replace(loss=LOSS_WGAN_GP),
    "c4_wgan": _c4(name="c4_wgan_gp_bf16").replace(loss=LOSS_WGAN_GP),
    # fp32 compute, one critic update per step: every tensor is updated once per step, so the step's stored gradient
    # says which elements Adam's sign-like early updates make ill-conditioned (the critic's exact +-1/B deltas cancel
    # to zero in many bias-gradient sums)
    "c4_mini_wgan_fp32": _c4(n=4, g=(16, 72, 136, 2), d=(2, 136, 72, 1), batch=48, eval_batch=160, pool=512, interval=2,
                             steps=4, name="c4_mini_wgan_fp32").replace(loss=LOSS_WGAN_GP, dtype=FP32, gan_d_steps=1),
    # staggered ready points (Algorithm 1's per-member `ready`): members exploit at different steps
    "c2_mini_stagger": _c2(n=6, widths=(40, 72, 56, 1), batch=24, eval_batch=40, pool=512, interval=3, steps=9,
                           name="c2_mini_stagger").replace(ready_offsets=(0, 1, 2, 0, 1, 2)),
    "c3_mini_stagger_tournament": _c3(n=6, widths=(72, 136, 200, 10), batch=40, eval_batch=96, pool=640, interval=3, steps=9,
                                      name="c3_mini_stagger_tournament").replace(ready_offsets=(2, 1, 0, 0, 1, 2),
                                                                                 exploit="tournament"),
    # t-test selection and resample-from-prior on the same small shapes
    "c2_mini_ttest": _c2(n=7, widths=(40, 72, 56, 1), batch=24, eval_batch=40, pool=512, interval=2, steps=12,
                         name="c2_mini_ttest").replace(exploit="ttest"),
    "c3_mini_resample": _c3(n=6, widths=(72, 136, 200, 10), batch=40, eval_batch=96, pool=640, interval=3, steps=9,
                            name="c3_mini_resample").replace(explore="resample", resample_prob=0.5),
    # mid-size: every big layer is a multiple of the tensor-core tile so the
    # tcgen05 path is exercised, still seconds on a CPU
    "c3_mid": _c3(n=4, widths=(784, 1024, 1024, 10), batch=256, eval_batch=512, pool=2048,
                  interval=2, steps=4, name="c3_mid"),
    "c5_mid": _c5(n=3, widths=(512, 768, 512, 256), batch=512, eval_batch=512, pool=2048,
                  interval=2, steps=4, name="c5_mid"),
    "c4_mid": _c4(n=3, batch=512, eval_batch=1024, pool=2048, interval=2, steps=4,
                  name="c4_mid"),
}


def get_config(name: str) -> PBTConfig:
    return CONFIGS[name]
