"""Parity at the full benchmark sizes, in the launch configuration bench.py times (fused optimiser,
gradients not stored): the whole population steps on the GPU, and a sample of members that the
oracle can afford is compared one by one.  Pools are shortened (the window start is still drawn
from the batch stream); population size, layer widths and batch are the benchmark's own."""
import numpy as np
import pytest

from oracle import pbt_oracle as O
from workloads import configs as C
from workloads import get_config, make_inputs

from util import TOL, assert_kept_fractions, assert_state_close, critic_offset, rel_err, tensor_slices

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    import paper_1711_09846_b200 as p
    p.load_library()
    return p


CASES = [("c2", [0, 7, 15], 4096, 2048), ("c3", [0, 13, 31], 4096, 2048),
         ("c4", [0, 11, 23], 4096, 4096), ("c5", [0, 37, 79], 2048, 512), ("c4_wgan", [0, 11, 23], 4096, 4096)]


@pytest.mark.parametrize("name,sample,pool,eval_rows", CASES)
def test_full_size_step_eval_and_exploit(pkg, name, sample, pool, eval_rows):
    cfg = get_config(name).replace(pool_rows=pool, eval_batch=eval_rows)
    inp = make_inputs(cfg)
    gpu = pkg.Population(cfg, inp)                       # the benchmarked configuration
    cpu = O.Population(cfg, inp, only_members=sample)
    t = TOL[cfg.dtype]
    tol = {"w": t["w"], "opt1": t["g"], "opt2": 2 * t["g"]}
    keys = ("w", "opt1") if cfg.optimizer == C.OPT_SGDM else ("w", "opt1", "opt2")
    ftol = 1e-4 if cfg.dtype == C.FP32 else 2e-2

    # initial weights of the sampled members are bit-exact
    for m in sample:
        assert np.array_equal(gpu.get_state(m)["w"], cpu.get_flat(m)["w"])

    gpu.step(1)
    cpu.step(1)
    ll = gpu.last_loss()
    for m in sample:
        g, c = gpu.get_state(m), cpu.get_flat(m)
        assert_state_close(cfg, g, c, keys, tol, what=f"{name} member {m}")
        assert np.array_equal(g["scalars"], c["scalars"])
        ncols = 2 if cfg.model == C.GAN else 1
        got, want = ll[m, :ncols].copy(), cpu.last_loss[m, :ncols].copy()
        got[0] += critic_offset(cfg, g)
        want[0] += critic_offset(cfg, c)
        np.testing.assert_allclose(got, want, rtol=ftol, atol=1e-5)
    assert_kept_fractions(name, 0.98, cfg)

    gpu.eval()
    cpu.eval(sample)
    f = gpu.fitness()
    np.testing.assert_allclose(f[sample], cpu.fitness[sample], rtol=ftol, atol=2e-5)
    assert np.isfinite(f).all()

    # ready point on the GPU's own fitness vector: decisions against the oracle's selection functions,
    # slabs of every recipient against its donor (read back before the copy), the rest untouched
    before = {m: gpu.get_state(m) for m in sample}
    h_before = gpu.hparams()
    gpu.exploit_explore()
    src = gpu.copy_map()
    expect = O.truncation_select(f.astype(np.float32), cpu.seed, 0, cfg.trunc_num, cfg.trunc_den)
    assert np.array_equal(src, expect)
    n_cut = O.n_cut_of(cfg.n_members, cfg.trunc_num, cfg.trunc_den)
    assert (src != np.arange(cfg.n_members)).sum() == n_cut
    h_after = gpu.hparams()
    for b in range(cfg.n_members):
        d = int(src[b])
        if d == b:
            assert np.array_equal(h_after[b], h_before[b])
        else:
            bits = O.explore_bits(cpu.seed, b, 0, cfg.nh)
            want = O.perturb(h_before[d].astype(np.float32), bits, cfg.perturb, cfg.factor_lo, cfg.factor_hi,
                             cfg.clamp_lo, cfg.clamp_hi)
            assert np.array_equal(h_after[b].astype(np.float32), want)
    recipients = [b for b in range(cfg.n_members) if src[b] != b][:2]
    for b in recipients:
        donor = gpu.get_state(int(src[b]))
        got = gpu.get_state(b)
        for key in ("w", "opt1", "opt2", "scalars"):
            assert np.array_equal(got[key], donor[key]), (name, b, key)
        assert got["fitness"] == donor["fitness"]
    for m in sample:
        if src[m] == m:
            now = gpu.get_state(m)
            for key in ("w", "opt1", "opt2"):
                assert np.array_equal(now[key], before[m][key])
    gpu.close()
