"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Integer / index / hyperparameter results must be bit-exact;
floating-point tensors must agree within tests/util.py's tolerances."""
import math

import numpy as np
import pytest

from oracle import pbt_oracle as O
from workloads import configs as C
from workloads import get_config, make_inputs

from util import TOL, assert_kept_fractions, assert_state_close, critic_offset, oracle_history_arrays, push_oracle_state, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    import paper_1711_09846_b200 as p
    p.load_library()
    return p


def _tol(cfg):
    t = TOL[cfg.dtype]
    return {"w": t["w"], "opt1": t["g"], "opt2": 2 * t["g"], "grad": t["g"]}


# ---------------------------------------------------------------------------
# config 1: the toy of Figure 2, fp64, everything bit-exact
# ---------------------------------------------------------------------------
def test_toy_full_run_bit_exact(pkg):
    cfg = get_config("c1")
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    for t in range(1, cfg.total_steps + 1):
        gpu.step(1)
        cpu.step(1)
        for m in range(2):
            assert np.array_equal(gpu.get_state(m)["w"], cpu.theta[m]), (t, m)
        if t % cfg.ready_interval == 0:
            gpu.eval()
            cpu.eval()
            assert np.array_equal(gpu.fitness(), cpu.fitness), t
            gpu.exploit_explore()
            src = cpu.exploit_explore()
            assert np.array_equal(gpu.copy_map(), src)
            assert np.array_equal(gpu.hparams(), cpu.H)
            assert np.array_equal(gpu.fitness(), cpu.fitness)
            for m in range(2):
                s = gpu.get_state(m)
                assert np.array_equal(s["w"], cpu.theta[m]) and s["round"] == cpu.round and s["step"] == t
    assert gpu.best() == cpu.best()
    gpu.close()


def test_toy_run_matches_oracle_run_and_leaves_the_plateau(pkg):
    cfg = get_config("c1")
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    gpu.run(400)
    cpu.run(400)
    gpu.eval()
    cpu.eval()
    assert np.array_equal(gpu.fitness(), cpu.fitness)
    assert max(gpu.fitness()) > 1.0          # Figure 2: PBT converges towards the optimum 1.2
    gpu.close()


# ---------------------------------------------------------------------------
# exploit / explore decisions: bit-exact for injected fitness vectors
# ---------------------------------------------------------------------------
def _tiny_cfg(n, dtype=C.FP32, flags=C.COPY_WEIGHTS | C.COPY_HPARAMS | C.EXPLORE, num=1, den=5):
    base = get_config("c3_mini" if dtype == C.BF16 else "c2_mini")
    return base.replace(n_members=n, flags=flags, trunc_num=num, trunc_den=den, name=f"tiny{n}")


@pytest.mark.parametrize("n", [1, 2, 3, 5, 16, 24, 32, 45, 80, 200])
@pytest.mark.parametrize("dtype", [C.FP32, C.BF16])
def test_select_copy_explore_bit_exact(pkg, n, dtype):
    cfg = _tiny_cfg(n, dtype)
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    rng = np.random.default_rng(n)
    gpu.step(1)
    cpu.step(1)
    push_oracle_state(gpu, cpu)
    for rnd in range(4):
        f = rng.standard_normal(n).astype(np.float32)
        if rnd == 1:
            f = np.round(f)                           # many exact ties, signed zeros
            f[::3] = -0.0
        if rnd == 2 and n > 2:
            f[rng.integers(0, n)] = np.nan
            f[rng.integers(0, n)] = -np.inf
        cpu.fitness[:] = f
        gpu.set_fitness(f.astype(np.float64))
        before = [gpu.get_state(m) for m in range(n)]
        gpu.exploit_explore()
        src = cpu.exploit_explore()
        assert np.array_equal(gpu.copy_map(), src)
        assert np.array_equal(gpu.hparams(), cpu.H.astype(np.float64))
        assert np.array_equal(gpu.fitness(), cpu.fitness.astype(np.float64), equal_nan=True)
        for m in range(n):
            now = gpu.get_state(m)
            assert now["round"] == cpu.round
            d = int(src[m])
            for key in ("w", "opt1", "opt2", "scalars"):
                assert np.array_equal(now[key], before[d][key]), (rnd, m, key)   # copy is bit-exact
                assert np.array_equal(now[key], cpu.get_flat(m)[key]), (rnd, m, key)
    gpu.close()


@pytest.mark.parametrize("n", [1, 2, 3, 6, 16, 45, 80, 200])
@pytest.mark.parametrize("dtype", [C.FP32, C.BF16])
def test_binary_tournament_bit_exact(pkg, n, dtype):
    """Section 4.3.1 (b): partners, decisions, copied records (donors that are recipients too are read before
    they are overwritten), explored hyperparameters and fitness, against the oracle, bit for bit."""
    cfg = _tiny_cfg(n, dtype).replace(exploit="tournament")
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    rng = np.random.default_rng(100 + n)
    gpu.step(1)
    cpu.step(1)
    push_oracle_state(gpu, cpu)
    chains = 0
    for rnd in range(5):
        f = rng.standard_normal(n).astype(np.float32)
        if rnd == 1:
            f = np.round(f)                               # ties: nobody copies an equal
        if rnd == 2 and n > 2:
            f[rng.integers(0, n)] = np.nan
        cpu.fitness[:] = f
        gpu.set_fitness(f.astype(np.float64))
        gpu.exploit_explore()
        src = cpu.exploit_explore()
        chains += sum(1 for i in range(n) if src[i] != i and src[src[i]] != src[i])
        assert np.array_equal(gpu.copy_map(), src)
        assert np.array_equal(gpu.hparams(), cpu.H.astype(np.float64))
        assert np.array_equal(gpu.fitness(), cpu.fitness.astype(np.float64), equal_nan=True)
        for m in range(n):
            now, ref = gpu.get_state(m), cpu.get_flat(m)
            assert now["round"] == cpu.round
            for key in ("w", "opt1", "opt2", "scalars"):
                assert np.array_equal(now[key], ref[key]), (rnd, m, key)
    if n >= 16:
        assert chains > 0                                 # the multi-pass copy was exercised
    gpu.close()


def test_toy_with_tournament_matches_oracle(pkg):
    cfg = get_config("c1").replace(exploit="tournament", n_members=2)
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    gpu.run(40)
    cpu.run(40)
    for m in range(2):
        assert np.array_equal(gpu.get_state(m)["w"], cpu.theta[m])
    assert np.array_equal(gpu.hparams(), cpu.H)
    gpu.close()


def test_toy_select_explore_bit_exact_at_the_largest_population(pkg):
    """The fp64 instantiation of the select / explore kernel with one member per thread at the largest population
    the library takes (1024), against the oracle, bit for bit."""
    n = 1024
    cfg = get_config("c1").replace(n_members=n, flags=C.COPY_WEIGHTS | C.COPY_HPARAMS | C.EXPLORE, name="toy1024")
    inp = make_inputs(cfg)
    h0 = np.random.default_rng(3).random((n, cfg.nh)) + 0.5
    inp = type(inp)(**{**inp.__dict__, "init_hparams": h0})
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    rng = np.random.default_rng(4)
    for rnd in range(3):
        gpu.step(2)
        cpu.step(2)
        f = np.round(rng.standard_normal(n), 2)          # ties included
        cpu.fitness[:] = f
        gpu.set_fitness(f)
        gpu.exploit_explore()
        src = cpu.exploit_explore()
        assert np.array_equal(gpu.copy_map(), src)
        assert np.array_equal(gpu.hparams(), cpu.H)
        assert np.array_equal(gpu.fitness(), cpu.fitness)
        for m in range(0, n, 37):
            assert np.array_equal(gpu.get_state(m)["w"], cpu.theta[m])
    gpu.close()


@pytest.mark.parametrize("flags", [0, C.COPY_WEIGHTS, C.COPY_HPARAMS | C.EXPLORE, C.COPY_WEIGHTS | C.EXPLORE])
def test_flag_variants_bit_exact(pkg, flags):
    cfg = _tiny_cfg(10, C.FP32, flags=flags, num=2, den=5)
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    f = np.arange(10, dtype=np.float32)[::-1].copy()
    cpu.fitness[:] = f
    gpu.set_fitness(f.astype(np.float64))
    gpu.exploit_explore()
    src = cpu.exploit_explore()
    assert np.array_equal(gpu.copy_map(), src) and (src != np.arange(10)).sum() == 4
    assert np.array_equal(gpu.hparams(), cpu.H.astype(np.float64))
    assert np.array_equal(gpu.fitness(), cpu.fitness.astype(np.float64))
    for m in range(10):
        assert np.array_equal(gpu.get_state(m)["w"], cpu.get_flat(m)["w"])
    gpu.close()


@pytest.mark.parametrize("rule", ["truncation", "tournament", "ttest"])
@pytest.mark.parametrize("n", [2, 5, 33, 80, 200, 1024])
def test_ready_mask_bit_exact(pkg, n, rule):
    """Algorithm 1's per-member `ready`: with a mask only ready members copy and explore; copy map, copied records,
    hyperparameters, fitness and (t-test) score histories against the oracle, bit for bit, for random masks, the
    empty mask and the full mask."""
    cfg = _tiny_cfg(n, C.FP32).replace(exploit=rule)
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    rng = np.random.default_rng(100 + n)
    gpu.step(1)
    cpu.step(1)
    push_oracle_state(gpu, cpu)
    masks = [rng.random(n) < 0.5, np.zeros(n, dtype=bool), rng.random(n) < 0.2, np.ones(n, dtype=bool), rng.random(n) < 0.8]
    for rnd, mask in enumerate(masks):
        f = rng.standard_normal(n).astype(np.float32)
        cpu.fitness[:] = f
        gpu.set_fitness(f.astype(np.float64))
        if rule == "ttest":
            for m in range(n):
                cnt = int(rng.integers(0, 11))
                cpu.history[m] = [np.float32(x) for x in rng.standard_normal(cnt) + (2.0 if m % 3 == 0 else 0.0)]
            ch, cc = oracle_history_arrays(cpu)
            gpu.set_history(ch, cc)
        before = [gpu.get_state(m) for m in range(n)]
        h_before = gpu.hparams()
        gpu.exploit_explore(mask)
        src = cpu.exploit_explore(mask)
        assert np.array_equal(gpu.copy_map(), src)
        assert all(src[m] == m for m in range(n) if not mask[m])
        assert np.array_equal(gpu.hparams(), cpu.H.astype(np.float64))
        assert np.array_equal(gpu.fitness(), cpu.fitness.astype(np.float64))
        if rule == "ttest":
            (gh, gc), (ch, cc) = gpu.history(), oracle_history_arrays(cpu)
            assert np.array_equal(gc, cc) and np.array_equal(gh, ch)
        for m in range(n):
            now = gpu.get_state(m)
            assert now["round"] == cpu.round
            for key in ("w", "opt1", "opt2", "scalars"):
                assert np.array_equal(now[key], before[int(src[m])][key]), (rnd, m, key)
            if not mask[m]:
                assert np.array_equal(gpu.hparams()[m], h_before[m])
    gpu.close()


def test_staggered_run_matches_the_oracle_schedule(pkg):
    """Population.run with staggered ready points: the host schedule (which members are ready at which step) is the
    binding's own; the copy maps it produces must be the oracle's when both see the same fitness."""
    cfg = get_config("c2_mini_stagger")
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    seen = []
    orig = gpu.exploit_explore

    def spy(ready=None):
        seen.append((None if ready is None else tuple(bool(r) for r in ready)))
        orig(ready)
    gpu.exploit_explore = spy
    gpu.run()
    want = []
    for t in range(1, cfg.total_steps + 1):
        r = O.ready_members(t, cfg.ready_interval, cfg.ready_offsets, cfg.n_members)
        if r.any():
            want.append(None if r.all() else tuple(bool(x) for x in r))
    assert seen == want
    assert gpu.get_state(0)["step"] == cfg.total_steps and gpu.get_state(0)["round"] == len(want)
    gpu.close()


@pytest.mark.parametrize("name", ["c1", "c2_mini_ttest", "c3_mini", "c4_mini_wgan", "c3_mini_stagger_tournament"])
def test_checkpoint_resume_is_bit_exact(pkg, name, tmp_path):
    """Appendix A.1: members are restored from checkpoints.  A population saved after some ready points and loaded
    into a fresh handle continues exactly like the one that kept running: records, score histories, counters and
    the decisions of the following ready points, bit for bit."""
    cfg = get_config(name)
    inp = make_inputs(cfg)
    iv = cfg.ready_interval
    a = pkg.Population(cfg, inp)
    a.run(2 * iv + 1)                       # stops in the middle of an interval
    path = str(tmp_path / "pop.npz")
    a.save(path)
    b = pkg.Population(cfg, inp)
    b.load(path)
    c = pkg.Population(cfg, inp)            # never interrupted
    for pop in (a, b, c):
        pop.run(4 * iv + 1)                 # absolute target: the ready points fall on the same steps for all three
    sa = a.state_dict()
    for other in (b, c):
        so = other.state_dict()
        assert set(sa) == set(so)
        for key in sa:
            assert np.array_equal(sa[key], so[key], equal_nan=True), (name, key)
        assert np.array_equal(a.copy_map(), other.copy_map())
    assert int(sa["step"]) == 4 * iv + 1
    for pop in (a, b, c):
        pop.close()


@pytest.mark.parametrize("name", ["c2_mini", "c3_mini", "c4_mini", "c4_mini_wgan", "c5_mini", "c3_mid", "c5_mid", "c4_mid_wgan",
                                  "c2_mini_ttest", "c3_mini_stagger_tournament"])
def test_no_kernel_writes_outside_the_workspace(pkg, name):
    """Every kernel of a run (steps, evaluations, ready points; ragged and tile-sized shapes) stays inside the
    workspace it was given: 1 MiB guard bands on both sides keep their fill, and the device status word stays 0."""
    cfg = get_config(name)
    inp = make_inputs(cfg)
    for kw in ({"keep_grad": True, "fuse_adam": False}, {}):
        gpu = pkg.Population(cfg, inp, guard_bytes=1 << 20, **kw)
        assert gpu.guards_intact()
        gpu.run(2 * cfg.ready_interval)
        gpu.eval()
        assert np.isfinite(gpu.fitness()).all()       # also reads the status word
        assert gpu.guards_intact(), (name, kw)
        gpu.close()


def test_ready_point_log_and_lineages(pkg):
    """The ready-point records of a run: one per ready point, copy maps consistent with the hyperparameter traces
    (only members that copied change h), and the number of surviving initial lineages never grows (Section 4.4)."""
    cfg = get_config("c3_mini").replace(total_steps=12)
    inp = make_inputs(cfg)
    gpu = pkg.Population(cfg, inp)
    log = []
    gpu.run(log=log)
    assert [r["step"] for r in log] == list(range(cfg.ready_interval, 13, cfg.ready_interval))
    alive = cfg.n_members
    for k, rec in enumerate(log):
        n_cut = O.n_cut_of(cfg.n_members, cfg.trunc_num, cfg.trunc_den)
        assert np.array_equal(rec["src"], O.truncation_select(rec["fitness"].astype(np.float32), cfg.seed, k,
                                                              cfg.trunc_num, cfg.trunc_den))
        assert (rec["src"] != np.arange(cfg.n_members)).sum() == n_cut
        for m in range(cfg.n_members):
            if rec["src"][m] == m:
                assert np.array_equal(rec["hparams_after"][m], rec["hparams_before"][m])
        now = len(set(pkg.Population.ancestors(log[:k + 1], cfg.n_members)))
        assert now <= alive
        alive = now
    gpu.close()


# ---------------------------------------------------------------------------
# initial population
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["c2_mini", "c3_mini", "c4_mini", "c5_mini", "c4_mini_wgan"])
def test_initial_population_bit_exact(pkg, name):
    cfg = get_config(name)
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    for m in range(cfg.n_members):
        g, c = gpu.get_state(m), cpu.get_flat(m)
        assert np.array_equal(g["w"], c["w"])
        assert not g["opt1"].any() and not g["opt2"].any()
        assert list(g["scalars"]) == [1.0] * 4 and g["step"] == 0 and g["round"] == 0
    assert np.array_equal(gpu.hparams(), cpu.H.astype(np.float64))
    gpu.close()


def _check_optimizer_arithmetic(cfg, s0, s1, h):
    """The fused optimiser kernel against the oracle's update formula on the GPU's own
    gradient and pre-step state: every element, well conditioned or not."""
    g = s1["grad"].astype(np.float64)
    w0, m0, v0 = (s0[k].astype(np.float64) for k in ("w", "opt1", "opt2"))
    lr = h[cfg.slot("lr")]
    if cfg.optimizer == C.OPT_SGD:
        np.testing.assert_allclose(s1["w"], O.sgd_update(w0, g, lr), rtol=2e-6, atol=1e-5 * lr)
        assert not s1["opt1"].any() and not s1["opt2"].any()
        return
    if cfg.optimizer == C.OPT_SGDM:
        w, m = O.sgdm_update(w0, m0, g, lr, h[cfg.slot("momentum")])
        v = v0
    elif cfg.optimizer == C.OPT_RMSPROP:
        w, m = O.rmsprop_update(w0, m0, g, lr, float(np.float32(cfg.beta2)), float(np.float32(cfg.eps)))
        v = v0
        np.testing.assert_allclose(s1["opt1"], m, rtol=2e-6, atol=2e-7 * max(np.abs(m0).max(), (g * g).max()))
        np.testing.assert_allclose(s1["w"], w, rtol=2e-6, atol=1e-5 * lr)
        return
    else:
        b1 = h[cfg.slot("beta1")] if cfg.slot("beta1") >= 0 else float(np.float32(cfg.beta1))
        wd = h[cfg.slot("wd")] if cfg.slot("wd") >= 0 else cfg.weight_decay
        w, m, v = O.adam_update(w0, m0, v0, g, lr, b1, float(np.float32(cfg.beta2)), float(np.float32(cfg.eps)),
                                wd, s1["scalars"][0], s1["scalars"][1])
    # fp32 roundings of the two terms of each moment: relative to the larger term, not to a cancelled sum
    np.testing.assert_allclose(s1["opt1"], m, rtol=2e-6, atol=2e-7 * max(np.abs(m0).max(), np.abs(g).max()))
    np.testing.assert_allclose(s1["opt2"], v, rtol=2e-6, atol=2e-7 * max(np.abs(v0).max(), (g * g).max()))
    np.testing.assert_allclose(s1["w"], w, rtol=2e-6, atol=1e-5 * lr)


# ---------------------------------------------------------------------------
# step / eval parity, step by step, re-seeding the GPU from the oracle at ready points
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["c2_mini", "c3_mini", "c4_mini", "c5_mini", "c3_mid", "c5_mid", "c4_mid", "c2_mini_rms",
                                  "c2_mini_sgd", "c3_mini_sgd",
                                  "c3_mini_rms", "c2_mini_ttest", "c3_mini_resample", "c4_mini_wgan", "c4_mini_wgan_fp32",
                                  "c4_mid_wgan", "c2_mini_stagger", "c3_mini_stagger_tournament"])
def test_step_eval_exploit_parity(pkg, name):
    cfg = get_config(name)
    inp = make_inputs(cfg)
    # keep_grad matters only for the fused variant (exercised below); the default path always stores gradients
    gpu, cpu = pkg.Population(cfg, inp, keep_grad=True), O.Population(cfg, inp)
    tol = _tol(cfg)
    ftol = 1e-4 if cfg.dtype == C.FP32 else 2e-2
    keys = ("w", "opt1", "opt2", "grad") if cfg.optimizer == C.OPT_ADAM else ("w", "opt1", "grad")
    for t in range(1, cfg.total_steps + 1):
        before = [gpu.get_state(m) for m in range(cfg.n_members)]
        h_now = gpu.hparams()
        gpu.step(1)
        cpu.step(1)
        ll = gpu.last_loss()
        for m in range(cfg.n_members):
            g, c = gpu.get_state(m), cpu.get_flat(m)
            assert g["step"] == t
            assert_state_close(cfg, g, c, keys, tol, what=f"{name} step {t} member {m}")
            if cfg.model != C.GAN:
                _check_optimizer_arithmetic(cfg, before[m], g, h_now[m])
            assert np.array_equal(g["scalars"], c["scalars"])
            ncols = 2 if cfg.model == C.GAN else 1
            got, want = ll[m, :ncols].copy(), cpu.last_loss[m, :ncols].copy()
            got[0] += critic_offset(cfg, g)
            want[0] += critic_offset(cfg, c)
            np.testing.assert_allclose(got, want, rtol=ftol, atol=1e-5)
        ready = O.ready_members(t, cfg.ready_interval, cfg.ready_offsets, cfg.n_members)
        if ready.any():
            mask = None if ready.all() else ready
            gpu.eval()
            cpu.eval()
            np.testing.assert_allclose(gpu.fitness(), cpu.fitness, rtol=ftol, atol=2e-5)
            # selection is compared on identical fitness vectors (and score histories)
            gpu.set_fitness(cpu.fitness.astype(np.float64))
            if cfg.exploit == "ttest":
                (gh, gc), (ch, cc) = gpu.history(), oracle_history_arrays(cpu)
                assert np.array_equal(gc, cc)
                np.testing.assert_allclose(gh[:, -1 if cc[0] == 10 else cc[0] - 1], cpu.fitness, rtol=ftol, atol=2e-5)
                gpu.set_history(ch, cc)
            gpu.exploit_explore(mask)
            src = cpu.exploit_explore(mask)
            assert np.array_equal(gpu.copy_map(), src)
            assert np.array_equal(gpu.hparams(), cpu.H.astype(np.float64))
            if cfg.exploit == "ttest":
                (gh, gc), (ch, cc) = gpu.history(), oracle_history_arrays(cpu)
                assert np.array_equal(gc, cc) and np.array_equal(gh, ch)
        # every step starts from identical state: training is chaotic, parity is per step
        push_oracle_state(gpu, cpu)
    assert_kept_fractions(name, 0.98, cfg)
    gpu.close()


@pytest.mark.parametrize("name", ["c2_mini", "c2_mini_rms", "c3_mini", "c3_mid", "c5_mid", "c4_mini", "c4_mid", "c4_mini_wgan",
                                  "c4_mid_wgan", "c4_mini_wgan_fp32"])
@pytest.mark.parametrize("fuse", [True, False])
def test_backward_on_two_streams_is_bit_identical(pkg, name, fuse):
    """A layer's weight and bias gradients beside its data gradient on a second stream (captured into the replayed
    step as parallel branches): the same kernels on the same inputs, so every tensor, the gradients included,
    and the fitness must equal the single-stream run bit for bit; plain (not replayed) steps and own-pace steps of
    a subset too."""
    cfg = get_config(name)
    inp = make_inputs(cfg)
    pops = [pkg.Population(cfg, inp, keep_grad=True, fuse_adam=fuse, backward_streams=k) for k in (1, 2)]
    active = np.zeros(cfg.n_members, dtype=np.uint8)
    active[1:cfg.n_members - 1] = 1
    for pop in pops:
        pop.step(3)                          # replayed graph
        pop.step_subset(active, 1)           # plain launches on a member window
        pop.eval()
        pop.exploit_explore()
        pop.step(2)
        pop.eval()
    a, b = pops
    assert np.array_equal(a.fitness(), b.fitness())
    for m in range(cfg.n_members):
        sa, sb = a.get_state(m), b.get_state(m)
        assert sa["step"] == sb["step"]
        for key in ("w", "opt1", "opt2", "scalars", "grad"):
            assert np.array_equal(sa[key], sb[key]), (name, m, key)
    for pop in pops:
        pop.close()


@pytest.mark.parametrize("name", ["c3_mid", "c5_mid", "c4_mid", "c5_mini", "c4_mid_wgan"])
def test_fused_update_is_the_same_with_and_without_stored_gradients(pkg, name):
    """The benchmarked configuration never writes the weight gradient of tensor-core layers to HBM.
    The fused and the separate optimiser pass, with and without stored gradients, must agree bit for bit."""
    cfg = get_config(name)
    inp = make_inputs(cfg)
    pops = [pkg.Population(cfg, inp, keep_grad=True, fuse_adam=False),
            pkg.Population(cfg, inp, keep_grad=True, fuse_adam=True),
            pkg.Population(cfg, inp, keep_grad=False, fuse_adam=True)]
    for pop in pops:
        pop.step(3)
        pop.eval()
    a = pops[0]
    for b in pops[1:]:
        assert np.array_equal(a.fitness(), b.fitness())
        for m in range(cfg.n_members):
            sa, sb = a.get_state(m), b.get_state(m)
            for key in ("w", "opt1", "opt2", "scalars"):
                assert np.array_equal(sa[key], sb[key]), (name, m, key)
    for pop in pops:
        pop.close()


def test_free_running_interval_stays_within_tolerance(pkg):
    """A whole ready interval without re-seeding (fp32: errors do not compound beyond the bar)."""
    cfg = get_config("c2_mini")
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    gpu.step(cfg.ready_interval)
    cpu.step(cfg.ready_interval)
    for m in range(cfg.n_members):
        assert_state_close(cfg, gpu.get_state(m), cpu.get_flat(m), ("w",), {"w": 1e-5})
    gpu.close()


@pytest.mark.parametrize("name", ["c3_mini", "c5_mini", "c4_mini", "c4_mini_wgan"])
def test_free_running_interval_bf16(pkg, name):
    """A whole ready interval without re-seeding, bf16 compute: the fitness that selection sees and
    every weight matrix stay within the bar.  (Bias vectors start at zero and are O(lr) after a few
    Adam steps, so a single near-zero gradient whose sign differs moves them by more than 2 % of
    their own norm; they are covered by the per-step test above.)"""
    cfg = get_config(name)
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    gpu.step(cfg.ready_interval)
    cpu.step(cfg.ready_interval)
    from util import tensor_slices
    for m in range(cfg.n_members):
        g, c = gpu.get_state(m), cpu.get_flat(m)
        for tname, sl in tensor_slices(cfg):
            if ".W" in tname:
                assert rel_err(g["w"][sl], c["w"][sl]) <= 2e-2, (name, m, tname)
    gpu.eval()
    cpu.eval()
    np.testing.assert_allclose(gpu.fitness(), cpu.fitness, rtol=2e-2, atol=1e-4)
    gpu.close()


def test_exploit_off_members_are_isolated_and_runs_are_deterministic(pkg):
    cfg = get_config("c3_mini").replace(flags=0)
    inp = make_inputs(cfg)
    a, b = pkg.Population(cfg, inp), pkg.Population(cfg, inp)
    a.run(6)
    # b: same seed, same steps -> bit-identical (fixed-order reductions, no float atomics)
    b.run(6)
    for m in range(cfg.n_members):
        sa, sb = a.get_state(m), b.get_state(m)
        for key in ("w", "opt1", "opt2", "grad"):
            assert np.array_equal(sa[key], sb[key])
    # a member's trajectory does not depend on the others: scramble every other member of b and re-run
    c = pkg.Population(cfg, inp)
    junk = np.random.default_rng(0).standard_normal(c.n_params).astype(np.float32)
    for m in range(1, cfg.n_members):
        c.set_state(m, w=junk)
    c.run(6)
    s0, c0 = a.get_state(0), c.get_state(0)
    for key in ("w", "opt1", "opt2"):
        assert np.array_equal(s0[key], c0[key])
    assert np.array_equal(a.hparams(), np.asarray(inp.init_hparams))
    for p in (a, b, c):
        p.close()


def test_supplied_batch_matches_oracle(pkg):
    import torch
    cfg = get_config("c2_mini")
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    rng = np.random.default_rng(5)
    x = rng.standard_normal((cfg.batch, cfg.widths[0][0])).astype(np.float32)
    y = rng.standard_normal((cfg.batch, 1)).astype(np.float32)
    xd = torch.from_numpy(np.tile(x, (cfg.n_members, 1, 1))).cuda().contiguous()
    yd = torch.from_numpy(np.tile(y, (cfg.n_members, 1, 1))).cuda().contiguous()
    gpu.set_batch(xd, yd)
    gpu.step(1)
    cpu.step(1, batch=(x, y))
    for m in range(cfg.n_members):
        assert_state_close(cfg, gpu.get_state(m), cpu.get_flat(m), ("w", "grad"), {"w": 1e-5, "grad": 1e-4})
    # the next step goes back to pool windows
    gpu.step(1)
    cpu.step(1)
    for m in range(cfg.n_members):
        assert_state_close(cfg, gpu.get_state(m), cpu.get_flat(m), ("w",), {"w": 1e-5})
    gpu.close()


def test_host_fed_steps_plain_and_prefetched_agree(pkg):
    import torch
    cfg = get_config("c3_mini")
    inp = make_inputs(cfg)
    rng = np.random.default_rng(9)
    xs = [torch.from_numpy(rng.random((cfg.n_members, cfg.batch, cfg.widths[0][0])).astype(np.float32)).bfloat16().pin_memory()
          for _ in range(3)]
    ys = [torch.from_numpy(rng.integers(0, 10, size=(cfg.n_members, cfg.batch)).astype(np.int32)).pin_memory() for _ in range(3)]
    a, b = pkg.Population(cfg, inp), pkg.Population(cfg, inp)
    la = [a.step_host(x, y).copy() for x, y in zip(xs, ys)]
    b.prefetch_host_batch(xs[0], ys[0])
    lb = []
    for j in range(3):
        b.step_prefetched(wait=False)
        if j + 1 < 3:
            b.prefetch_host_batch(xs[j + 1], ys[j + 1])      # uploads while step j runs
            with pytest.raises(pkg.PbtError) as e:           # one batch may be pending at a time
                b.prefetch_host_batch(xs[j + 1], ys[j + 1])
            assert e.value.code == 6
        lb.append(b.last_loss().copy())
    with pytest.raises(pkg.PbtError) as e:
        b.step_prefetched()
    assert e.value.code == 6
    assert all(np.array_equal(p, q) for p, q in zip(la, lb))
    b.step(1)                                                 # pool-window steps still work after the buffer swaps
    a.step(1)
    for m in range(cfg.n_members):
        sa, sb = a.get_state(m), b.get_state(m)
        for key in ("w", "opt1", "opt2"):
            assert np.array_equal(sa[key], sb[key])
    a.close()
    b.close()


def test_ready_point_is_enqueue_only_under_the_tournament_rule(pkg):
    """step -> eval -> ready point (binary tournament, whose copies may need several passes) -> step, enqueued
    behind a busy stream: none of the calls waits for the device (the number of copy passes stays on the device),
    and the result is the oracle's."""
    import torch
    cfg = _tiny_cfg(24, C.FP32).replace(exploit="tournament")
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    gpu.step(1)
    cpu.step(1)
    push_oracle_state(gpu, cpu)
    gpu.synchronize()
    done = torch.cuda.Event()
    with torch.cuda.stream(gpu.stream):
        torch.cuda._sleep(int(1.5e9))            # keeps the stream busy for most of a second
    gpu.step(2)
    gpu.eval()
    gpu.exploit_explore()
    gpu.step(1)
    done.record(gpu.stream)
    assert not done.query(), "a call of the training loop waited for the device"
    gpu.synchronize()
    cpu.step(2)
    cpu.eval()
    src = cpu.exploit_explore()
    cpu.step(1)
    assert np.array_equal(gpu.copy_map(), src)
    assert (src != np.arange(cfg.n_members)).sum() > 0
    assert np.array_equal(gpu.hparams(), cpu.H.astype(np.float64))
    for m in range(cfg.n_members):
        g = gpu.get_state(m)
        assert g["step"] == 4 and g["round"] == 1
        assert_state_close(cfg, g, cpu.get_flat(m), ("w", "opt1"), {"w": 1e-5, "opt1": 1e-4}, what="enqueue_only")
    gpu.close()


def test_prefetched_steps_after_pool_steps_match_the_oracle(pkg):
    """pbt_step(k) followed at once by two prefetched host-fed steps without waiting: the uploads must not land in
    row buffers that the still-running pool steps read (the spare buffer pair of the second upload is the pair the
    pool steps used)."""
    import torch
    cfg = get_config("c2_mini")
    inp = make_inputs(cfg)
    gpu, cpu = pkg.Population(cfg, inp), O.Population(cfg, inp)
    rng = np.random.default_rng(11)
    xs = [rng.standard_normal((cfg.batch, cfg.widths[0][0])).astype(np.float32) for _ in range(2)]
    ys = [rng.standard_normal((cfg.batch, 1)).astype(np.float32) for _ in range(2)]
    hx = [torch.from_numpy(np.tile(x, (cfg.n_members, 1, 1))).contiguous().pin_memory() for x in xs]
    hy = [torch.from_numpy(np.tile(y, (cfg.n_members, 1, 1))).contiguous().pin_memory() for y in ys]
    k = 40
    gpu.step(k)
    gpu.prefetch_host_batch(hx[0], hy[0])
    gpu.step_prefetched(wait=False)
    gpu.prefetch_host_batch(hx[1], hy[1])
    gpu.step_prefetched(wait=False)
    gpu.synchronize()
    cpu.step(k)
    cpu.step(1, batch=(xs[0], ys[0]))
    cpu.step(1, batch=(xs[1], ys[1]))
    for m in range(cfg.n_members):
        g = gpu.get_state(m)
        assert g["step"] == k + 2
        assert_state_close(cfg, g, cpu.get_flat(m), ("w",), {"w": 1e-5}, what="prefetch_after_pool_steps")
    gpu.close()


def test_degenerate_populations_and_empty_calls(pkg):
    """step(0) and an all-inactive subset step change nothing; a population of one steps like member 0 of a larger
    one and its ready point is a no-op; a fitness vector of NaNs and one of equal values select by index alone."""
    cfg = get_config("c3_mini")
    inp = make_inputs(cfg)
    gpu = pkg.Population(cfg, inp)
    before = [gpu.get_state(m) for m in range(cfg.n_members)]
    gpu.step(0)
    gpu.step_subset(np.zeros(cfg.n_members, dtype=bool), 3)
    for m in range(cfg.n_members):
        now = gpu.get_state(m)
        assert now["step"] == 0
        for key in ("w", "opt1", "opt2", "scalars"):
            assert np.array_equal(now[key], before[m][key])
    cpu = O.Population(cfg, inp)
    for f in (np.full(cfg.n_members, np.nan), np.full(cfg.n_members, 0.25)):
        cpu.fitness[:] = f
        gpu.set_fitness(f)
        gpu.exploit_explore()
        src = cpu.exploit_explore()
        assert np.array_equal(gpu.copy_map(), src)
        assert (src != np.arange(cfg.n_members)).sum() == O.n_cut_of(cfg.n_members, cfg.trunc_num, cfg.trunc_den)
        assert np.array_equal(gpu.hparams(), cpu.H.astype(np.float64))
    gpu.close()
    one = cfg.replace(n_members=1)
    inp1 = make_inputs(one)
    solo, many = pkg.Population(one, inp1), pkg.Population(cfg, inp)
    many.set_hparams(np.tile(np.asarray(inp1.init_hparams, dtype=np.float64), (cfg.n_members, 1)))
    solo.step(2)
    many.step(2)
    for key in ("w", "opt1", "opt2"):
        assert np.array_equal(solo.get_state(0)[key], many.get_state(0)[key])
    solo.eval()
    solo.exploit_explore()
    assert list(solo.copy_map()) == [0] and solo.get_state(0)["round"] == 1
    solo.close()
    many.close()


def test_invalid_arguments_are_reported_not_fatal(pkg):
    cfg = get_config("c2_mini")
    inp = make_inputs(cfg)
    gpu = pkg.Population(cfg, inp)
    with pytest.raises(pkg.PbtError) as e:
        gpu.get_state(99)
    assert e.value.code == 1
    with pytest.raises(pkg.PbtError):
        gpu.step(-1)
    gpu.step(1)      # the handle is still usable
    gpu.close()
    bad = cfg.replace(widths=((40, 0, 1),))
    with pytest.raises(pkg.PbtError):
        pkg.Population(bad, inp)
