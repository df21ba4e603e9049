"""Members at their own pace on the GPU (pbt_step_subset; Algorithm 1's per-member loop, Section 3's asynchronous
workers) against the oracle's run_schedule: which rows a member trains on follows its own step count, members that
sit out are not touched, `ready` is decided on the member's own count, decisions are bit-exact and weights within
the per-step tolerances."""
import numpy as np
import pytest

from oracle import pbt_oracle as O
from workloads import configs as C
from workloads import get_config, make_inputs

from util import TOL, assert_state_close, push_oracle_state

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    import paper_1711_09846_b200 as p
    p.load_library()
    return p


def _tol(cfg):
    t = TOL[cfg.dtype]
    return {"w": t["w"], "opt1": t["g"], "opt2": 2 * t["g"], "grad": t["g"]}


@pytest.mark.parametrize("name", ["c1", "c2_mini", "c3_mini", "c5_mid", "c4_mini", "c4_mini_wgan"])
def test_all_members_active_equals_the_lockstep_step_bit_for_bit(pkg, name):
    cfg = get_config(name)
    inp = make_inputs(cfg)
    a, b = pkg.Population(cfg, inp), pkg.Population(cfg, inp)
    a.step(3)
    b.step_subset(np.ones(cfg.n_members, dtype=bool), 3)
    for m in range(cfg.n_members):
        sa, sb = a.get_state(m), b.get_state(m)
        assert sa["step"] == sb["step"] == 3
        for key in (("w",) if cfg.model == C.TOY else ("w", "opt1", "opt2", "scalars")):
            assert np.array_equal(sa[key], sb[key]), (name, m, key)
    assert np.array_equal(a.last_loss(), b.last_loss())
    a.close()
    b.close()


@pytest.mark.parametrize("name", ["c2_mini", "c3_mini", "c5_mid", "c4_mini_wgan", "c3_mini_stagger_tournament"])
def test_schedule_with_members_sitting_out_matches_the_oracle(pkg, name):
    """About a third of the members skip each tick (runs of one, two and more consecutive active members occur)."""
    cfg = get_config(name)
    if cfg.n_members < 6:
        cfg = cfg.replace(n_members=6)
    cfg = cfg.replace(ready_interval=2)
    inp = make_inputs(cfg)
    n = cfg.n_members
    gpu, cpu = pkg.Population(cfg, inp, keep_grad=True), O.Population(cfg, inp)
    tol = _tol(cfg)
    ftol = 1e-4 if cfg.dtype == C.FP32 else 2e-2
    keys = ("w", "opt1", "opt2", "grad") if cfg.optimizer == C.OPT_ADAM else ("w", "opt1", "grad")
    rng = np.random.default_rng(7)
    ticks = 7
    sched = rng.random((ticks, n)) < 0.67
    sched[0] = [True, False, True, True, False, True][:n] + [True] * (n - 6)     # runs of 1, 2, 1
    ready_points = 0
    for tick in range(ticks):
        mask = sched[tick]
        if not mask.any():
            continue
        before = [gpu.get_state(m) for m in range(n)]
        gpu.step_subset(mask, 1)
        cpu.step(1, members=[m for m in range(n) if mask[m]])
        for m in range(n):
            g = gpu.get_state(m)
            assert g["step"] == cpu.t[m], (tick, m)
            if mask[m]:
                assert_state_close(cfg, g, cpu.get_flat(m), keys, tol, what=f"{name}_own_pace tick {tick} member {m}")
                assert np.array_equal(g["scalars"], cpu.get_flat(m)["scalars"])
            else:
                for key in ("w", "opt1", "opt2", "scalars"):
                    assert np.array_equal(g[key], before[m][key]), (tick, m, key)      # sat out: untouched
        ready = O.ready_members_own(cpu.t, cfg.ready_interval, cfg.ready_offsets) & mask
        if ready.any():
            ready_points += 1
            gpu.eval()
            cpu.eval()
            np.testing.assert_allclose(gpu.fitness(), cpu.fitness, rtol=ftol, atol=2e-5)
            gpu.set_fitness(cpu.fitness.astype(np.float64))
            rmask = None if ready.all() else ready
            gpu.exploit_explore(rmask)
            src = cpu.exploit_explore(rmask)
            assert np.array_equal(gpu.copy_map(), src)
            assert np.array_equal(gpu.hparams(), cpu.H.astype(np.float64))
            for m in range(n):
                assert gpu.get_state(m)["step"] == cpu.t[m]          # a copy does not move a member's own count
        push_oracle_state(gpu, cpu)
    assert ready_points >= 2
    assert len(set(int(x) for x in cpu.t)) > 1                        # the members really are at different steps
    gpu.close()


def test_subset_step_rejects_a_pending_supplied_batch(pkg):
    import torch
    cfg = get_config("c2_mini")
    inp = make_inputs(cfg)
    gpu = pkg.Population(cfg, inp)
    x = torch.zeros((cfg.n_members, cfg.batch, cfg.widths[0][0]), device="cuda")
    y = torch.zeros((cfg.n_members, cfg.batch, 1), device="cuda")
    gpu.set_batch(x, y)
    with pytest.raises(pkg.PbtError) as e:
        gpu.step_subset(np.ones(cfg.n_members, dtype=bool), 1)
    assert e.value.code == 6
    gpu.step(1)
    gpu.close()
