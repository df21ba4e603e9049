"""Invariants of exploit / explore on whole populations (oracle side).

* a copy leaves every non-bottom member bit-unchanged and makes each bottom
  member bit-equal to its donor's pre-copy state (the multiset of winner
  states is preserved);
* explore touches only members that copied (the guard of Algorithm 1) and
  multiplies by one of the two factors;
* with a single donor per copy the number of surviving round-0 lineages never
  grows (Section 4.4, phylogenetic analysis);
* with exploit off the population is N independent runs (random search).
"""
import math

import numpy as np
import pytest

from oracle import pbt_oracle as O
from workloads import get_config, make_inputs


def _snapshot(p):
    return [{k: v.copy() for k, v in p.get_flat(m).items()} for m in range(p.N)], p.H.copy(), p.fitness.copy()


@pytest.mark.parametrize("name", ["c2_mini", "c3_mini", "c4_mini", "c5_mini"])
def test_copy_and_explore_invariants(name):
    cfg = get_config(name)
    p = O.Population(cfg, make_inputs(cfg))
    lineage = list(range(p.N))
    alive = p.N
    for rnd in range(3):
        p.step(1)
        p.eval()
        state, H, fit = _snapshot(p)
        src = p.exploit_explore()
        order = O.rank_members(fit)
        c = O.n_cut_of(p.N)
        assert sorted(b for b in range(p.N) if src[b] != b) == sorted(order[p.N - c:])
        for m in range(p.N):
            now = p.get_flat(m)
            d = int(src[m])
            for key in ("w", "opt1", "opt2", "scalars"):
                assert np.array_equal(now[key], state[d][key]), (m, key)
            assert p.fitness[m] == fit[d]
            if d == m:
                assert np.array_equal(p.H[m], H[m])
            else:
                assert d in order[:c]
                for k in range(cfg.nh):
                    lo, hi = np.float32(cfg.clamp_lo[k]), np.float32(cfg.clamp_hi[k])
                    cands = {min(max(np.float32(H[d, k] * np.float32(f)), lo), hi) for f in (0.8, 1.2)}
                    assert p.H[m, k] in cands
        lineage = [lineage[int(s)] for s in src]
        assert len(set(lineage)) <= alive
        alive = len(set(lineage))
        assert p.round == rnd + 1


def test_exploit_off_is_independent_runs():
    cfg = get_config("c3_mini").replace(flags=0)
    inp = make_inputs(cfg)
    full = O.Population(cfg, inp)
    full.run(4)
    for m in (0, 3):
        solo = O.Population(cfg, inp)
        for _ in range(4):
            solo.step(1, members=[m])
        a, b = full.get_flat(m), solo.get_flat(m)
        for key in a:
            assert np.array_equal(a[key], b[key])
    assert np.array_equal(full.H, np.asarray(inp.init_hparams, dtype=np.float32))


def test_weight_init_distribution():
    cfg = get_config("c3_mini")
    p = O.Population(cfg, make_inputs(cfg))
    for t, (s, l, fo, fi) in enumerate(p.shapes):
        a = math.sqrt(6.0 / fi)
        w = np.stack([p.W[m][t] for m in range(p.N)])
        assert w.dtype == np.float32 and np.all(np.abs(w) <= np.float32(a))
        assert abs(w.mean()) < 4 * a / math.sqrt(3 * w.size)
        assert abs(w.var() / (a * a / 3) - 1) < 0.05 or w.size < 5000
        assert not np.array_equal(w[0], w[1])
        assert all(np.all(p.b[m][t] == 0) for m in range(p.N))
    # a different seed gives different weights; the same seed the same
    q = O.Population(cfg, make_inputs(cfg), seed=1)
    r = O.Population(cfg, make_inputs(cfg))
    assert not np.array_equal(q.W[0][0], p.W[0][0]) and np.array_equal(r.W[0][0], p.W[0][0])


def test_batch_windows_stay_inside_the_pool_and_vary():
    cfg = get_config("c3_mini")
    p = O.Population(cfg, make_inputs(cfg))
    offs = set()
    for step in range(50):
        p.step_count = step
        for m in range(p.N):
            off = p._window(m, 0, 0, cfg.pool_rows, cfg.batch)
            assert off % 128 == 0 and 0 <= off and off + cfg.batch <= cfg.pool_rows
            offs.add(off)
    assert offs == {0, 128, 256, 384, 512}


def test_training_reduces_the_loss():
    cfg = get_config("c2_mini")
    p = O.Population(cfg, make_inputs(cfg))
    p.eval()
    before = p.fitness.copy()
    p.step(30)
    p.eval()
    assert np.mean(p.fitness) > np.mean(before)


@pytest.mark.parametrize("name", ["c2_mini_stagger", "c3_mini_stagger_tournament"])
def test_staggered_ready_points_touch_only_ready_members(name):
    """Algorithm 1 applies exploit / explore to the member that is ready: at a staggered ready point the record
    (weights, optimiser state, h, p) of every member that is not ready is bit-unchanged, a ready member either keeps
    its record or holds a copy of its donor's record as it was before the ready point, and the number of surviving
    initial lineages never grows (Section 4.4)."""
    cfg = get_config(name)
    inp = make_inputs(cfg)
    pop = O.Population(cfg, inp)
    lineage = list(range(cfg.n_members))
    ready_steps = {m: [] for m in range(cfg.n_members)}
    state = {}

    def on_ready(p, when):
        nonlocal lineage
        ready = O.ready_members(p.step_count, cfg.ready_interval, cfg.ready_offsets, p.N)
        if when == "pre":
            state["before"] = [p.get_flat(m) for m in range(p.N)]
            state["H"] = p.H.copy()
            state["fit"] = p.fitness.copy()
            return
        before, n_before = state["before"], len(set(lineage))
        for m in range(p.N):
            if ready[m]:
                ready_steps[m].append(p.step_count)
            d = int(p.src[m])
            if not ready[m]:
                assert d == m
            now = p.get_flat(m)
            for key in ("w", "opt1", "opt2", "scalars"):
                assert np.array_equal(now[key], before[d][key]), (m, key)
            if d == m:
                assert np.array_equal(p.H[m], state["H"][m]) and p.fitness[m] == state["fit"][m]
        lineage = [lineage[int(p.src[m])] for m in range(p.N)]
        assert len(set(lineage)) <= n_before

    pop.run(on_ready=on_ready)
    for m in range(cfg.n_members):
        want = [t for t in range(1, cfg.total_steps + 1)
                if t > cfg.ready_offsets[m] and (t - cfg.ready_offsets[m]) % cfg.ready_interval == 0]
        assert ready_steps[m] == want


def test_all_ready_mask_is_the_lockstep_ready_point():
    cfg = get_config("c2_mini")
    inp = make_inputs(cfg)
    a, b = O.Population(cfg, inp), O.Population(cfg, inp)
    for p in (a, b):
        p.step(2)
        p.eval()
    sa = a.exploit_explore()
    sb = b.exploit_explore(np.ones(cfg.n_members, dtype=bool))
    assert np.array_equal(sa, sb) and np.array_equal(a.H, b.H) and a.round == b.round
    # nobody ready: nothing moves, but the ready point is counted (the draws of the next one differ)
    H0, r0 = a.H.copy(), a.round
    s = a.exploit_explore(np.zeros(cfg.n_members, dtype=bool))
    assert np.array_equal(s, np.arange(cfg.n_members)) and np.array_equal(a.H, H0) and a.round == r0 + 1
