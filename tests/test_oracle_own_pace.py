"""Pins for members that advance at their own pace (Algorithm 1's per-member loop; Section 3: asynchronous workers).

What is fixed without any implementation to compare with:
  * between ready points a member's trajectory depends on its own record and its own step count only, so under ANY
    schedule of who steps when, a member that has taken c steps equals the same member run alone for c steps
    (enumerated over every schedule of a small population);
  * the all-ones schedule is the lockstep run;
  * `ready` looks at the member's own count: its definition, enumerated;
  * a ready point under a schedule applies to the members that stepped and are ready by their own count, and the
    records of the others do not change.
"""
import itertools

import numpy as np

from oracle import pbt_oracle as O
from workloads import configs as C
from workloads import get_config, make_inputs


def _flat_equal(a, b, m):
    fa, fb = a.get_flat(m), b.get_flat(m)
    return all(np.array_equal(fa[k], fb[k]) for k in fa)


def test_every_schedule_equals_each_member_run_alone():
    """N = 2, T = 3 ticks: all 64 schedules.  Exploit off, so members never interact."""
    for name in ("c2_mini", "c3_mini", "c1"):
        cfg = get_config(name).replace(n_members=2, flags=0, ready_interval=10 ** 6)
        inp = make_inputs(cfg)
        alone = {}
        for m in range(2):
            for c in range(4):
                p = O.Population(cfg, inp, only_members=[m])
                p.step(c, members=[m])
                alone[(m, c)] = p
        for bits in itertools.product([0, 1], repeat=6):
            sched = np.array(bits, dtype=bool).reshape(3, 2)
            pop = O.Population(cfg, inp)
            pop.run_schedule(sched)
            for m in range(2):
                c = int(sched[:, m].sum())
                assert pop.t[m] == c
                assert _flat_equal(pop, alone[(m, c)], m), (name, bits, m)


def test_member_held_back_and_resumed_continues_where_it_stopped():
    """A member that sits out k ticks and then resumes is, step for step, the member that never paused: the rows it
    trains on are keyed by its own count, not by the population's clock."""
    cfg = get_config("c3_mini").replace(flags=0, ready_interval=10 ** 6)
    inp = make_inputs(cfg)
    ref = O.Population(cfg, inp)
    ref.step(5)
    for k in (1, 3):
        pop = O.Population(cfg, inp)
        sched = np.ones((5 + k, cfg.n_members), dtype=bool)
        sched[2:2 + k, 1] = False            # member 1 pauses after two steps
        sched[5:, 0] = False                 # the others are done after five ticks
        sched[5:, 2:] = False
        pop.run_schedule(sched)
        assert list(pop.t) == [5] * cfg.n_members
        for m in range(cfg.n_members):
            assert _flat_equal(pop, ref, m), (k, m)


def test_all_ones_schedule_is_the_lockstep_run():
    for name in ("c1", "c2_mini", "c3_mini_stagger_tournament"):
        cfg = get_config(name)
        inp = make_inputs(cfg)
        a, b = O.Population(cfg, inp), O.Population(cfg, inp)
        a.run(cfg.total_steps)
        b.run_schedule(np.ones((cfg.total_steps, cfg.n_members), dtype=bool))
        assert a.round == b.round and np.array_equal(a.H, b.H) and np.array_equal(a.fitness, b.fitness)
        assert np.array_equal(a.src, b.src)
        for m in range(cfg.n_members):
            assert _flat_equal(a, b, m), (name, m)


def test_own_clock_ready_definition():
    iv = 3
    for t in itertools.product(range(8), repeat=3):
        for offs in ((), (0, 1, 2)):
            got = O.ready_members_own(t, iv, offs)
            for m in range(3):
                d = t[m] - (offs[m] if offs else 0)
                assert bool(got[m]) == (d > 0 and d % iv == 0)
    # equal counts: the lockstep rule
    for step in range(10):
        assert np.array_equal(O.ready_members_own([step] * 4, iv, ()), O.ready_members(step, iv, (), 4))


def test_ready_point_under_a_schedule_touches_only_members_ready_by_their_own_count():
    cfg = get_config("c2_mini").replace(n_members=6, ready_interval=2, trunc_num=2, trunc_den=5)
    inp = make_inputs(cfg)
    pop = O.Population(cfg, inp)
    rng = np.random.default_rng(0)
    sched = rng.random((9, 6)) < 0.6
    seen = []

    def on_ready(p, when):
        if when == "pre":
            seen.append((p.t.copy(), [p.get_flat(m) for m in range(6)], p.H.copy()))
        else:
            t, before, h = seen[-1]
            ready_now = O.ready_members_own(t, 2, ())
            for m in range(6):
                if p.src[m] != m:
                    assert ready_now[m]                        # only members ready by their own count copy
                else:
                    assert all(np.array_equal(before[m][k], p.get_flat(m)[k]) for k in before[m])
                    assert np.array_equal(h[m], p.H[m])
            assert np.array_equal(p.t, t)                      # a copy does not move anybody's step count
    pop.run_schedule(sched, on_ready)
    assert list(pop.t) == [int(c) for c in sched.sum(axis=0)]
    assert seen, "the schedule produced no ready point"
