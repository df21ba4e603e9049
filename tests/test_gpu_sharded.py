"""A population sharded over several library handles against the same population in one handle, bit for bit.

One GPU is enough: the shards are separate handles with separate workspaces that exchange records only through the
copy plan (device-to-device copies here; send / receive between processes is covered by the gloo test).  Everything
drawn per member is keyed by the member's index in the whole population, so weights, optimiser state,
hyperparameters, fitness and copy maps of the sharded run must equal the unsharded run exactly, ready point after
ready point, for truncation selection and for the binary tournament (chained copies across shards)."""
import numpy as np
import pytest

from workloads import configs as C
from workloads import get_config, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    import paper_1711_09846_b200 as p
    p.load_library()
    return p


@pytest.mark.parametrize("name,n,world,rule", [("c2_mini", 10, 2, "truncation"), ("c3_mini", 11, 3, "truncation"),
                                               ("c3_mini", 12, 2, "tournament"), ("c5_mid", 6, 2, "truncation"),
                                               ("c1", 9, 3, "tournament"), ("c4_mini_wgan", 7, 2, "truncation"),
                                               ("c2_mini", 9, 2, "ttest"), ("c3_mini", 10, 3, "ttest")])
def test_sharded_run_equals_the_unsharded_run_bit_for_bit(pkg, name, n, world, rule):
    from paper_1711_09846_b200 import sharding as S
    cfg = get_config(name).replace(n_members=n, exploit=rule, ready_interval=2, trunc_num=2, trunc_den=5)
    if cfg.model == C.TOY:
        cfg = cfg.replace(flags=C.COPY_WEIGHTS | C.COPY_HPARAMS | C.EXPLORE)
    inp = make_inputs(cfg)
    if cfg.model == C.TOY:
        h0 = np.random.default_rng(2).random((n, cfg.nh)) + 0.5        # members that differ
        inp = type(inp)(**{**inp.__dict__, "init_hparams": h0})
    whole = pkg.Population(cfg, inp)
    shards = [S.ShardedPopulation(pkg, cfg, inp, r, world, transport=object()) for r in range(world)]
    crossed = 0
    for rnd in range(5 if rule == "ttest" else 3):
        whole.step(cfg.ready_interval)
        whole.eval()
        for s in shards:
            s.step(cfg.ready_interval)
            s.eval()
        f_sharded = np.concatenate([s.local.fitness() for s in shards])
        assert np.array_equal(whole.fitness(), f_sharded, equal_nan=True), (name, rnd)
        whole.exploit_explore()
        src = S.ready_point_in_process(shards)
        assert np.array_equal(whole.copy_map(), src), (name, rnd)
        crossed += shards[0].last_plan.crossing()
        assert np.array_equal(whole.hparams(), np.concatenate([s.local.hparams() for s in shards], axis=0))
        assert np.array_equal(whole.fitness(), np.concatenate([s.local.fitness() for s in shards]), equal_nan=True)
        if rule == "ttest":
            hw, cw = whole.history()
            parts = [s.local.history() for s in shards]
            assert np.array_equal(cw, np.concatenate([p[1] for p in parts]))
            assert np.array_equal(hw, np.concatenate([p[0] for p in parts], axis=0))
        for m in range(n):
            r = S.owner_of(m, world, n)
            a, b = whole.get_state(m), shards[r].local.get_state(m - shards[r].first)
            assert a["step"] == b["step"] and a["round"] == b["round"]
            for key in (("w",) if cfg.model == C.TOY else ("w", "opt1", "opt2", "scalars")):
                assert np.array_equal(a[key], b[key]), (name, rnd, m, key)
    assert crossed > 0, "no record crossed shards: the test did not exercise the exchange"
    whole.close()
    for s in shards:
        s.close()


def test_a_shard_refuses_the_unsharded_ready_point_and_t_test_selection_without_histories(pkg):
    from paper_1711_09846_b200 import sharding as S
    cfg = get_config("c2_mini").replace(n_members=6)
    inp = make_inputs(cfg)
    s = S.ShardedPopulation(pkg, cfg, inp, 0, 2, transport=object())
    with pytest.raises(pkg.PbtError) as e:
        s.local.exploit_explore()
    assert e.value.code == 6
    s.close()
    t = S.ShardedPopulation(pkg, cfg.replace(exploit="ttest"), inp, 1, 2, transport=object())
    with pytest.raises(pkg.PbtError) as e:                 # t-test selection wants the whole population's histories first
        t.decide(np.zeros(6), np.asarray(inp.init_hparams))
    assert e.value.code == 6
    t.close()
