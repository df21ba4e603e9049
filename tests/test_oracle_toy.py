"""Pins for the oracle on the paper's toy example (Figure 2)."""
import os

import numpy as np

from oracle import pbt_oracle as O
from workloads import get_config, make_inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "toy_figure2.txt")


def _golden():
    g = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            g[k] = [float(x) for x in v]
    return g


def _pop(flags=None):
    cfg = get_config("c1")
    if flags is not None:
        cfg = cfg.replace(flags=flags)
    return O.Population(cfg, make_inputs(cfg))


def test_config_matches_the_printed_setup():
    g = _golden()
    cfg = get_config("c1")
    inp = make_inputs(cfg)
    assert list(cfg.toy_theta0) == g["theta0"]
    assert list(inp.init_hparams[0]) == g["h_worker0"] and list(inp.init_hparams[1]) == g["h_worker1"]
    assert cfg.ready_interval == int(g["exploit_every"][0])


def test_no_pbt_follows_closed_form_and_ends_near_printed_value():
    """Without exploit/explore theta_i(t) = 0.9 (1 - 2 eta h_i)^t, so worker 0 ends at
    Q = 1.2 - 0.81 (0.98^(2t) + 1), whose limit 0.39 is the caption's "~0.4"."""
    g = _golden()
    p = _pop(flags=0)
    for t in range(1, 41):
        p.step(1)
        p.eval()
        for m in range(2):
            expect = [0.9 * (1 - 0.02 * h) ** t for h in p.H[m]]
            np.testing.assert_allclose(p.theta[m], expect, rtol=1e-13)
            q = 1.2 - sum(e * e for e in expect)
            assert abs(p.fitness[m] - q) < 1e-13
        # flags == 0: a ready point must change nothing
        if t % 4 == 0:
            before = (p.theta.copy(), p.H.copy())
            p.exploit_explore()
            assert np.array_equal(before[0], p.theta) and np.array_equal(before[1], p.H)
    assert abs(p.fitness[0] - 0.22909443143354702) < 1e-12
    # run long: converges to the printed value
    p.step(2000)
    p.eval()
    assert abs(p.fitness[0] - 0.39) < 1e-6 and abs(p.fitness[0] - g["no_pbt_final_q_approx"][0]) < 0.02
    assert abs(p.fitness[1] - 0.39) < 1e-6


def test_first_ready_point_is_an_exact_tie_and_lower_index_wins():
    p = _pop()
    p.step(4)
    f = p.eval()
    assert f[0] == f[1]                      # symmetric workers: bit-identical Q
    src = p.exploit_explore()
    assert list(src) == [0, 0]               # worker 1 copies worker 0
    assert np.array_equal(p.theta[1], p.theta[0])
    assert list(p.H[0]) == [1.0, 0.0]        # the winner is untouched (guard of Algorithm 1)
    assert p.H[1][0] == 0.0 and p.H[1][1] in (0.8, 1.2)   # own h explored, not the donor's


def test_pbt_run_along_the_lineage_closed_form():
    """Replay the run with exact bookkeeping: every theta component is 0.9 times a
    product of (1 - 0.02 h) factors inherited along the copy lineage."""
    p = _pop()
    theta = [[0.9, 0.9], [0.9, 0.9]]
    h = [[1.0, 0.0], [0.0, 1.0]]
    for t in range(1, 41):
        p.step(1)
        for m in range(2):
            theta[m] = [theta[m][i] * (1 - 0.02 * h[m][i]) for i in range(2)]
        if t % 4 == 0:
            f = p.eval()
            q = [1.2 - (theta[m][0] ** 2 + theta[m][1] ** 2) for m in range(2)]
            np.testing.assert_allclose(f, q, rtol=0, atol=1e-12)
            src = p.exploit_explore()
            # the weaker worker copies the better one (ties: worker 0 is the better one)
            loser = 1 if q[0] >= q[1] - 1e-15 else 0
            if abs(q[0] - q[1]) > 1e-9:
                assert src[loser] == 1 - loser and src[1 - loser] == 1 - loser
            loser = [m for m in range(2) if src[m] != m][0]
            theta[loser] = list(theta[1 - loser])
            for i in range(2):
                ratio = p.H[loser][i] / h[loser][i] if h[loser][i] != 0 else None
                assert ratio is None or abs(ratio - 0.8) < 1e-12 or abs(ratio - 1.2) < 1e-12
                h[loser][i] = float(p.H[loser][i])
            assert list(p.H[1 - loser]) == h[1 - loser]
        np.testing.assert_allclose(p.theta, theta, rtol=1e-12)
    p.eval()
    # PBT leaves the Q ~ 0.4 plateau behind (the caption: converges towards the optimum 1.2)
    assert max(p.fitness) > 0.5
    assert p.best() == int(np.argmax(p.fitness))
    p.run(400)
    p.eval()
    assert max(p.fitness) > 1.0


def test_copying_h_too_stalls_at_the_plateau():
    """With hyperparameters copied as well both workers share one axis and stay near 0.39;
    the exploit-only ablation of Figure 2 (weights copied, no explore) still improves."""
    cfg = get_config("c1")
    stall = O.Population(cfg.replace(flags=O.COPY_WEIGHTS | O.COPY_HPARAMS | O.EXPLORE), make_inputs(cfg))
    stall.run(400)
    stall.eval()
    assert max(stall.fitness) < 0.45
    only_exploit = O.Population(cfg.replace(flags=O.COPY_WEIGHTS), make_inputs(cfg))
    only_exploit.run(400)
    only_exploit.eval()
    assert max(only_exploit.fitness) > 1.0
