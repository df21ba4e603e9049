"""Pins for the oracle's t-test selection (Section 4.1.1, exploit (a)) and resample-from-prior explore
(Section 4.1.1, explore (b)).

Welch's test is pinned to things other than the oracle's own formula: the printed two-sided 5 % critical values
of Student's t (the textbook table), the closed-form t distributions with one and two degrees of freedom, an
independent library routine, and symmetry.  Selection is pinned by clear-cut cases (a plausible sign or
condition mistake fails one of them) and by uniformity of the partner draw; resampling by its rate, range,
distribution and the slots it must leave alone.
"""
import math

import numpy as np
import pytest
from scipy import stats

from oracle import pbt_oracle as O
from oracle import philox as px
from workloads import get_config, make_inputs

# two-sided 5 % critical values of Student's t, as printed in any statistics table
T_TABLE_975 = {4: 2.776, 10: 2.228, 18: 2.101}


def _pair_with_t(n, t_target):
    """Two samples of n values with equal variances whose Welch statistic is t_target; df = 2 (n - 1)."""
    base = np.arange(n, dtype=np.float64) - (n - 1) / 2.0        # mean 0, unbiased variance n (n + 1) / 12
    var = n * (n + 1) / 12.0
    shift = t_target * math.sqrt(2.0 * var / n)
    return base, base + shift


@pytest.mark.parametrize("df", sorted(T_TABLE_975))
def test_welch_p_value_crosses_five_percent_at_the_tabulated_critical_value(df):
    n = df // 2 + 1
    crit = T_TABLE_975[df]
    a, b = _pair_with_t(n, crit - 0.002)
    t, d, p = O.welch_t_test(a, b)
    assert abs(d - df) < 1e-9 and abs(t - (crit - 0.002)) < 1e-9
    assert p > 0.05
    a, b = _pair_with_t(n, crit + 0.002)
    assert O.welch_t_test(a, b)[2] < 0.05


def test_welch_closed_forms_one_and_two_degrees_of_freedom():
    # a constant sample against two values: df = n_b - 1 = 1, Student's t is the Cauchy distribution
    a, b = [1.0, 1.0, 1.0], [2.0, 5.0]
    t, df, p = O.welch_t_test(a, b)
    assert abs(df - 1.0) < 1e-12
    assert abs(t - (3.5 - 1.0) / math.sqrt(4.5 / 2)) < 1e-12
    assert abs(p - (1.0 - 2.0 / math.pi * math.atan(abs(t)))) < 1e-12
    # two pairs with equal variances: df = 2, P(|T| >= t) = 1 - t / sqrt(2 + t^2)
    a, b = [0.0, 1.0], [2.5, 3.5]
    t, df, p = O.welch_t_test(a, b)
    assert abs(df - 2.0) < 1e-12 and abs(t - 2.5 / math.sqrt(0.5)) < 1e-12
    assert abs(p - (1.0 - t / math.sqrt(2.0 + t * t))) < 1e-12


def test_welch_matches_an_independent_library_routine_and_is_antisymmetric():
    rng = np.random.default_rng(5)
    for _ in range(50):
        na, nb = int(rng.integers(2, 11)), int(rng.integers(2, 11))
        a = rng.normal(rng.normal(), abs(rng.normal()) + 0.1, na)
        b = rng.normal(rng.normal(), abs(rng.normal()) + 0.1, nb)
        t, df, p = O.welch_t_test(a, b)
        ref = stats.ttest_ind(b, a, equal_var=False)
        assert abs(t - ref.statistic) <= 1e-12 * max(1.0, abs(t))
        assert abs(df - ref.df) <= 1e-10 * df
        assert abs(p - ref.pvalue) <= 1e-10
        t2, df2, p2 = O.welch_t_test(b, a)
        assert abs(t2 + t) < 1e-12 * max(1.0, abs(t)) and abs(df2 - df) < 1e-9 * df and abs(p2 - p) < 1e-12


def test_ttest_better_clear_cases():
    rng = np.random.default_rng(1)
    low = list(rng.normal(0.0, 0.1, 10))
    high = list(rng.normal(1.0, 0.1, 10))
    noisy = list(rng.normal(0.05, 1.0, 10))
    assert O.ttest_better(low, high, 0.05)           # clearly better: copied
    assert not O.ttest_better(high, low, 0.05)       # significant but worse: never copied
    assert not O.ttest_better(low, low, 0.05)        # equal means
    assert not O.ttest_better(low, noisy, 0.05) or np.mean(noisy) > np.mean(low)
    # a higher mean that is not significant is not copied
    a = [0.0, 1.0, 2.0, 3.0]
    b = [0.5, 1.5, 2.5, 3.5]
    assert np.mean(b) > np.mean(a) and not O.ttest_better(a, b, 0.05)
    # stricter level: the same pair can pass at 5 % and fail at 0.1 %
    a, b = _pair_with_t(6, 3.0)
    assert O.ttest_better(a, b, 0.05) and not O.ttest_better(a, b, 0.001)


def test_ttest_better_degenerate_histories():
    assert not O.ttest_better([1.0], [5.0, 6.0], 0.05)            # one score: no test
    assert not O.ttest_better([1.0, 1.5], [5.0], 0.05)
    assert not O.ttest_better([], [], 0.05)
    assert O.ttest_better([1.0, 1.0], [2.0, 2.0], 0.05)           # zero variance, larger mean
    assert not O.ttest_better([2.0, 2.0], [2.0, 2.0], 0.05)
    assert O.ttest_better([float("nan"), 1.0], [0.0, 0.1], 0.05)  # a diverged member is replaced ...
    assert not O.ttest_better([0.0, 0.1], [float("nan"), 9.0], 0.05)   # ... and never copied
    assert not O.ttest_better([float("nan"), 1.0], [float("nan"), 2.0], 0.05)
    assert not O.ttest_better([0.0, 0.1], [float("inf"), 1.0], 0.05)   # non-finite statistic: no copy


def test_ttest_select_partner_is_uniform_over_the_others_and_decisions_follow_the_test():
    n = 6
    rng = np.random.default_rng(2)
    hist = [list(rng.normal(0.3 * i, 0.05, 10)) for i in range(n)]     # member i+1 is clearly better than member i
    counts = np.zeros((n, n), dtype=int)
    for rnd in range(3000):
        src = O.ttest_select(hist, 99, rnd, 0.05)
        for i in range(n):
            word = px.draw(99, i, rnd, px.STREAM_EXPLOIT, 2)[0]
            j = (word * (n - 1)) >> 32
            j += j >= i
            assert j != i
            counts[i, j] += 1
            assert src[i] == (j if j > i else i)      # better members have the larger index by construction
    for i in range(n):
        others = np.delete(counts[i], i)
        assert counts[i, i] == 0
        assert stats.chisquare(others).pvalue > 1e-4
    # the draw is the t-test's own: it differs from the tournament's draw for the same member and round
    w1 = [px.draw(99, i, 0, px.STREAM_EXPLOIT, 1)[0] for i in range(n)]
    w2 = [px.draw(99, i, 0, px.STREAM_EXPLOIT, 2)[0] for i in range(n)]
    assert w1 != w2


def test_history_keeps_the_last_ten_scores_and_travels_with_a_copy():
    cfg = get_config("c2_mini_ttest")
    pop = O.Population(cfg, make_inputs(cfg))
    seen = [[] for _ in range(pop.N)]
    for r in range(13):
        pop.step(1)
        f = pop.eval()
        for m in range(pop.N):
            seen[m].append(f[m])
    for m in range(pop.N):
        assert len(pop.history[m]) == O.HISTORY
        assert pop.history[m] == seen[m][-O.HISTORY:]
    before = [list(h) for h in pop.history]
    src = pop.exploit_explore()
    for m in range(pop.N):
        assert pop.history[m] == before[int(src[m])]


def test_ttest_population_run_copies_only_significantly_better_members():
    cfg = get_config("c2_mini_ttest")
    pop = O.Population(cfg, make_inputs(cfg))
    copies = 0
    for r in range(6):
        pop.step(cfg.ready_interval)
        pop.eval()
        hist = [list(h) for h in pop.history]
        src = pop.exploit_explore()
        for b in range(pop.N):
            d = int(src[b])
            if d != b:
                copies += 1
                assert len(hist[b]) >= 2 and len(hist[d]) >= 2
                assert np.mean(hist[d]) > np.mean(hist[b])
                assert stats.ttest_ind(hist[d], hist[b], equal_var=False).pvalue < cfg.ttest_alpha
        if r == 0:
            assert (src == np.arange(pop.N)).all()       # one score each: no test possible yet
    assert copies > 0


# ----- resample ------------------------------------------------------------------------------------------------
PRIORS = (("logu", 1e-5, 1e-2), ("u", 0.8, 0.95), ("fixed", 3.0, 3.0), ("logu", 1e-6, 1e-3))
MASK = (True, True, True, False)
NOCLAMP_LO, NOCLAMP_HI = (-math.inf,) * 4, (math.inf,) * 4


def test_resample_rate_range_and_untouched_slots():
    h0 = np.array([5e-4, 0.9, 3.0, 2e-5], dtype=np.float32)
    q = 0.3
    changed = np.zeros(4)
    vals = {0: [], 1: []}
    trials = 4000
    for t in range(trials):
        out = O.resample(h0, 11, t % 50, t // 50, MASK, PRIORS, q, NOCLAMP_LO, NOCLAMP_HI)
        assert out.dtype == np.float32
        for k in range(4):
            if out[k] != h0[k]:
                changed[k] += 1
                if k in vals:
                    vals[k].append(float(out[k]))
        assert out[2] == h0[2] and out[3] == h0[3]       # fixed prior and unmasked slot: never redrawn
    for k in (0, 1):
        rate = changed[k] / trials
        assert abs(rate - q) < 4 * math.sqrt(q * (1 - q) / trials)
        lo, hi = PRIORS[k][1], PRIORS[k][2]
        assert min(vals[k]) >= np.float32(lo) and max(vals[k]) <= np.float32(hi)
    # the redrawn values follow the prior: log-uniform for slot 0, uniform for slot 1
    assert stats.kstest(vals[0], stats.loguniform(1e-5, 1e-2).cdf).pvalue > 1e-3
    assert stats.kstest(vals[1], stats.uniform(0.8, 0.15).cdf).pvalue > 1e-3
    # the two slots decide independently
    both = sum(1 for t in range(trials)
               if (lambda o: o[0] != h0[0] and o[1] != h0[1])(
                   O.resample(h0, 11, t % 50, t // 50, MASK, PRIORS, q, NOCLAMP_LO, NOCLAMP_HI)))
    assert abs(both / trials - q * q) < 4 * math.sqrt(q * q * (1 - q * q) / trials)


def test_resample_probability_zero_and_one_and_clamp():
    h0 = np.array([5e-4, 0.9, 3.0, 2e-5], dtype=np.float64)
    for m in range(20):
        assert np.array_equal(O.resample(h0, 3, m, 0, MASK, PRIORS, 0.0, NOCLAMP_LO, NOCLAMP_HI), h0)
        out = O.resample(h0, 3, m, 0, MASK, PRIORS, 1.0, NOCLAMP_LO, NOCLAMP_HI)
        assert out[0] != h0[0] and out[1] != h0[1] and out[2] == h0[2] and out[3] == h0[3]
        # clamp bounds tighter than the prior win
        out = O.resample(h0, 3, m, 0, MASK, PRIORS, 1.0, (1e-4, 0.85, -math.inf, -math.inf), (2e-4, 0.86, math.inf, math.inf))
        assert 1e-4 <= out[0] <= 2e-4 and 0.85 <= out[1] <= 0.86
    assert O.resample_threshold(0.0) == 0 and O.resample_threshold(0.5) == 1 << 31
    assert O.resample_threshold(1.0) == 0xFFFFFFFF


def test_resample_uniform_value_is_the_affine_map_of_the_word():
    # u = (word + 1/2) / 2^32 lies strictly inside (0, 1): the ends of the prior are never produced exactly,
    # and the value is a monotone function of the word
    h0 = np.array([0.5], dtype=np.float64)
    pri = (("u", 2.0, 6.0),)
    seen = []
    for m in range(200):
        out = O.resample(h0, 8, m, 4, (True,), pri, 1.0, (-math.inf,), (math.inf,))
        w = px.draw(8, m, 4, px.STREAM_EXPLORE, 16)[1]
        seen.append((w, float(out[0])))
        assert 2.0 < out[0] < 6.0
    seen.sort()
    assert all(a[1] <= b[1] for a, b in zip(seen, seen[1:]))
    assert abs(np.mean([v for _, v in seen]) - 4.0) < 0.4


def test_resample_population_keeps_hparams_of_members_that_did_not_copy():
    cfg = get_config("c3_mini_resample")
    pop = O.Population(cfg, make_inputs(cfg))
    for r in range(3):
        pop.step(cfg.ready_interval)
        pop.eval()
        h_before = pop.H.copy()
        src = pop.exploit_explore()
        for b in range(pop.N):
            d = int(src[b])
            if d == b:
                assert np.array_equal(pop.H[b], h_before[b])
            else:
                for k in range(cfg.nh):
                    kind, lo, hi = cfg.priors[k]
                    assert pop.H[b, k] == h_before[d, k] or np.float32(lo) <= pop.H[b, k] <= np.float32(hi)
