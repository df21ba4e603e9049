"""Pins for the oracle's exploit / explore decisions (Section 4.1.1 (b), (a)).

Nothing here re-types the oracle's formulas: selection is checked against a
definitional enumerator ("a member is in the bottom set iff at least N - n_cut
members beat it"), the donor draw against uniformity, Philox against the
published known-answer vectors.
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import pbt_oracle as O
from oracle import philox as px

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert list(px.philox4x32_10(v[0:4], v[4:6])) == v[6:10]
        out = px.philox4x32_10_np(v[0], v[1], v[2], v[3], v[4] | (v[5] << 32))
        assert [int(o) for o in out] == v[6:10]


def test_philox_vector_matches_scalar():
    rng = np.random.default_rng(0)
    c = rng.integers(0, 2**32, size=(4, 64), dtype=np.uint64)
    seed = 0x1234567890ABCDEF
    out = px.philox4x32_10_np(c[0], c[1], c[2], c[3], seed)
    for i in range(64):
        ref = px.philox4x32_10([int(c[j, i]) for j in range(4)], (seed & 0xFFFFFFFF, seed >> 32))
        assert [int(o[i]) for o in out] == list(ref)


def _beats(fa, ia, fb, ib):
    """a ranks strictly ahead of b: larger fitness, or equal fitness and smaller index."""
    fa = -math.inf if math.isnan(fa) else fa
    fb = -math.inf if math.isnan(fb) else fb
    return fa > fb or (fa == fb and ia < ib)


def _definitional_sets(f, c):
    n = len(f)
    beaten_by = [sum(_beats(f[j], j, f[i], i) for j in range(n) if j != i) for i in range(n)]
    top = sorted((i for i in range(n) if beaten_by[i] < c), key=lambda i: beaten_by[i])
    bottom = [i for i in range(n) if beaten_by[i] >= n - c]
    return top, bottom


@pytest.mark.parametrize("num,den", [(1, 5), (2, 5)])
def test_truncation_brute_force_small_populations(num, den):
    """Every fitness vector over {0,1,2}^N (all tie patterns), N = 2..5, several rounds."""
    for n in range(2, 6):
        c = O.n_cut_of(n, num, den)
        assert c == max(1, (n * num) // den) and 2 * c <= n
        for f in itertools.product((0.0, 1.0, 2.0), repeat=n):
            top, bottom = _definitional_sets(f, c)
            assert len(top) == c and len(bottom) == c and not set(top) & set(bottom)
            for rnd in range(3):
                src = O.truncation_select(f, seed=7, rnd=rnd, num=num, den=den)
                for i in range(n):
                    if i in bottom:
                        assert src[i] in top
                        w = px.draw(7, i, rnd, px.STREAM_EXPLOIT, 0)[0]
                        # the drawn word picks the floor(w * c / 2^32)-th best member
                        assert top.index(src[i]) == int(w * c / 2**32) or \
                            top.index(src[i]) == (w * c) >> 32
                    else:
                        assert src[i] == i


def test_truncation_all_donors_reachable_and_round_dependent():
    f = [5.0, 4.0, 3.0, 2.0, 1.0, 0.0, -1.0, -2.0, -3.0, -4.0]   # N=10, n_cut=2
    seen = set()
    for rnd in range(64):
        src = O.truncation_select(f, seed=3, rnd=rnd)
        assert list(src[:8]) == list(range(8))
        assert src[8] in (0, 1) and src[9] in (0, 1)
        seen.add((int(src[8]), int(src[9])))
    assert seen == {(0, 0), (0, 1), (1, 0), (1, 1)}


def test_n_cut_values():
    # two workers: "the weaker of the two copies the better one" (Figure 2) -> n_cut(2) = 1
    assert [O.n_cut_of(n) for n in (1, 2, 3, 5, 9, 10, 16, 24, 32, 45, 80)] == \
        [0, 1, 1, 1, 1, 2, 3, 4, 6, 9, 16]


def test_ties_nan_and_signed_zero():
    assert O.rank_members([1.0, 1.0, 1.0]) == [0, 1, 2]
    assert O.rank_members([0.0, -0.0, 0.0]) == [0, 1, 2]
    assert O.rank_members([-0.0, 0.0]) == [0, 1]
    assert O.rank_members([float("nan"), -1e30, 2.0, float("nan")]) == [2, 1, 0, 3]
    assert O.rank_members([-math.inf, float("nan")]) == [0, 1]
    src = O.truncation_select([float("nan"), 3.0, 1.0, 2.0, 0.5], seed=0, rnd=0)
    assert src[0] == 1 and list(src[1:]) == [1, 2, 3, 4]


def test_donor_index_uniform():
    words = np.arange(0, 2**32, 2**16, dtype=np.uint64)   # an even grid of 2^16 words
    for c in (1, 2, 3, 4, 6, 9, 16):
        idx = np.array([O.donor_index(int(w), c) for w in words])
        assert idx.min() == 0 and idx.max() == c - 1
        counts = np.bincount(idx, minlength=c)
        assert counts.max() - counts.min() <= 1
        assert np.all(np.diff(idx) >= 0)


def test_explore_bits_are_fair_and_keyed():
    bits = np.array([O.explore_bits(11, m, r, 8) for m in range(40) for r in range(25)])
    assert bits.shape == (1000, 8)
    assert np.all(np.abs(bits.mean(axis=0) - 0.5) < 0.06)
    assert O.explore_bits(11, 3, 4, 8) != O.explore_bits(12, 3, 4, 8) or \
        O.explore_bits(11, 3, 5, 8) != O.explore_bits(11, 3, 4, 8)
    # slots 4..7 come from a second counter block, not a repeat of 0..3
    assert any(tuple(b[:4]) != tuple(b[4:]) for b in bits)


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_perturb_only_multiplies_by_the_two_factors(dtype):
    rng = np.random.default_rng(1)
    h = rng.uniform(1e-4, 1.0, size=8).astype(dtype)
    inf = math.inf
    for trial in range(32):
        bits = [int(b) for b in rng.integers(0, 2, size=8)]
        mask = [True] * 6 + [False, True]
        out = O.perturb(h, bits, mask, 0.8, 1.2, [-inf] * 8, [inf] * 8)
        assert out.dtype == h.dtype
        for k in range(8):
            if not mask[k]:
                assert out[k] == h[k]
            else:
                # the factor literal in h's precision, one correctly rounded product
                expect = dtype(dtype(1.2 if bits[k] else 0.8) * h[k])
                assert out[k] == expect
                assert abs(float(out[k]) / float(h[k]) - (1.2 if bits[k] else 0.8)) < 1e-6


def test_perturb_clamps_and_keeps_zero():
    h = np.array([0.99, 0.0, 0.5], dtype=np.float32)
    out = O.perturb(h, [1, 1, 0], [True, True, True], 0.8, 1.2,
                    [-math.inf, -math.inf, 0.45], [0.999, math.inf, math.inf])
    assert out[0] == np.float32(0.999) and out[1] == 0.0 and out[2] == np.float32(0.45)


# ---------------------------------------------------------------------------
# binary tournament (Section 4.3.1 (b))
# ---------------------------------------------------------------------------
def test_tournament_brute_force_small_populations():
    """Every fitness vector over {0,1,2}^N, N = 2..5: a member copies only a strictly better OTHER member,
    the partner is the one the drawn word designates among the other N-1, and the best never copies."""
    for n in range(2, 6):
        for f in itertools.product((0.0, 1.0, 2.0), repeat=n):
            for rnd in range(3):
                src = O.tournament_select(f, seed=5, rnd=rnd)
                for i in range(n):
                    w = px.draw(5, i, rnd, px.STREAM_EXPLOIT, 1)[0]
                    others = [j for j in range(n) if j != i]
                    partner = others[min(int(w / 2**32 * (n - 1)), n - 2)]
                    if f[partner] > f[i]:
                        assert src[i] == partner
                    else:
                        assert src[i] == i
                    if f[i] == max(f):
                        assert src[i] == i


def test_tournament_partner_is_uniform_over_the_others_and_uses_its_own_draw():
    n = 7
    f = list(range(n))                       # member 0 is the worst: it copies whoever it draws
    seen = collections_counter = {}
    for rnd in range(700):
        s0 = int(O.tournament_select(f, seed=9, rnd=rnd)[0])
        seen[s0] = seen.get(s0, 0) + 1
    assert set(seen) == set(range(1, n))
    assert max(seen.values()) - min(seen.values()) < 70          # ~117 each
    # the tournament draw is not the truncation draw (different counter block)
    a = [px.draw(9, 0, r, px.STREAM_EXPLOIT, 0)[0] for r in range(4)]
    b = [px.draw(9, 0, r, px.STREAM_EXPLOIT, 1)[0] for r in range(4)]
    assert a != b
    # NaN is the worst score; a NaN member copies any real partner, nobody copies a NaN member
    src = O.tournament_select([float("nan"), 1.0, 2.0], seed=1, rnd=0)
    assert src[0] in (1, 2) and all(src[i] != 0 for i in (1, 2))


def test_tournament_copies_read_the_state_before_the_ready_point():
    """i <- j while j <- k: i must receive j's OLD record.  Searched over rounds until a chain occurs."""
    from workloads import get_config, make_inputs
    cfg = get_config("c2_mini").replace(n_members=6, exploit="tournament")
    inp = make_inputs(cfg)
    found = False
    for rnd in range(40):
        p = O.Population(cfg, inp)
        p.round = rnd
        p.fitness[:] = np.arange(6, dtype=np.float32)
        for m in range(6):
            p.W[m][0][:] = float(m)                      # tag every member's weights with its index
        before_H = p.H.copy()
        src = p.exploit_explore()
        chain = [i for i in range(6) if src[i] != i and src[src[i]] != src[i]]
        for i in range(6):
            assert np.all(p.W[i][0] == float(src[i]))    # the donor's pre-copy weights, even when the donor copied too
            assert p.fitness[i] == float(src[i])
            if src[i] != i:
                for k in range(cfg.nh):
                    lo, hi = np.float32(cfg.clamp_lo[k]), np.float32(cfg.clamp_hi[k])
                    cands = {min(max(np.float32(before_H[src[i], k] * np.float32(fc)), lo), hi) for fc in (0.8, 1.2)}
                    assert p.H[i, k] in cands
        found = found or bool(chain)
    assert found


# ---------------------------------------------------------------------------
# per-member `ready` (Algorithm 1: `if ready(p, t, P)`): only ready members exploit
# ---------------------------------------------------------------------------
def test_ready_mask_truncation_brute_force():
    """All fitness vectors over {0,1,2}^N, N = 2..5, ALL ready masks: a member copies iff it is ready and in the
    definitional bottom set; its donor is the one its own draw picks from the definitional top set; a member that is
    not ready keeps its state even when it ranks last."""
    for n in range(2, 6):
        c = O.n_cut_of(n, 2, 5)
        for f in itertools.product((0.0, 1.0, 2.0), repeat=n):
            top, bottom = _definitional_sets(f, c)
            for mask in itertools.product((False, True), repeat=n):
                src = O.truncation_select(f, seed=11, rnd=1, num=2, den=5, ready=mask)
                for i in range(n):
                    if mask[i] and i in bottom:
                        w = px.draw(11, i, 1, px.STREAM_EXPLOIT, 0)[0]
                        assert src[i] == top[(w * c) >> 32]
                    else:
                        assert src[i] == i


def test_ready_mask_tournament_and_ttest():
    rng = np.random.default_rng(5)
    n = 9
    f = rng.standard_normal(n)
    hist = [list(rng.standard_normal(10) + (3.0 if i % 2 else 0.0)) for i in range(n)]
    full_t = O.tournament_select(f, 3, 2)
    full_w = O.ttest_select(hist, 3, 2, 0.05)
    assert (full_t != np.arange(n)).any() and (full_w != np.arange(n)).any()
    for mask in itertools.product((False, True), repeat=n):
        if sum(mask) not in (0, 1, 4, n):
            continue
        st = O.tournament_select(f, 3, 2, ready=mask)
        sw = O.ttest_select(hist, 3, 2, 0.05, ready=mask)
        for i in range(n):
            # a ready member decides exactly as it does when everybody is ready; the others keep their state
            assert st[i] == (full_t[i] if mask[i] else i)
            assert sw[i] == (full_w[i] if mask[i] else i)
    assert np.array_equal(O.tournament_select(f, 3, 2, ready=None), full_t)


def test_ready_schedule():
    """Lockstep: everybody at multiples of the interval, never at step 0.  Staggered: each member once per interval,
    first at offset + interval."""
    assert not O.ready_members(0, 4, None, 3).any()
    assert O.ready_members(8, 4, None, 3).all() and not O.ready_members(9, 4, None, 3).any()
    offs = (0, 1, 3)
    seen = {m: [] for m in range(3)}
    for t in range(0, 13):
        r = O.ready_members(t, 4, offs, 3)
        for m in range(3):
            if r[m]:
                seen[m].append(t)
    assert seen == {0: [4, 8, 12], 1: [5, 9], 2: [7, 11]}
