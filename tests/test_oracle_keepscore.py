"""Pins for the oracle's attention-aware LRFU keep-score (Section 5.1, Algorithm 1 steps 2-5)."""
import numpy as np

from oracle import actkv_oracle as O

from conftest import read_golden


def _plain_hits(score, p):
    """The plain real-valued rule, with no quantisation anywhere: the float32 scores as the exact rationals
    they are, p as the exact decimal, the shortest prefix of the entries ordered by (score descending, index
    ascending) whose sum reaches p times the total; the crossing entry is in.  Also returns how far (as a
    fraction of the total) the sums just before and just after the last hit are from the mark."""
    from fractions import Fraction
    vals = [max(Fraction(float(x)), Fraction(0)) for x in score]
    total = sum(vals)
    mark = Fraction(str(p)) * total
    order = sorted(range(len(score)), key=lambda i: (-vals[i], i))
    hit, acc, margin = [], Fraction(0), None
    for i in order:
        if acc >= mark or vals[i] == 0:
            break
        hit.append(i)
        margin = min(mark - acc, acc + vals[i] - mark) / total if total else None
        acc += vals[i]
    return sorted(hit), margin


def test_paper_constants_present():
    g = read_golden("monitor_constants.txt")
    assert g["lambda"][0] == 0.5 and g["top_p"][0] == 0.9


def test_hit_mask_against_brute_force_with_ties():
    rng = np.random.default_rng(0)
    for seed in range(6):
        s = (rng.integers(0, 9, 61).astype(np.float32) / 64.0)            # many exact ties, some zeros
        for p in (0.0, 0.5, 0.9, 0.99, 1.0):
            # multiples of 1/64 have integer masses, so the integer rule and the real-valued rule coincide exactly,
            # also when a prefix lands on the mark
            assert np.nonzero(O.hit_mask_unit(s, p))[0].tolist() == _plain_hits(s, p)[0]


def test_integer_masses_give_the_real_valued_top_p_set():
    """The oracle counts mass in integers of 2^-32 so that the set does not depend on a summation order.  Against
    the plain rule on the real values of the float32 scores: the same set whenever the mark is further from a
    prefix sum than the truncation can move it (L x 2^-32 of mass), which random inputs always are."""
    rng = np.random.default_rng(5)
    checked = 0
    for seed in range(8):
        L = int(rng.integers(50, 400))
        s = (rng.random(L) ** 6).astype(np.float32) * np.float32(0.05)       # skewed, pooled-probability sized
        for p in (0.3, 0.9, 0.97):
            want, margin = _plain_hits(s, p)
            total = float(np.sum(s.astype(np.float64)))
            if margin is not None and float(margin) * total > 4 * L * 2.0 ** -32:
                assert np.nonzero(O.hit_mask_unit(s, p))[0].tolist() == want
                checked += 1
    assert checked >= 20


def test_hit_mask_is_a_prefix_that_just_reaches_the_mark():
    rng = np.random.default_rng(1)
    s = rng.random(500).astype(np.float32) ** 4                            # skewed like attention
    hit = O.hit_mask_unit(s, 0.9)
    order = np.lexsort((np.arange(500), -s.astype(np.float64)))
    n = int(hit.sum())
    assert hit[order[:n]].all() and not hit[order[n:]].any()               # a prefix of the descending order
    mass = np.floor(s.astype(np.float64) * 2**32)
    assert mass[order[:n]].sum() >= 0.9 * mass.sum() > mass[order[:n - 1]].sum()   # minimal
    assert 0 < n < 500


def test_hit_mask_extremes():
    s = np.array([0.5, 0.25, 0.125, 0.125, 0.0], dtype=np.float32)
    assert O.hit_mask_unit(s, 1.0).tolist() == [True, True, True, True, False]   # zero mass is never needed
    assert O.hit_mask_unit(s, 0.5).tolist() == [True, False, False, False, False]
    assert O.hit_mask_unit(s, 0.5001).tolist() == [True, True, False, False, False]
    assert O.hit_mask_unit(s, 0.76).tolist() == [True, True, True, False, False]  # tie: the lower index is hit
    assert not O.hit_mask_unit(s, 0.0).any()
    assert not O.hit_mask_unit(np.zeros(7, dtype=np.float32), 0.9).any()


def test_keep_score_recurrence_closed_forms():
    lam = np.float32(0.5)
    s = np.float32(0.125)
    ks = np.zeros(1, dtype=np.float32)
    for t in range(1, 12):                                                  # hit every round: geometric series
        ks = O.keep_score_update(ks, np.array([s]), np.array([True]), lam)
        assert abs(float(ks[0]) - float(s) * (1 - 0.5**t) / 0.5) < 1e-7
    peak = ks.copy()
    for t in range(1, 6):                                                   # then never hit: pure decay
        ks = O.keep_score_update(ks, np.array([s]), np.array([False]), lam)
        assert ks[0] == np.float32(peak[0] * 0.5**t)
    # lambda = 0: recency only; lambda = 1: frequency only
    assert O.keep_score_update(np.array([3.0], np.float32), np.array([s]), np.array([True]), 0.0)[0] == s
    assert O.keep_score_update(np.array([3.0], np.float32), np.array([s]), np.array([True]), 1.0)[0] == np.float32(3.125)
    assert O.keep_score_update(np.array([3.0], np.float32), np.array([s]), np.array([False]), 1.0)[0] == np.float32(3.0)


def test_intermittent_entry_outlives_a_stale_continuous_one():
    """The paper's motivation: a strongly but intermittently attended entry must survive a pause that a
    weakly, continuously attended entry does not compensate."""
    lam = 0.5
    ks = np.zeros(2, dtype=np.float32)
    strong, weak = np.float32(0.4), np.float32(0.05)
    pattern = [(True, True), (False, True), (False, True), (True, True)]
    for hit_strong, hit_weak in pattern:
        ks = O.keep_score_update(ks, np.array([strong, weak]), np.array([hit_strong, hit_weak]), lam)
    assert ks[0] > ks[1]
    kept = O.select_unit(O.rank_keys(ks, 0), 1)
    assert kept.tolist() == [0]


def test_protected_prefix_is_always_retained():
    ks = np.array([0.0, 0.0, 0.9, 0.8, 0.7, 0.6], dtype=np.float32)
    keys = O.rank_keys(ks, 2)
    assert np.isinf(keys[:2]).all() and np.array_equal(keys[2:], ks[2:])
    assert O.select_unit(keys, 3).tolist() == [0, 1, 2]
    assert O.select_unit(O.rank_keys(ks, 0), 3).tolist() == [2, 3, 4]
