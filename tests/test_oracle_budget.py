"""Pins for the oracle's confidence monitor and budget update (CPU only)."""
import math

import numpy as np

from oracle import actkv_oracle as O

from conftest import read_golden


def _params():
    g = read_golden("monitor_constants.txt")
    return O.BudgetParams(k=g["k"][0], w=g["w"][0], s=g["s"][0], b_percent=float(g["b"][0]),
                          scale_up=g["scale_up"][0], B_upper=g["budget_upper"][0]), g


def test_uniform_distribution_confidence_is_log_vocab():
    """P uniform over V tokens: every log P = -log V, so T = log V for any k."""
    V = 151936
    T = O.token_confidence(np.full((2, V), 0.37, dtype=np.float32), 20)
    assert np.abs(T - math.log(V)).max() < 1e-12
    assert abs(math.log(V) - 11.931214658529285) < 1e-12


def test_two_level_distribution_closed_form():
    """k logits at a, the other V-k at 0: P(top) = e^a / (k e^a + V - k), T = -log P(top)."""
    V, k, a = 1000, 20, 3.0
    z = np.zeros((1, V))
    z[0, 5:5 + k] = a
    T = O.token_confidence(z, k)
    assert abs(T[0] - (math.log(k * math.exp(a) + V - k) - a)) < 1e-12
    # top-k smaller than the plateau: k' = 7 of the 20 high logits still all equal a
    assert abs(O.token_confidence(z, 7)[0] - T[0]) < 1e-12


def test_token_confidence_is_minus_mean_log_prob_of_topk():
    rng = np.random.default_rng(0)
    z = rng.standard_normal((3, 500)) * 2.0
    p = np.exp(z) / np.exp(z).sum(axis=1, keepdims=True)
    ref = [-np.mean(np.log(np.sort(p[i])[-20:])) for i in range(3)]
    assert np.abs(O.token_confidence(z, 20) - ref).max() < 1e-12


def test_window_min_pooling_and_bottom_percent():
    TL = np.arange(100, dtype=np.float32)[::-1].copy()           # strictly decreasing 99..0
    Rp_expected = [99 - (m * 8 + 63) for m in range((100 - 64) // 8 + 1)]   # min of each window = its last
    R = O.trace_confidence(TL, 64, 8, 100.0)
    assert R.tolist() == Rp_expected and len(R) == 5
    # bottom 10% of 5 values: nearest rank ceil(0.5) = 1 -> only the smallest
    assert O.trace_confidence(TL, 64, 8, 10.0).tolist() == [min(Rp_expected)]
    # history shorter than the window: empty
    assert len(O.trace_confidence(TL[:63], 64, 8, 10.0)) == 0
    # ties are all kept (values <= the percentile value)
    TL2 = np.ones(200, dtype=np.float32)
    assert len(O.trace_confidence(TL2, 64, 8, 10.0)) == (200 - 64) // 8 + 1


def test_fit_slope_closed_forms_and_library():
    assert O.fit_slope(np.array([3.0, 1.0])) == -2.0              # two points: y1 - y0
    assert O.fit_slope(np.array([5.0])) == 0.0 and O.fit_slope(np.zeros(0)) == 0.0
    y = np.float32(11.931214) * np.ones(37, dtype=np.float32)
    assert O.fit_slope(y) == 0.0                                  # constant: exactly zero
    rng = np.random.default_rng(1)
    y = rng.standard_normal(50)
    ref = np.polyfit(np.arange(50), y, 1)[0]
    assert abs(O.fit_slope(y) - ref) < 1e-12
    assert abs(O.fit_slope(2.5 * np.arange(10) + 1.0) - 2.5) < 1e-12


def test_budget_chain_from_paper_constants():
    p, g = _params()
    B = g["budget_start"][0]
    chain = [B]
    while chain[-1] < p.B_upper:
        chain.append(O.budget_update(chain[-1], -1.0, p))
    assert chain == [512, 896, 1568, 2744, 4802, 8403, 14705, 25733, 30000]
    assert O.budget_update(4802, 0.0, p) == 4802 and O.budget_update(4802, 0.3, p) == 4802
    assert O.budget_update(30000, -1.0, p) == 30000


def test_budget_clamp_integer_rule():
    p = O.BudgetParams(clamp_lo_ppm=150000, clamp_hi_ppm=400000)
    assert O.budget_update(100, 0.0, p, L=35000) == 5250          # raised to ceil(0.15 L)
    assert O.budget_update(20000, 0.0, p, L=35000) == 14000       # lowered to floor(0.40 L)
    assert O.budget_update(7000, -1.0, p, L=35000) == 12250       # 7000*1.75 inside the clamp
    p2 = O.BudgetParams(clamp_lo_ppm=260000, clamp_hi_ppm=260000)
    assert O.budget_update(5, 0.0, p2, L=35000) == 9100


def test_budget_end_to_end_decreasing_and_constant_confidence():
    """Linearly decreasing confidence -> negative slope -> budget scaled; constant -> kept."""
    p, _ = _params()
    V, T = 64, 200
    # confidence decreases when logits flatten: two-level rows with shrinking gap a_i
    gaps = np.linspace(6.0, 1.0, T)
    z = np.zeros((2 * T, V))
    for i, a in enumerate(gaps):
        z[i, :20] = a
    z[T:, :20] = 3.0                                              # request 1: constant rows
    tok = np.array([0, T, 2 * T])
    hist = np.zeros((2, 512), dtype=np.float32)
    h, hl, out, slopes, Tc = O.budget(z, tok, hist, [0, 0], [512, 512], p)
    assert hl.tolist() == [T, T]
    assert np.all(np.diff(Tc[:T]) > 0) or np.all(np.diff(Tc[:T]) < 0)
    # T = log(20 e^a + 44) - a decreases... check direction explicitly
    expected_sign = np.sign(Tc[T - 1] - Tc[0])
    assert np.sign(slopes[0]) == expected_sign and slopes[1] == 0.0
    assert out[1] == 512
    assert out[0] == (896 if expected_sign < 0 else 512)
    # reversed order gives the opposite decision
    z2 = z.copy()
    z2[:T] = z[:T][::-1]
    _, _, out2, slopes2, _ = O.budget(z2, tok, hist, [0, 0], [512, 512], p)
    assert np.sign(slopes2[0]) == -expected_sign
    assert {int(out[0]), int(out2[0])} == {512, 896}


def test_budget_history_persists_and_caps():
    p, _ = _params()
    rng = np.random.default_rng(2)
    z = rng.standard_normal((40, 100))
    tok = np.array([0, 40])
    hist = np.zeros((1, 64), dtype=np.float32)
    h1, hl1, _, s1, _ = O.budget(z, tok, hist, [0], [100], p)
    assert hl1.tolist() == [40] and s1[0] == 0.0                  # 40 < w: no trend yet
    h2, hl2, _, _, T2 = O.budget(z, tok, h1, hl1, [100], p)
    assert hl2.tolist() == [64]                                   # capped at the history size
    assert np.array_equal(h2[0, 40:64], T2[:24].astype(np.float32))
