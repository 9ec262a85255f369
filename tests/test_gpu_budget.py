"""GPU parity of actkv_budget against the oracle's confidence monitor."""
import math

import numpy as np
import pytest
import torch

from oracle import actkv_oracle as O
from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
T_ATOL = 2e-5          # float32 logsumexp / mean against float64, values of order 10


def _run(logits, tok_indptr, hist, hist_len, budget_in, params, seq_len=None):
    R = hist.shape[0]
    cap = hist.shape[1]
    n_rows = 0 if logits is None else logits.shape[0]
    vocab = 0 if logits is None else logits.shape[1]
    ws = torch.empty(B.actkv_budget_workspace_bytes(n_rows, R, cap) + 256, dtype=torch.uint8, device=DEV)
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    out = torch.zeros(R, dtype=torch.int32, device=DEV)
    slopes = torch.zeros(R, dtype=torch.float64, device=DEV)
    B.actkv_budget(logits, tok_indptr, n_rows, vocab, hist, hist_len, cap, params, seq_len, budget_in, out, slopes,
                   R, ws, status)
    torch.cuda.synchronize()
    return out.cpu().numpy(), slopes.cpu().numpy(), status.cpu().tolist()


def _oracle_params(p: B.BudgetParams) -> O.BudgetParams:
    return O.BudgetParams(p.k, p.w, p.s, p.b_percent, p.scale_up, p.B_upper, p.clamp_lo_ppm, p.clamp_hi_ppm)


def _compare(logits, tok, hist0, len0, budget_in, params, seq_len=None):
    R = hist0.shape[0]
    hist = hist0.clone().to(DEV)
    hist_len = len0.clone().to(DEV)
    got_B, got_a, st = _run(logits, tok, hist, hist_len, budget_in.to(DEV), params,
                            None if seq_len is None else seq_len.to(DEV))
    assert st[0] == 0
    op = _oracle_params(params)
    tok_np = tok.cpu().numpy()
    oh, ol, oB, oa, oT = O.budget(logits.cpu().numpy(), tok_np, hist0.numpy(), len0.numpy(), budget_in.numpy(), op,
                                  None if seq_len is None else seq_len.numpy())
    gh = hist.cpu().numpy()
    gl = hist_len.cpu().numpy()
    assert np.array_equal(gl, ol)
    for r in range(R):
        if gl[r]:
            assert np.abs(gh[r, :gl[r]].astype(np.float64) - oh[r, :ol[r]]).max() <= T_ATOL
    # the decision part on the GPU's own stored history must match the oracle exactly
    borderline = 0
    for r in range(R):
        Rr = O.trace_confidence(gh[r, :gl[r]], op.w, op.s, op.b_percent)
        a = O.fit_slope(Rr)
        assert abs(got_a[r] - a) <= 1e-12 * max(1.0, abs(a))
        want = O.budget_update(int(budget_in[r]), a, op, None if seq_len is None else int(seq_len[r]))
        assert got_B[r] == want
        if got_B[r] != oB[r]:
            borderline += 1
            assert abs(oa[r]) < 1e-4           # full-pipeline disagreement only when the slope is ~0
    return got_B, got_a, borderline


def test_uniform_rows_give_log_vocab_and_zero_slope():
    V, T, R = 151936, 80, 2
    logits = torch.full((R * T, V), 0.37, dtype=torch.float32, device=DEV)
    tok = torch.arange(0, (R + 1) * T, T, dtype=torch.int32, device=DEV)
    hist = torch.zeros((R, 256), dtype=torch.float32)
    p = B.BudgetParams.paper_defaults()
    hist_d = hist.clone().to(DEV)
    len_d = torch.zeros(R, dtype=torch.int32, device=DEV)
    got_B, got_a, st = _run(logits, tok, hist_d, len_d, torch.tensor([512, 896], dtype=torch.int32, device=DEV), p)
    assert st[0] == 0
    h = hist_d.cpu().numpy()
    assert np.abs(h[:, :T] - math.log(V)).max() < T_ATOL
    assert (got_a == 0.0).all() and got_B.tolist() == [512, 896]


@pytest.mark.parametrize("vocab,R,T", [(151936, 3, 96), (1000, 6, 400), (37, 6, 400)])
def test_against_oracle_gaussian_logits(vocab, R, T):
    logits, tok = synth.confidence_logits(R, T, vocab, seed=vocab, device=DEV)
    hist0 = torch.zeros((R, 512), dtype=torch.float32)
    len0 = torch.zeros(R, dtype=torch.int32)
    budget_in = torch.tensor([512, 896, 1568, 20000, 29000, 100][:R], dtype=torch.int32)
    p = B.BudgetParams.paper_defaults()
    got_B, got_a, _ = _compare(logits, tok, hist0, len0, budget_in, p)
    if vocab == 1000:
        assert (got_a < 0).any() and (got_a == 0).any()      # both outcomes occur in this draw
    for r in range(R):
        if got_a[r] < 0:
            assert got_B[r] == min(int(budget_in[r] * 1.75), 30000)


def test_sorted_rows_overflow_the_candidate_list_and_are_redone():
    """Ascending rows make every later logit a top-k candidate: the single-sweep kernel gives them up
    and the three-sweep kernel redoes them; descending and shuffled rows stay on the fast path."""
    R, T, V = 3, 70, 151936
    g = torch.Generator(device=DEV)
    g.manual_seed(77)
    base = torch.randn((R * T, V), generator=g, device=DEV) * 2.0
    logits = base.clone()
    logits[:T] = torch.sort(base[:T], dim=1).values                       # ascending
    logits[T:2 * T] = torch.sort(base[T:2 * T], dim=1, descending=True).values
    tok = torch.arange(0, (R + 1) * T, T, dtype=torch.int32, device=DEV)
    hist0 = torch.zeros((R, 128), dtype=torch.float32)
    len0 = torch.zeros(R, dtype=torch.int32)
    _compare(logits, tok, hist0, len0, torch.tensor([512, 512, 512], dtype=torch.int32),
             B.BudgetParams.paper_defaults())


def test_rows_the_single_sweep_cannot_take_are_redone():
    """The single-sweep kernel takes its exp reference from the head of the row and its threshold from 64
    chunk maxima: rows whose later logits dwarf the head (the sum would overflow) and calls with k > 64 go
    to the three-sweep kernel."""
    R, T, V = 2, 70, 151936
    g = torch.Generator(device=DEV)
    g.manual_seed(78)
    logits = torch.randn((R * T, V), generator=g, device=DEV)
    logits[:T, 100000:100040] += 95.0                                      # exp(95 - head maximum) is beyond float32
    tok = torch.arange(0, (R + 1) * T, T, dtype=torch.int32, device=DEV)
    hist0 = torch.zeros((R, 128), dtype=torch.float32)
    len0 = torch.zeros(R, dtype=torch.int32)
    _compare(logits, tok, hist0, len0, torch.tensor([512, 512], dtype=torch.int32), B.BudgetParams.paper_defaults())
    p = B.BudgetParams.paper_defaults()
    p.k = 100
    _compare(logits[T:], tok[:2].clone(), hist0[:1], len0[:1], torch.tensor([512], dtype=torch.int32), p)


def test_history_accumulates_across_calls_and_clamp():
    R, T, V = 4, 40, 2048
    p = B.BudgetParams.paper_defaults(clamp_lo_ppm=150000, clamp_hi_ppm=400000)
    seq_len = torch.tensor([35000, 8192, 65536, 1000], dtype=torch.int32)
    budget_in = torch.tensor([7000, 100, 30000, 500], dtype=torch.int32)
    hist = torch.zeros((R, 128), dtype=torch.float32)
    lens = torch.zeros(R, dtype=torch.int32)
    op = _oracle_params(p)
    hist_d, len_d = hist.clone().to(DEV), lens.clone().to(DEV)
    oh, ol = hist.numpy(), lens.numpy()
    for call in range(3):
        logits, tok = synth.confidence_logits(R, T, V, seed=100 + call, device=DEV)
        got_B, got_a, st = _run(logits, tok, hist_d, len_d, budget_in.to(DEV), p, seq_len.to(DEV))
        oh, ol, oB, oa, _ = O.budget(logits.cpu().numpy(), tok.cpu().numpy(), oh, ol, budget_in.numpy(), op,
                                     seq_len.numpy())
        assert st[0] == 0
        assert np.array_equal(len_d.cpu().numpy(), ol)
        assert np.abs(hist_d.cpu().numpy() - oh).max() <= T_ATOL
        lo = [-(-int(L) * 150000 // 1000000) for L in seq_len]
        hi = [int(L) * 400000 // 1000000 for L in seq_len]
        assert all(lo[r] <= got_B[r] <= hi[r] for r in range(R))
    assert ol.tolist() == [120] * R


def test_history_overflow_is_reported():
    R, T, V = 1, 50, 64
    logits, tok = synth.confidence_logits(R, T, V, seed=1, device=DEV)
    hist = torch.zeros((R, 32), dtype=torch.float32, device=DEV)
    lens = torch.zeros(R, dtype=torch.int32, device=DEV)
    _, _, st = _run(logits, tok, hist, lens, torch.tensor([10], dtype=torch.int32, device=DEV),
                    B.BudgetParams.paper_defaults())
    assert st[0] == B.E_INVALID
    assert lens.cpu().tolist() == [32]


def test_trend_only_call_and_ties_at_top_k():
    # top-k boundary inside a run of equal logits: 30 logits at 2.0, k = 20
    V = 500
    z = torch.zeros((70, V), dtype=torch.float32, device=DEV)
    z[:, 100:130] = 2.0
    z[:, 7] = 5.0
    tok = torch.tensor([0, 70], dtype=torch.int32, device=DEV)
    hist0 = torch.zeros((1, 128), dtype=torch.float32)
    len0 = torch.zeros(1, dtype=torch.int32)
    p = B.BudgetParams.paper_defaults()
    _compare(z, tok, hist0, len0, torch.tensor([512], dtype=torch.int32), p)
    # trend-only call on a stored decreasing history
    hist = torch.linspace(9.0, 3.0, 512).view(1, 512).contiguous().to(DEV)
    lens = torch.tensor([512], dtype=torch.int32, device=DEV)
    got_B, got_a, st = _run(None, None, hist, lens, torch.tensor([512], dtype=torch.int32, device=DEV), p)
    assert st[0] == 0 and got_a[0] < 0 and got_B[0] == 896 and lens.cpu().tolist() == [512]


def test_trend_on_a_history_of_the_maximum_length():
    """hist_cap 65536 (the documented maximum): about 8000 pooled windows per request, with runs of equal values
    (window-min pooling) and values drawn on a coarse grid so that the percentile falls among exact ties; the
    percentile, the slope and the decision against the oracle run on the same stored history."""
    cap, R = 65536, 3
    g = torch.Generator().manual_seed(11)
    hist = (torch.randint(0, 4000, (R, cap), generator=g).float() / 256.0 + 2.0)
    hist[1] += torch.linspace(3.0, 0.0, cap)                    # a downward trend
    hist[2] -= torch.linspace(3.0, 0.0, cap)                    # an upward trend
    lens = torch.tensor([cap, 60001, 33333], dtype=torch.int32)
    p = B.BudgetParams.paper_defaults()
    budget_in = torch.tensor([512, 896, 30000], dtype=torch.int32)
    hist_dev, lens_dev = hist.clone().to(DEV), lens.clone().to(DEV)
    got_B, got_a, st = _run(None, None, hist_dev, lens_dev, budget_in.to(DEV), p)
    assert st[0] == 0 and lens_dev.cpu().tolist() == lens.tolist()
    op = _oracle_params(p)
    for r in range(R):
        Rr = O.trace_confidence(hist[r, :int(lens[r])].numpy(), op.w, op.s, op.b_percent)
        a = O.fit_slope(Rr)
        assert abs(got_a[r] - a) <= 1e-12 * max(1.0, abs(a))
        assert got_B[r] == O.budget_update(int(budget_in[r]), a, op, None)
    assert got_a[1] < 0 < got_a[2]


@pytest.mark.parametrize("seed", range(16))
def test_random_monitor_calls(seed):
    """Seeded random calls: ragged row counts per request (some with none), vocabularies that are not multiples
    of the vector width, k from 1 to above the single-sweep limit, window / stride / percentile / scale drawn,
    a history that already holds entries, clamps on or off; history, slope and decision against the oracle."""
    rng = np.random.default_rng(9000 + seed)
    R = int(rng.integers(1, 8))
    V = int(rng.choice([37, 130, 1000, 4099, 32003, 151936]))
    rows = [int(rng.choice([0, rng.integers(1, 30), rng.integers(30, 200)])) for _ in range(R)]
    if V > 30000:
        rows = [min(t, 60) for t in rows]
    if sum(rows) == 0:
        rows[0] = 5
    tok = torch.tensor(np.concatenate([[0], np.cumsum(rows)]), dtype=torch.int32, device=DEV)
    g = torch.Generator(device=DEV).manual_seed(9100 + seed)
    sharp = torch.tensor(rng.uniform(0.3, 5.0, size=sum(rows)), dtype=torch.float32, device=DEV)
    logits = torch.randn((sum(rows), V), generator=g, device=DEV) * sharp[:, None]
    if rng.integers(0, 3) == 0:                                   # a few rows in adversarial order
        n = min(3, sum(rows))
        logits[:n] = torch.sort(logits[:n], dim=1).values
    cap = int(rng.choice([256, 512, 1024]))
    len0 = torch.tensor([int(rng.integers(0, cap - max(rows) + 1)) if rng.integers(0, 2) else 0 for _ in range(R)],
                        dtype=torch.int32)
    hist0 = torch.zeros((R, cap), dtype=torch.float32)
    for r in range(R):
        n = int(len0[r])
        hist0[r, :n] = torch.tensor(rng.uniform(1.0, 9.0, size=n) + np.linspace(0, rng.uniform(-3, 3), n), dtype=torch.float32)
    k = int(rng.choice([1, 5, 20, 20, 64, 65, 100]))
    p = B.BudgetParams(min(k, V), int(rng.choice([8, 32, 64, 100])), int(rng.choice([1, 4, 8, 16])),
                       float(rng.choice([5.0, 10.0, 25.0, 50.0])), float(rng.choice([1.25, 1.75, 2.0])), 30000,
                       150000 if rng.integers(0, 2) else 0, 0)
    if p.clamp_lo_ppm:
        p.clamp_hi_ppm = 400000
    seq_len = torch.tensor(rng.integers(100, 70000, size=R), dtype=torch.int32) if p.clamp_lo_ppm else None
    budget_in = torch.tensor(rng.integers(1, 29000, size=R), dtype=torch.int32)
    _compare(logits, tok, hist0, len0, budget_in, p, seq_len)
