"""GPU parity of the attention-aware LRFU stage (Section 5.1; Algorithm 1 steps 2-5) through the C ABI:
hit masks, keep-scores and ranking keys bit-exact against the oracle on the same float32 scores;
the survivors' keep-scores gathered exactly; a multi-round agent trace in which keep-scores are
carried through selection and compaction from round to round."""
import math

import numpy as np
import pytest
import torch

from oracle import actkv_oracle as O
from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import harness as H
from paper_2609_31395_b200 import synth

import parity_util as U
import test_gpu_configs as TC

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _f32_bits(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def _unpack_hits(mask_row: np.ndarray, lo: int, hi: int) -> np.ndarray:
    idx = np.arange(lo, hi)
    return ((mask_row.view(np.uint32)[idx >> 5] >> (idx & 31).astype(np.uint32)) & 1).astype(bool)


def _synthetic_scores(rng, n_outer, lens):
    """Pooled-probability-like rows: heavy-tailed values in (0, 1], one unit quantised so that many
    entries tie at the threshold, one unit with exact zeros, a few subnormals."""
    tok = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    sc = np.zeros((n_outer, int(tok[-1])), dtype=np.float32)
    for o in range(n_outer):
        for r, L in enumerate(lens):
            if L == 0:
                continue
            x = rng.exponential(1.0, L) ** 3
            x = (x / x.sum()).astype(np.float32)
            if (o + r) % 3 == 0:
                x = (np.round(x * 2048) / 2048).astype(np.float32)       # a handful of distinct values, zeros
                x[rng.integers(0, L, max(1, L // 7))] = np.float32(1.0 / 2048)
            if (o + r) % 3 == 1 and L > 8:
                x[rng.integers(0, L, 3)] = np.float32(1e-41)             # subnormal scores
            sc[o, tok[r]:tok[r + 1]] = x
    return sc, tok


@pytest.mark.parametrize("top_p", [0.0, 0.5, 0.9, 1.0])
def test_keepscore_matches_oracle_bit_exact(top_p):
    rng = np.random.default_rng(11)
    # empty, tiny, one sweep, exactly one, three sweeps, more than shared memory holds
    lens = [0, 5, 1500, 4096, 9001, 60001]
    n_outer, lam = 3, 0.9
    protect = [0, 2, 100, 0, 5000, 7]
    sc, tok = _synthetic_scores(rng, n_outer, lens)
    ks0 = (rng.random(sc.shape) ** 4).astype(np.float32)
    ks0[:, ::5] = 0.0
    ks0[:, 1::97] = np.float32(3e-42)                    # the decay reaches subnormals
    sum_tok = int(tok[-1])
    d_sc = torch.from_numpy(sc.copy()).to(DEV)
    d_ks = torch.from_numpy(ks0.copy()).to(DEV)
    d_hit = torch.zeros((n_outer, (sum_tok + 31) // 32), dtype=torch.int32, device=DEV)
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    B.actkv_keepscore(d_sc, torch.from_numpy(tok).to(DEV), sum_tok, n_outer, len(lens), top_p, lam,
                      torch.tensor(protect, dtype=torch.int32, device=DEV), d_ks, d_hit, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    got_key, got_ks, got_hit = d_sc.cpu().numpy(), d_ks.cpu().numpy(), d_hit.cpu().numpy()
    n_hits = 0
    for o in range(n_outer):
        for r, L in enumerate(lens):
            a, b = int(tok[r]), int(tok[r + 1])
            hit = O.hit_mask_unit(sc[o, a:b], top_p)
            ks = O.keep_score_update(ks0[o, a:b], sc[o, a:b], hit, lam)
            key = O.rank_keys(ks, min(protect[r], L))
            assert np.array_equal(_unpack_hits(got_hit[o], a, b), hit), f"hit mask of unit ({o},{r})"
            assert np.array_equal(_f32_bits(got_ks[o, a:b]), _f32_bits(ks)), f"keep-score of unit ({o},{r})"
            assert np.array_equal(_f32_bits(got_key[o, a:b]), _f32_bits(key)), f"ranking key of unit ({o},{r})"
            n_hits += int(hit.sum())
    if top_p == 0.0:
        assert n_hits == 0
    else:
        assert n_hits > 0


def test_keepscore_without_optional_arguments_and_empty_calls():
    rng = np.random.default_rng(12)
    lens = [700, 33]
    sc, tok = _synthetic_scores(rng, 2, lens)
    sum_tok = int(tok[-1])
    d_sc = torch.from_numpy(sc.copy()).to(DEV)
    d_ks = torch.zeros_like(d_sc)
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    d_tok = torch.from_numpy(tok).to(DEV)
    B.actkv_keepscore(d_sc, d_tok, sum_tok, 2, 2, 0.9, 0.9, None, d_ks, None, status)
    torch.cuda.synchronize()
    for o in range(2):
        for r in range(2):
            a, b = int(tok[r]), int(tok[r + 1])
            hit = O.hit_mask_unit(sc[o, a:b], 0.9)
            ks = O.keep_score_update(np.zeros(b - a, np.float32), sc[o, a:b], hit, 0.9)
            assert np.array_equal(_f32_bits(d_ks.cpu().numpy()[o, a:b]), _f32_bits(ks))
            assert np.array_equal(_f32_bits(d_sc.cpu().numpy()[o, a:b]), _f32_bits(ks))   # no protected prefix
    before = d_ks.clone()
    B.actkv_keepscore(d_sc, d_tok, sum_tok, 0, 2, 0.9, 0.9, None, d_ks, None, status)       # nothing to do
    torch.cuda.synchronize()
    assert torch.equal(before, d_ks)
    with pytest.raises(B.ActKVError):
        B.actkv_keepscore(d_sc, d_tok, sum_tok, 2, 2, 1.5, 0.9, None, d_ks, None, status)
    with pytest.raises(B.ActKVError):
        B.actkv_keepscore(d_sc, d_tok, sum_tok, 2, 2, 0.9, -0.1, None, d_ks, None, status)


def test_gather_f32_follows_the_index_lists():
    rng = np.random.default_rng(13)
    lens, keep = [50, 0, 3000, 17], [20, 0, 1111, 17]
    tok = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    ki = np.concatenate([[0], np.cumsum(keep)]).astype(np.int32)
    n_outer, stride = 5, int(ki[-1]) + 3
    src = rng.random((n_outer, int(tok[-1]) + 4)).astype(np.float32)
    sel = np.full((n_outer, stride), -1, dtype=np.int32)
    for o in range(n_outer):
        for r in range(len(lens)):
            sel[o, ki[r]:ki[r + 1]] = np.sort(rng.permutation(lens[r])[:keep[r]])
    dst = torch.full((n_outer, stride + 2), -7.0, dtype=torch.float32, device=DEV)
    B.actkv_gather_f32(torch.from_numpy(src).to(DEV), src.shape[1], torch.from_numpy(tok).to(DEV),
                       torch.from_numpy(sel).to(DEV), stride, torch.from_numpy(ki).to(DEV), n_outer, len(lens),
                       stride, dst, stride + 2)
    torch.cuda.synchronize()
    got = dst.cpu().numpy()
    for o in range(n_outer):
        for r in range(len(lens)):
            want = src[o, tok[r] + sel[o, ki[r]:ki[r + 1]]]
            assert np.array_equal(got[o, ki[r]:ki[r + 1]], want)
        assert (got[o, ki[-1]:] == -7.0).all()


@pytest.mark.parametrize("inplace", [False, True])
def test_lrfu_trace_keepscores_travel_with_the_survivors(inplace):
    """Six rounds of a small agent trace under the LRFU policy (p = 0.9, lambda = 0.5, protected
    prompt head): every round the raw scores match the oracle on sampled units, and hit masks,
    keep-scores, index lists, gathered keep-scores, pool and tables match the oracle's policy run on
    the GPU's own float32 scores, with the oracle carrying its own keep-score state.  With
    `inplace` the cache is compacted into the tail blocks (Algorithm 4) and the keep-scores follow
    the new slot order."""
    tr = synth.AgentTrace(n_layers=2, n_kv_heads=2, group=4, n_req=3, n_rounds=6, device=DEV, prompt=(700, 1500),
                          obs=(150, 300), reason=(40, 120), action=(16, 48), max_tokens_per_req=4096, seed=9)
    Hkv, R, NL = tr.Hkv, tr.R, tr.NL
    n_outer = NL * Hkv
    wl_like = (Hkv, tr.G, tr.D, tr.P, True, 1.0 / math.sqrt(tr.D))
    top_p, lam = 0.9, 0.5                                # the Section 8.1 settings
    protect = [64, 0, 200]
    d_protect = torch.tensor(protect, dtype=torch.int32, device=DEV)
    rng = np.random.default_rng(3)
    ks_gpu_prev = None                 # [n_outer, sum kept] packed by the previous round's keep counts
    ks_orc_prev = None                 # [o][r] -> float32 array
    keep_prev = [0] * R
    evicted_protected = 0
    for rnd in range(tr.n_rounds):
        q, win_indptr, tok_indptr, budget, windows, seq = tr.next_round()
        budgets = budget.cpu().tolist()
        keep = [min(b, L) for b, L in zip(budgets, seq)]
        sz = H.StepSizes(R, sum(windows), max(windows), sum(seq), max(seq), max(1, sum(keep)), max(keep))
        comp = H.Compressor(tr.pool, tr.page_table, tr.seq_len, tr.free_list, tr.free_count, Hkv * tr.G, sz)
        # fresh pages keep ascending order, so the protected prompt head stays the first n_protect slots;
        # in place the order changes, so protection travels with the tokens instead: their keep-score
        # starts at +inf (and stays there under the recurrence) and no prefix is named
        lrfu = H.LrfuState(n_outer, sz, DEV, top_p, lam, None if inplace else d_protect, want_hits=True)
        if ks_gpu_prev is not None:
            lrfu.keep_score.copy_(H.extend_keep_scores(ks_gpu_prev, keep_prev, seq))
        elif inplace:
            t0 = tok_indptr.cpu().tolist()
            for r in range(R):
                lrfu.keep_score[:, t0[r]:t0[r] + protect[r]] = float("inf")
        tables_before = O.Tables(tr.page_table.cpu().numpy().copy(), tr.seq_len.cpu().numpy().copy(),
                                 tr.free_list.cpu().numpy().copy(), int(tr.free_count.cpu()))
        pt_before, sl_before = tr.page_table.clone(), tr.seq_len.clone()
        pool_snap = tr.pool.clone()
        snap = pool_snap[0]
        raw = {}

        def marks(name):
            if name == "score":
                raw["score"] = comp.score.clone()

        comp.step(q, win_indptr, tok_indptr, budget, wl_like[5], True, marks=marks, lrfu=lrfu, inplace=inplace)
        torch.cuda.synchronize()
        comp.check_status()
        units = [(int(rng.integers(0, NL)), int(rng.integers(0, Hkv)), int(rng.integers(0, R))) for _ in range(2)]
        TC._check_sampled_scores(pool_snap, pt_before, sl_before, q, win_indptr, tok_indptr, wl_like, raw["score"], units)

        tok = tok_indptr.cpu().numpy()
        ki = comp.keep_indptr.cpu().numpy()
        raw_np = raw["score"].cpu().numpy().reshape(n_outer, -1)
        ks_np = lrfu.keep_score.cpu().numpy()
        kept_np = lrfu.kept.cpu().numpy()
        sel_np = comp.sel_idx.cpu().numpy()
        hit_np = lrfu.hit_mask.cpu().numpy()
        order_np = comp.new_order.cpu().numpy() if inplace else None
        ks_orc_new = [[None] * R for _ in range(n_outer)]
        for o in range(n_outer):
            for r in range(R):
                a, b = int(tok[r]), int(tok[r + 1])
                prev = np.zeros(b - a, dtype=np.float32)
                if ks_orc_prev is not None:
                    prev[: keep_prev[r]] = ks_orc_prev[o][r]
                elif inplace:
                    prev[: protect[r]] = np.inf
                hit = O.hit_mask_unit(raw_np[o, a:b], top_p)
                ks = O.keep_score_update(prev, raw_np[o, a:b], hit, lam)
                sel = O.select_unit(O.rank_keys(ks, 0 if inplace else min(protect[r], b - a)), budgets[r])
                assert np.array_equal(_unpack_hits(hit_np[o], a, b), hit), f"round {rnd} unit ({o},{r}): hit mask"
                assert np.array_equal(_f32_bits(ks_np[o, a:b]), _f32_bits(ks)), f"round {rnd} unit ({o},{r}): KS"
                assert np.array_equal(sel_np[o, ki[r]:ki[r + 1]], sel), f"round {rnd} unit ({o},{r}): TopK"
                now = sel                                       # original token index at every new logical slot
                if inplace and budgets[r] < b - a:
                    src, dst = O.copy_pairs_unit(sel, b - a, budgets[r], tr.P)
                    start = O.tail_region(b - a, budgets[r], tr.P)[2]
                    now = np.arange(start, start + budgets[r])
                    now[dst - start] = src
                if inplace:
                    assert np.array_equal(order_np[o, ki[r]:ki[r + 1]], now), f"round {rnd} unit ({o},{r}): order"
                assert np.array_equal(_f32_bits(kept_np[o, ki[r]:ki[r + 1]]), _f32_bits(ks[now]))
                n_prot = min(protect[r], b - a, budgets[r])
                if inplace:                                     # protected tokens are the +inf ones, wherever they sit
                    evicted_protected += int(n_prot - np.isinf(kept_np[o, ki[r]:ki[r + 1]]).sum())
                else:
                    evicted_protected += int(n_prot - np.isin(np.arange(n_prot), sel).sum())
                ks_orc_new[o][r] = ks[now]
        if inplace:
            lists = [[[sel_np[h, ki[r]:ki[r + 1]] for r in range(R)] for h in range(Hkv)]]
            want_pool, want_t, _ = O.compact_inplace(U.bits(snap)[None], tables_before, lists, budgets, layers=[0])
            assert np.array_equal(U.bits(tr.pool[0])[None], want_pool)
        else:
            want_t = TC._check_layer_compaction(snap, tr.pool[0], tables_before, comp.sel_idx, comp.keep_indptr,
                                                budgets, Hkv, 0)
        TC._check_tables((tr.page_table, tr.seq_len, tr.free_list, tr.free_count), want_t)
        ks_gpu_prev = lrfu.kept[:, : int(ki[-1])].clone()
        ks_orc_prev, keep_prev = ks_orc_new, keep
    assert evicted_protected == 0


@pytest.mark.parametrize("long_unit", [False, True])
def test_fused_keepscore_select_matches_oracle_bit_exact(long_unit):
    """actkv_keepscore_select: keep-score update and TopK in one launch.  Hit masks, keep-scores and index lists
    bit-exact against the oracle run on the same float32 scores (the ranking keys never pass through memory, so the
    index lists are held against the oracle's TopK of the oracle's keys); tie report and keep bitmap consistent;
    with a unit longer than shared memory holds the call falls back to the two kernels and gives the same."""
    rng = np.random.default_rng(21)
    lens = [0, 5, 1500, 4096, 9001, 45568] + ([60001] if long_unit else [])
    budgets = [3, 5, 400, 0, 9001, 12000] + ([15000] if long_unit else [])
    protect = [0, 2, 100, 0, 5000, 7] + ([20000] if long_unit else [])            # one prefix longer than its budget
    n_outer, lam, top_p, R = 3, 0.5, 0.9, len(lens)
    sc, tok = _synthetic_scores(rng, n_outer, lens)
    ks0 = (rng.random(sc.shape) ** 4).astype(np.float32)
    ks0[:, ::5] = 0.0
    sum_tok = int(tok[-1])
    keep = [min(b, L) for b, L in zip(budgets, lens)]
    ki = np.concatenate([[0], np.cumsum(keep)]).astype(np.int32)
    d_sc = torch.from_numpy(sc.copy()).to(DEV)
    d_ks = torch.from_numpy(ks0.copy()).to(DEV)
    d_hit = torch.zeros((n_outer, (sum_tok + 31) // 32), dtype=torch.int32, device=DEV)
    d_keep = torch.zeros_like(d_hit)
    d_sel = torch.full((n_outer, int(ki[-1])), -1, dtype=torch.int32, device=DEV)
    d_tie = torch.zeros((n_outer * R, 4), dtype=torch.int32, device=DEV)
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    B.actkv_keepscore_select(d_sc, torch.from_numpy(tok).to(DEV), sum_tok, max(lens), n_outer, R, top_p, lam,
                             torch.tensor(protect, dtype=torch.int32, device=DEV), d_ks, d_hit,
                             torch.tensor(budgets, dtype=torch.int32, device=DEV), torch.from_numpy(ki).to(DEV), d_sel,
                             int(ki[-1]), d_keep, d_tie, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    if not long_unit:
        assert np.array_equal(_f32_bits(d_sc.cpu().numpy()), _f32_bits(sc)), "the fused form leaves the scores as they were"
    got_ks, got_hit, got_sel = d_ks.cpu().numpy(), d_hit.cpu().numpy(), d_sel.cpu().numpy()
    got_keep, got_tie = d_keep.cpu().numpy(), d_tie.cpu().numpy()
    for o in range(n_outer):
        for r, L in enumerate(lens):
            a, b = int(tok[r]), int(tok[r + 1])
            hit = O.hit_mask_unit(sc[o, a:b], top_p)
            ks = O.keep_score_update(ks0[o, a:b], sc[o, a:b], hit, lam)
            want = O.select_unit(O.rank_keys(ks, min(protect[r], L)), budgets[r])
            assert np.array_equal(_unpack_hits(got_hit[o], a, b), hit), f"hit mask of unit ({o},{r})"
            assert np.array_equal(_f32_bits(got_ks[o, a:b]), _f32_bits(ks)), f"keep-score of unit ({o},{r})"
            assert np.array_equal(got_sel[o, ki[r]:ki[r + 1]], want), f"index list of unit ({o},{r})"
            kept = np.zeros(L, dtype=bool)
            kept[want] = True
            assert np.array_equal(_unpack_hits(got_keep[o], a, b), kept)
            assert got_tie[o * R + r, 3] == keep[r]
    # a budget the index buffer was not sized for is reported and nothing is stored
    status.zero_()
    d_sel.fill_(-7)
    big = torch.tensor([b + 50 for b in budgets], dtype=torch.int32, device=DEV)
    B.actkv_keepscore_select(d_sc, torch.from_numpy(tok).to(DEV), sum_tok, max(lens), n_outer, R, top_p, lam, None, d_ks,
                             None, big, torch.from_numpy(ki).to(DEV), d_sel, int(ki[-1]), None, None, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == B.E_INVALID


@pytest.mark.parametrize("seed", range(12))
def test_random_keepscore_select(seed):
    """Seeded random calls of the fused keep-score update + TopK: unit lengths from empty to beyond one sweep,
    budgets 0 .. above the length, protected prefixes shorter and longer than the budget, top-p and decay drawn
    (including their end points); hit masks, keep-scores and index lists bit-exact against the oracle."""
    rng = np.random.default_rng(8000 + seed)
    R = int(rng.integers(1, 7))
    lens = [int(rng.choice([0, rng.integers(1, 40), rng.integers(40, 5000), rng.integers(5000, 30000)])) for _ in range(R)]
    if max(lens) == 0:
        lens[0] = 17
    budgets = [int(rng.choice([0, 1, L, L + 3, max(1, L // 4), rng.integers(0, L + 1)])) for L in lens]
    protect = [int(rng.choice([0, 0, 1, rng.integers(0, L + 1), L + 2])) for L in lens]
    n_outer = int(rng.integers(1, 4))
    top_p = float(rng.choice([0.0, 0.3, 0.9, 0.99, 1.0]))
    lam = float(rng.choice([0.0, 0.5, 0.9, 1.0]))
    sc, tok = _synthetic_scores(rng, n_outer, lens)
    ks0 = (rng.random(sc.shape) ** 4).astype(np.float32)
    ks0[:, ::3] = 0.0
    sum_tok = int(tok[-1])
    keep = [min(b, L) for b, L in zip(budgets, lens)]
    ki = np.concatenate([[0], np.cumsum(keep)]).astype(np.int32)
    stride = int(ki[-1]) + 3
    d_sc = torch.from_numpy(sc.copy()).to(DEV)
    d_ks = torch.from_numpy(ks0.copy()).to(DEV)
    d_hit = torch.zeros((n_outer, (sum_tok + 31) // 32), dtype=torch.int32, device=DEV)
    d_sel = torch.full((n_outer, stride), -1, dtype=torch.int32, device=DEV)
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    B.actkv_keepscore_select(d_sc, torch.from_numpy(tok).to(DEV), sum_tok, max(lens), n_outer, R, top_p, lam,
                             torch.tensor(protect, dtype=torch.int32, device=DEV), d_ks, d_hit,
                             torch.tensor(budgets, dtype=torch.int32, device=DEV), torch.from_numpy(ki).to(DEV), d_sel,
                             stride, None, None, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0, status.cpu().tolist()
    got_ks, got_hit, got_sel = d_ks.cpu().numpy(), d_hit.cpu().numpy(), d_sel.cpu().numpy()
    for o in range(n_outer):
        for r, L in enumerate(lens):
            a, b = int(tok[r]), int(tok[r + 1])
            hit = O.hit_mask_unit(sc[o, a:b], top_p)
            ks = O.keep_score_update(ks0[o, a:b], sc[o, a:b], hit, lam)
            want = O.select_unit(O.rank_keys(ks, min(protect[r], L)), budgets[r])
            assert np.array_equal(_unpack_hits(got_hit[o], a, b), hit), f"hit mask of unit ({o},{r})"
            assert np.array_equal(_f32_bits(got_ks[o, a:b]), _f32_bits(ks)), f"keep-score of unit ({o},{r})"
            assert np.array_equal(got_sel[o, ki[r]:ki[r + 1]], want), f"index list of unit ({o},{r})"
    assert (got_sel[:, ki[-1]:] == -1).all()
