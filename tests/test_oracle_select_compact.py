"""Pins for the oracle's TopK and compaction (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import actkv_oracle as O
from paper_2609_31395_b200 import synth


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


# ---------------------------------------------------------------------------------- TopK


def _rank_count(score, B):
    """Brute force: entry i is kept iff fewer than n entries beat it (higher score, or equal
    score and lower index)."""
    L = len(score)
    n = min(B, L)
    keep = []
    for i in range(L):
        beats = sum(1 for j in range(L) if score[j] > score[i] or (score[j] == score[i] and j < i))
        if beats < n:
            keep.append(i)
    return keep


@pytest.mark.parametrize("seed", range(5))
def test_select_against_rank_count_with_ties(seed):
    rng = np.random.default_rng(seed)
    L = 97
    score = rng.integers(0, 12, L).astype(np.float32) / 16.0     # many exact ties
    for B in (0, 1, 13, 50, 96, 97, 200):
        assert O.select_unit(score, B).tolist() == _rank_count(score, B)


def test_select_equals_stable_argsort():
    rng = np.random.default_rng(7)
    score = rng.random(5000).astype(np.float32)
    score[100:200] = score[300]                                   # a run of duplicates
    B = 1234
    ref = np.sort(np.argsort(-score, kind="stable")[:B])
    assert np.array_equal(O.select_unit(score, B), ref)


def test_select_tie_rule_visible_on_duplicates():
    score = np.array([0.5, 0.25, 0.5, 0.5, 0.125, 0.5], dtype=np.float32)
    assert O.select_unit(score, 2).tolist() == [0, 2]
    assert O.select_unit(score, 3).tolist() == [0, 2, 3]
    assert O.select_unit(score, 5).tolist() == [0, 1, 2, 3, 5]


def test_select_budget_at_least_length_is_identity():
    score = np.random.default_rng(8).random(33).astype(np.float32)
    assert O.select_unit(score, 33).tolist() == list(range(33))
    assert O.select_unit(score, 1000).tolist() == list(range(33))
    assert O.select_unit(score, 0).tolist() == []


# ---------------------------------------------------------------------------------- compaction


def test_compact_hand_example():
    """P=4, table [7,2,5], L=10, B=5, survivors [1,4,5,8,9], free stack [0,1,3,4,6] (top = 6).
    X=2 -> new pages [6,4]; sources 7*4+1, 2*4+0, 2*4+1, 5*4+0, 5*4+1 = [29,8,9,20,21] go to
    [24,25,26,27,16]; table [6,4,-1]; seq_len 5; free stack [0,1,3,7,2,5], count 6."""
    P, Hkv, D, n_pages = 4, 1, 2, 8
    pool = np.arange(1 * 2 * n_pages * P * Hkv * D, dtype=np.uint16).reshape(1, 2, n_pages, P, Hkv, D)
    tables = O.Tables(np.array([[7, 2, 5]], dtype=np.int32), np.array([10], dtype=np.int32),
                      np.array([0, 1, 3, 4, 6, -1, -1, -1], dtype=np.int32), 5)
    sel = [[[np.array([1, 4, 5, 8, 9])]]]
    new_pool, nt = O.compact(pool, tables, sel, [5])
    flat_old = pool.reshape(1, 2, n_pages * P, Hkv, D)
    flat_new = new_pool.reshape(1, 2, n_pages * P, Hkv, D)
    for s_, d_ in zip([29, 8, 9, 20, 21], [24, 25, 26, 27, 16]):
        assert np.array_equal(flat_new[0, :, d_], flat_old[0, :, s_])
    assert nt.page_table.tolist() == [[6, 4, -1]]
    assert nt.seq_len.tolist() == [5]
    assert nt.free_count == 6
    assert nt.free_list[:6].tolist() == [0, 1, 3, 7, 2, 5]
    # nothing else moved
    untouched = np.ones(n_pages * P, dtype=bool)
    untouched[[24, 25, 26, 27, 16]] = False
    assert np.array_equal(flat_new[:, :, untouched], flat_old[:, :, untouched])


def _instance():
    wl = synth.Workload("tiny", 2, 2, 2, [37, 20, 9], [3, 2, 2], [10, 25, 4], head_dim=8, page_size=4,
                        table_style="fragmented", seed=3, plant_frac=0.0)
    return synth.generate(wl, "cpu")


def _random_sel(inst, rng):
    wl = inst.wl
    return [[[np.sort(rng.choice(L, size=min(B, L), replace=False)) for L, B in zip(wl.seq_lens, wl.budgets)]
             for _ in range(wl.n_kv_heads)] for _ in range(wl.n_layers)]


def test_compact_is_a_selection_of_bytes_and_conserves_pages():
    inst = _instance()
    wl = inst.wl
    P = wl.page_size
    pool = _bits(inst.pool)
    tables = O.Tables(inst.page_table.numpy().copy(), inst.seq_len.numpy().copy(),
                      inst.free_list.numpy().copy(), int(inst.free_count))
    rng = np.random.default_rng(0)
    sel = _random_sel(inst, rng)
    new_pool, nt = O.compact(pool, tables, sel, wl.budgets)
    n_pages = pool.shape[2]
    written = np.zeros(n_pages * P, dtype=bool)
    for r in range(wl.n_req):
        L, B = wl.seq_lens[r], wl.budgets[r]
        if B >= L:                                    # untouched request
            assert np.array_equal(nt.page_table[r], tables.page_table[r]) and nt.seq_len[r] == L
            continue
        old_slots = O.slot_map(tables.page_table[r], L, P)
        new_slots = O.slot_map(nt.page_table[r], B, P)
        written[new_slots] = True
        assert nt.seq_len[r] == B
        assert (nt.page_table[r][-(-B // P):] == -1).all()
        for l in range(wl.n_layers):
            for kv in range(2):
                for h in range(wl.n_kv_heads):
                    got = O.gather_rows(new_pool, l, kv, h, new_slots)
                    want = O.gather_rows(pool, l, kv, h, old_slots[sel[l][h][r]])
                    assert np.array_equal(got, want)
    # bytes outside the destination slots are unchanged
    flat_old = pool.reshape(wl.n_layers, 2, n_pages * P, -1)
    flat_new = new_pool.reshape(wl.n_layers, 2, n_pages * P, -1)
    assert np.array_equal(flat_old[:, :, ~written], flat_new[:, :, ~written])
    # page conservation: every page id exactly once in (tables in use) + (free stack)
    in_use = nt.page_table[nt.page_table >= 0].tolist()
    free = nt.free_list[:nt.free_count].tolist()
    assert sorted(in_use + free) == list(range(n_pages))
    # destination pages came from the top of the old free stack, in pop order
    popped = [int(tables.free_list[tables.free_count - 1 - i]) for i in range(len(in_use))]
    comp_pages = [p for r in range(wl.n_req) if wl.budgets[r] < wl.seq_lens[r]
                  for p in nt.page_table[r][nt.page_table[r] >= 0].tolist()]
    assert comp_pages == popped[:len(comp_pages)]


def test_compact_noop_when_budget_covers_length():
    inst = _instance()
    wl = inst.wl
    pool = _bits(inst.pool)
    tables = O.Tables(inst.page_table.numpy().copy(), inst.seq_len.numpy().copy(),
                      inst.free_list.numpy().copy(), int(inst.free_count))
    big = [L + 5 for L in wl.seq_lens]
    sel = [[[np.arange(L) for L in wl.seq_lens] for _ in range(wl.n_kv_heads)] for _ in range(wl.n_layers)]
    new_pool, nt = O.compact(pool, tables, sel, big)
    assert np.array_equal(new_pool, pool)
    assert np.array_equal(nt.page_table, tables.page_table) and np.array_equal(nt.seq_len, tables.seq_len)
    assert np.array_equal(nt.free_list, tables.free_list) and nt.free_count == tables.free_count


def test_compact_budget_zero_empties_request():
    inst = _instance()
    wl = inst.wl
    pool = _bits(inst.pool)
    tables = O.Tables(inst.page_table.numpy().copy(), inst.seq_len.numpy().copy(),
                      inst.free_list.numpy().copy(), int(inst.free_count))
    budgets = [0, 100, 100]
    sel = [[[np.arange(min(B, L)) for L, B in zip(wl.seq_lens, budgets)] for _ in range(wl.n_kv_heads)]
           for _ in range(wl.n_layers)]
    new_pool, nt = O.compact(pool, tables, sel, budgets)
    assert nt.seq_len[0] == 0 and (nt.page_table[0] == -1).all()
    assert nt.free_count == tables.free_count + -(-wl.seq_lens[0] // wl.page_size)
    assert np.array_equal(new_pool, pool)


def test_compact_free_list_short_raises():
    inst = _instance()
    wl = inst.wl
    tables = O.Tables(inst.page_table.numpy().copy(), inst.seq_len.numpy().copy(),
                      inst.free_list.numpy().copy(), 1)
    sel = _random_sel(inst, np.random.default_rng(1))
    with pytest.raises(RuntimeError):
        O.compact(_bits(inst.pool), tables, sel, wl.budgets)
