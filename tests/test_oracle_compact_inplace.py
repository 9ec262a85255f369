"""Pins for the oracle's in-place tail compaction (Section 7.2 equations, Algorithm 4)."""
import numpy as np
import pytest

from oracle import actkv_oracle as O


def test_region_equations_worked_by_hand():
    # block size 4, 10 used slots in 3 blocks, budget 5 -> 2 blocks: region = slots 4..8
    assert O.tail_region(10, 5, 4) == (3, 2, 4, 9)
    # the region may end past the used length, inside the last block (9 used, budget 8 -> slots 4..11)
    assert O.tail_region(9, 8, 4) == (3, 2, 4, 12)
    # budget a whole number of blocks: the region is exactly the last X blocks
    assert O.tail_region(64, 32, 16) == (4, 2, 32, 64)
    # budget 0: nothing is kept, every block is dropped
    assert O.tail_region(10, 0, 4) == (3, 0, 12, 12)
    for L in range(1, 40):
        for B in range(0, L):
            Y, X, s, e = O.tail_region(L, B, 4)
            assert 0 <= s <= e <= Y * 4 and e - s == B and s % 4 == 0      # inside the allocated blocks


def test_copy_pairs_worked_by_hand():
    # keep mask 0100110011 over 10 slots, budget 5, block size 4: inside the region (4..8) slots 6, 7 are
    # holes; survivors outside it are 1 (before) and 9 (after); zipped in ascending order
    src, dst = O.copy_pairs_unit([1, 4, 5, 8, 9], 10, 5, 4)
    assert src.tolist() == [1, 9] and dst.tolist() == [6, 7]
    # region reaching into the unused slots of the last block: 9 used, budget 8; slots 9, 10, 11 are holes
    src, dst = O.copy_pairs_unit([0, 1, 2, 3, 4, 5, 7, 8], 9, 8, 4)
    assert src.tolist() == [0, 1, 2, 3] and dst.tolist() == [6, 9, 10, 11]
    # everything kept already sits in the region: nothing moves
    src, dst = O.copy_pairs_unit([4, 5, 6, 7], 8, 4, 4)
    assert src.size == 0 and dst.size == 0


def test_copy_pairs_against_brute_force_sets():
    rng = np.random.default_rng(0)
    for _ in range(200):
        P = int(rng.choice([1, 2, 4, 16]))
        L = int(rng.integers(1, 90))
        B = int(rng.integers(0, L))
        kept = np.sort(rng.permutation(L)[:B])
        src, dst = O.copy_pairs_unit(kept, L, B, P)
        Y, X, s, e = O.tail_region(L, B, P)
        kept_set = set(kept.tolist())
        want_dst = [p for p in range(s, e) if p not in kept_set]
        want_src = [p for p in sorted(kept_set) if not (s <= p < e)]
        assert dst.tolist() == want_dst and src.tolist() == want_src
        assert not (set(src.tolist()) & set(dst.tolist()))              # conflict-free: one pass suffices
        assert all(d not in kept_set for d in dst.tolist())             # nothing live is overwritten


def _random_case(rng, R=3, P=4, Hkv=2, D=4, NL=2, max_pages=8):
    n_pages = R * max_pages + 5
    perm = rng.permutation(n_pages).astype(np.int32)
    pt = np.full((R, max_pages), -1, dtype=np.int32)
    sl = np.zeros(R, dtype=np.int32)
    used = 0
    for r in range(R):
        L = int(rng.integers(1, max_pages * P + 1))
        Y = -(-L // P)
        pt[r, :Y] = perm[used:used + Y]
        used += Y
        sl[r] = L
    fl = np.full(n_pages, -1, dtype=np.int32)
    fc = n_pages - used
    fl[:fc] = perm[used:]
    pool = rng.integers(0, 2 ** 16, size=(NL, 2, n_pages, P, Hkv, D), dtype=np.uint16)
    return pool, O.Tables(pt, sl, fl, fc)


def test_inplace_compaction_properties():
    rng = np.random.default_rng(1)
    for trial in range(20):
        pool, t = _random_case(rng)
        NL, _, n_pages, P, Hkv, D = pool.shape
        R = len(t.seq_len)
        budget = [int(rng.integers(0, int(t.seq_len[r]) + 3)) for r in range(R)]       # some do not compact
        sel = [[[np.sort(rng.permutation(int(t.seq_len[r]))[:min(budget[r], int(t.seq_len[r]))])
                 for r in range(R)] for _ in range(Hkv)] for _ in range(NL)]
        new_pool, nt, order = O.compact_inplace(pool, t, sel, budget)
        moved_slots_total = 0
        for r in range(R):
            L, B = int(t.seq_len[r]), budget[r]
            if B >= L:                                                   # untouched request
                assert np.array_equal(nt.page_table[r], t.page_table[r]) and nt.seq_len[r] == L
                continue
            Y, X, s, e = O.tail_region(L, B, P)
            assert nt.seq_len[r] == B
            assert nt.page_table[r, :X].tolist() == t.page_table[r, Y - X:Y].tolist()  # the last X blocks stay
            assert (nt.page_table[r, X:] == -1).all()
            new_slots = O.slot_map(nt.page_table[r], B, P)
            old_slots = O.slot_map(t.page_table[r], L, P)
            for a in range(NL):
                for h in range(Hkv):
                    od = order[a][h][r]
                    assert sorted(od.tolist()) == sel[a][h][r].tolist()                # exactly the survivors
                    for kv in range(2):                                                # each where `order` says
                        got = new_pool[a, kv].reshape(n_pages * P, Hkv, D)[new_slots, h]
                        want = pool[a, kv].reshape(n_pages * P, Hkv, D)[old_slots[od], h]
                        assert np.array_equal(got, want)
                    moved_slots_total += int((od != np.arange(s, e)).sum())
        # only destination rows changed: count differing (slot, head) rows <= moves
        diff_rows = (new_pool != pool).any(axis=-1)                                      # [NL, 2, pages, P, Hkv]
        assert int(diff_rows.sum()) <= 2 * moved_slots_total
        # pages are conserved: dropped blocks are on the free list, in request and logical order
        dropped = []
        for r in range(R):
            L, B = int(t.seq_len[r]), budget[r]
            if B < L:
                Y, X, _, _ = O.tail_region(L, B, P)
                dropped += t.page_table[r, :Y - X].tolist()
        assert nt.free_count == t.free_count + len(dropped)
        assert nt.free_list[t.free_count:nt.free_count].tolist() == dropped
        assert np.array_equal(nt.free_list[:t.free_count], t.free_list[:t.free_count])
        live = nt.page_table[nt.page_table >= 0].tolist() + nt.free_list[:nt.free_count].tolist()
        assert sorted(live) == list(range(n_pages))


def test_inplace_and_fresh_page_compaction_hold_the_same_survivors():
    """Both forms keep exactly the selected rows; they differ in slot order (ascending for fresh pages,
    the region's order in place) and in which pages the request ends up holding."""
    rng = np.random.default_rng(2)
    pool, t = _random_case(rng, R=2, max_pages=6)
    NL, _, n_pages, P, Hkv, D = pool.shape
    R = 2
    budget = [max(0, int(t.seq_len[r]) // 2) for r in range(R)]
    sel = [[[np.sort(rng.permutation(int(t.seq_len[r]))[:budget[r]]) for r in range(R)] for _ in range(Hkv)]
           for _ in range(NL)]
    a_pool, a_t, order = O.compact_inplace(pool, t, sel, budget)
    b_pool, b_t = O.compact(pool, t, sel, budget)
    for r in range(R):
        if budget[r] >= int(t.seq_len[r]):
            continue
        sa, sb = O.slot_map(a_t.page_table[r], budget[r], P), O.slot_map(b_t.page_table[r], budget[r], P)
        for a in range(NL):
            for h in range(Hkv):
                rank = np.argsort(order[a][h][r], kind="stable")        # in-place slots in ascending token order
                for kv in range(2):
                    rows_a = a_pool[a, kv].reshape(n_pages * P, Hkv, D)[sa[rank], h]
                    rows_b = b_pool[a, kv].reshape(n_pages * P, Hkv, D)[sb, h]
                    assert np.array_equal(rows_a, rows_b)
    assert a_t.free_count - t.free_count >= 0 and (a_t.seq_len == b_t.seq_len).all()


def test_budget_zero_and_noop():
    rng = np.random.default_rng(3)
    pool, t = _random_case(rng, R=2)
    NL, _, n_pages, P, Hkv, D = pool.shape
    L0, L1 = int(t.seq_len[0]), int(t.seq_len[1])
    budget = [0, L1 + 5]
    sel = [[[np.zeros(0, dtype=np.int64), np.arange(L1)] for _ in range(Hkv)] for _ in range(NL)]
    new_pool, nt, _ = O.compact_inplace(pool, t, sel, budget)
    assert np.array_equal(new_pool, pool)                                # nothing to move in either case
    assert nt.seq_len.tolist() == [0, L1] and (nt.page_table[0] == -1).all()
    assert np.array_equal(nt.page_table[1], t.page_table[1])
    assert nt.free_count == t.free_count + -(-L0 // P)
