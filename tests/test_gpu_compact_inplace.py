"""GPU parity of the in-place tail compaction (Section 7.2 region equations, Algorithm 4) through the
C ABI: pool (every byte), tables, free list and the new slot order bit-exact against the oracle."""
import numpy as np
import pytest
import torch

from oracle import actkv_oracle as O
from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import harness as H
from paper_2609_31395_b200 import synth

import parity_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _lists(sel_idx, keep_indptr, n_layers, Hkv, R):
    return [[[sel_idx[a * Hkv + h, keep_indptr[r]:keep_indptr[r + 1]] for r in range(R)] for h in range(Hkv)]
            for a in range(n_layers)]


def _check_against_oracle(inst, pool_before, tables_before, sel_idx, keep_indptr, budgets, new_order=None):
    wl = inst.wl
    NL, Hkv, R = pool_before.shape[0], wl.n_kv_heads, wl.n_req
    want_pool, want_t, order = O.compact_inplace(pool_before, tables_before, _lists(sel_idx, keep_indptr, NL, Hkv, R),
                                                 budgets)
    assert np.array_equal(U.bits(inst.pool), want_pool)              # valid slots equal, nothing else touched
    fc = int(inst.free_count.cpu())
    assert np.array_equal(inst.page_table.cpu().numpy(), want_t.page_table)
    assert np.array_equal(inst.seq_len.cpu().numpy(), want_t.seq_len)
    assert fc == want_t.free_count
    assert np.array_equal(inst.free_list.cpu().numpy()[:fc], want_t.free_list[:fc])
    if new_order is not None:
        for a in range(NL):
            for h in range(Hkv):
                for r in range(R):
                    got = new_order[a * Hkv + h, keep_indptr[r]:keep_indptr[r + 1]]
                    want = order[a][h][r]
                    if want is None:                                 # untouched request: the list itself
                        want = sel_idx[a * Hkv + h, keep_indptr[r]:keep_indptr[r + 1]]
                    assert np.array_equal(got, want), f"order of unit ({a},{h},{r})"
    return want_t


def _direct_case(rng, lens, budgets, P, Hkv, D, NL, slack_pages=3):
    """Random pool bits, a permuted page table, random ascending keep lists (not from TopK)."""
    R = len(lens)
    max_pages = max(-(-L // P) for L in lens) + 1
    wl = synth.Workload("direct", NL, Hkv, 1, list(lens), [1] * R, list(budgets), head_dim=D, page_size=P,
                        table_style="permutation", seed=int(rng.integers(1 << 20)))
    inst = synth.generate(wl, DEV)
    inst.pool.view(torch.int16).copy_(torch.from_numpy(
        rng.integers(-2 ** 15, 2 ** 15, size=tuple(inst.pool.shape), dtype=np.int16)).to(DEV))
    keep = [min(b, L) for b, L in zip(budgets, lens)]
    ki = np.concatenate([[0], np.cumsum(keep)]).astype(np.int32)
    stride = int(ki[-1]) + 5
    sel = np.full((NL * Hkv, stride), -1, dtype=np.int32)
    for o in range(NL * Hkv):
        for r in range(R):
            sel[o, ki[r]:ki[r + 1]] = np.sort(rng.permutation(lens[r])[:keep[r]])
    return inst, sel, ki, stride, max(keep + [1])


@pytest.mark.parametrize("P,Hkv,D", [(16, 2, 128), (8, 3, 64), (4, 1, 72), (16, 4, 256)])
def test_direct_call_random_lists(P, Hkv, D):
    rng = np.random.default_rng(P * 1000 + D)
    lens = [1000, 333, 130, 17, 33, 64, 1]
    budgets = [250, 333, 0, 20, 30, 16, 0]          # compacting, no-op (B = L), empty, no-op (B > L), region past L, ...
    NL = 2
    inst, sel, ki, stride, max_keep = _direct_case(rng, lens, budgets, P, Hkv, D, NL)
    pool_before, tables_before = U.bits(inst.pool), U.oracle_tables(inst)
    d_sel = torch.from_numpy(sel).to(DEV)
    d_order = torch.full_like(d_sel, -9)
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    B.actkv_compact_inplace(B.pool_desc(inst.pool), B.tables_desc(inst.page_table, inst.seq_len, inst.free_list,
                                                                  inst.free_count), 0, NL, d_sel, stride,
                            torch.from_numpy(ki).to(DEV), torch.tensor(budgets, dtype=torch.int32, device=DEV), max_keep,
                            d_order, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    _check_against_oracle(inst, pool_before, tables_before, sel, ki, budgets, d_order.cpu().numpy())
    assert (d_order.cpu().numpy()[:, ki[-1]:] == -9).all()


def test_layer_sub_ranges_and_no_order_output():
    rng = np.random.default_rng(5)
    lens, budgets, NL = [700, 90], [300, 33], 3
    inst, sel, ki, stride, max_keep = _direct_case(rng, lens, budgets, 16, 2, 128, NL)
    pool_before, tables_before = U.bits(inst.pool), U.oracle_tables(inst)
    pd = B.pool_desc(inst.pool)
    td = B.tables_desc(inst.page_table, inst.seq_len, inst.free_list, inst.free_count)
    d_sel, d_ki = torch.from_numpy(sel).to(DEV), torch.from_numpy(ki).to(DEV)
    d_bud = torch.tensor(budgets, dtype=torch.int32, device=DEV)
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    Hkv = 2
    for l0, l1 in ((0, 1), (1, 3)):                 # tables change only on the call that ends at the last layer
        B.actkv_compact_inplace(pd, td, l0, l1, d_sel[l0 * Hkv:l1 * Hkv], stride, d_ki, d_bud, max_keep, None, status)
        torch.cuda.synchronize()
        if l1 < NL:
            assert np.array_equal(inst.page_table.cpu().numpy(), tables_before.page_table)
            assert np.array_equal(inst.seq_len.cpu().numpy(), tables_before.seq_len)
    assert status.cpu().tolist()[0] == 0
    _check_against_oracle(inst, pool_before, tables_before, sel, ki, budgets)


@pytest.mark.parametrize("causal", [False, True])
def test_step_with_inplace_compaction(causal):
    wl = synth.Workload("small", 2, 2, 4, [1000, 333, 130, 17], [8, 5, 16, 3], [250, 100, 130, 4],
                        causal=causal, table_style="fragmented", seed=3, poison_tail=True)
    inst = synth.generate(wl, DEV)
    pool_before, tables_before = U.bits(inst.pool), U.oracle_tables(inst)
    sz = H.sizes_of(inst)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads, sz)
    comp.step(inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, wl.sm_scale, wl.causal, inplace=True)
    torch.cuda.synchronize()
    comp.check_status()
    sel_idx, ki = comp.sel_idx.cpu().numpy(), comp.keep_indptr.cpu().numpy()
    score_gpu = comp.score.cpu().numpy().reshape(-1, comp.score.shape[-1])
    U.check_select_exact(score_gpu, inst.tok_indptr.cpu().numpy(), wl.budgets, sel_idx, ki)
    _check_against_oracle(inst, pool_before, tables_before, sel_idx, ki, wl.budgets)
    # fewer rows moved than the fresh-page form would copy: only survivors outside the tail region
    free_after = int(inst.free_count.cpu())
    assert free_after > tables_before.free_count                       # pages came back, none were taken


def test_status_already_set_and_bad_lists_leave_tables_alone():
    rng = np.random.default_rng(6)
    lens, budgets, NL = [400, 50], [100, 20], 1
    inst, sel, ki, stride, max_keep = _direct_case(rng, lens, budgets, 16, 2, 128, NL)
    tables_before = U.oracle_tables(inst)
    pool_before = U.bits(inst.pool)
    pd = B.pool_desc(inst.pool)
    td = B.tables_desc(inst.page_table, inst.seq_len, inst.free_list, inst.free_count)
    d_ki = torch.from_numpy(ki).to(DEV)
    d_bud = torch.tensor(budgets, dtype=torch.int32, device=DEV)
    # an earlier stage reported an error: nothing runs
    status = torch.tensor([B.E_BADPAGE, 0, 0, 0], dtype=torch.int32, device=DEV)
    B.actkv_compact_inplace(pd, td, 0, NL, torch.from_numpy(sel).to(DEV), stride, d_ki, d_bud, max_keep, None, status)
    torch.cuda.synchronize()
    assert np.array_equal(U.bits(inst.pool), pool_before)
    assert np.array_equal(inst.page_table.cpu().numpy(), tables_before.page_table)
    # a list that is not ascending / out of range is reported, tables stay, live rows stay
    bad = sel.copy()
    bad[0, ki[0]:ki[0] + 100] = bad[0, ki[0]:ki[0] + 100][::-1]
    bad[1, ki[1] + 3] = 10 ** 6
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    B.actkv_compact_inplace(pd, td, 0, NL, torch.from_numpy(bad).to(DEV), stride, d_ki, d_bud, max_keep, None, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == B.E_BADINDEX
    assert np.array_equal(inst.page_table.cpu().numpy(), tables_before.page_table)
    assert np.array_equal(inst.seq_len.cpu().numpy(), tables_before.seq_len)
    assert int(inst.free_count.cpu()) == tables_before.free_count


def test_host_argument_errors():
    rng = np.random.default_rng(7)
    inst, sel, ki, stride, max_keep = _direct_case(rng, [64], [16], 16, 1, 128, 1)
    pd = B.pool_desc(inst.pool)
    td = B.tables_desc(inst.page_table, inst.seq_len, inst.free_list, inst.free_count)
    args = (torch.from_numpy(sel).to(DEV), stride, torch.from_numpy(ki).to(DEV),
            torch.tensor([16], dtype=torch.int32, device=DEV), max_keep, None,
            torch.zeros(4, dtype=torch.int32, device=DEV))
    with pytest.raises(B.ActKVError):
        B.actkv_compact_inplace(pd, td, 1, 0, *args)                    # empty / reversed layer range
    with pytest.raises(B.ActKVError):
        B.actkv_compact_inplace(pd, td, 0, 2, *args)                    # past the pool's layers
