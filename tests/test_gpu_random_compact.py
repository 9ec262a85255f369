"""Seeded random cases of the compaction forms called directly, with random ascending keep lists (not
from TopK) on random pool bits: the fresh-page compaction in one call (actkv_compact), the same split into
actkv_compact_begin / actkv_compact_end (work queue, resolve table, drain kernel), the in-place tail
compaction (Algorithm 4) in one call and split into actkv_compact_inplace_begin / _end, each against the oracle
on every byte of the pool, the tables and the free list.
Shapes the step never produces are drawn on purpose: pages of 4 to 64 tokens, 1 to 8 KV heads, head
dimensions whose rows are not a power of two of 16-byte vectors, requests shorter than a page.
"""
import numpy as np
import pytest
import torch

from oracle import actkv_oracle as O
from paper_2609_31395_b200 import binding as B

import parity_util as U
import test_gpu_compact_inplace as TI

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _draw(seed):
    rng = np.random.default_rng(7000 + seed)
    P = int(rng.choice([4, 8, 16, 16, 32, 64]))
    Hkv = int(rng.choice([1, 2, 3, 4, 8]))
    D = int(rng.choice([64, 72, 128, 128, 256]))
    NL = int(rng.integers(1, 4))
    R = int(rng.integers(1, 9))
    lens, budgets = [], []
    for _ in range(R):
        L = int(rng.choice([rng.integers(1, 2 * P + 1), rng.integers(1, 300), rng.integers(300, 1500)]))
        kind = int(rng.integers(0, 7))
        b = [0, 1, L, L + 3, max(1, L // 4), int(rng.integers(1, L + 1)), max(1, L - 1)][kind]
        lens.append(L); budgets.append(int(b))
    return rng, P, Hkv, D, NL, lens, budgets


def _fresh_page_oracle(inst, pool_before, tables_before, sel, ki, budgets, NL):
    wl = inst.wl
    lists = TI._lists(sel, ki, NL, wl.n_kv_heads, wl.n_req)
    return O.compact(pool_before, tables_before, lists, budgets)


def _check_fresh(inst, want_pool, want_t):
    assert np.array_equal(U.bits(inst.pool), want_pool)
    fc = int(inst.free_count.cpu())
    assert np.array_equal(inst.page_table.cpu().numpy(), want_t.page_table)
    assert np.array_equal(inst.seq_len.cpu().numpy(), want_t.seq_len)
    assert fc == want_t.free_count
    assert np.array_equal(inst.free_list.cpu().numpy()[:fc], want_t.free_list[:fc])


@pytest.mark.parametrize("seed", range(24))
@pytest.mark.parametrize("form", ["one call", "begin + end", "in place", "in place, begin + end"])
def test_random_compaction(seed, form):
    rng, P, Hkv, D, NL, lens, budgets = _draw(seed)
    inst, sel, ki, stride, max_keep = TI._direct_case(rng, lens, budgets, P, Hkv, D, NL)
    pool_before, tables_before = U.bits(inst.pool), U.oracle_tables(inst)
    pd = B.pool_desc(inst.pool)
    td = B.tables_desc(inst.page_table, inst.seq_len, inst.free_list, inst.free_count)
    d_sel, d_ki = torch.from_numpy(sel).to(DEV), torch.from_numpy(ki).to(DEV)
    d_bud = torch.tensor(budgets, dtype=torch.int32, device=DEV)
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    if form == "in place":
        d_order = torch.full_like(d_sel, -9)
        B.actkv_compact_inplace(pd, td, 0, NL, d_sel, stride, d_ki, d_bud, max_keep, d_order, status)
        torch.cuda.synchronize()
        assert status.cpu().tolist()[0] == 0, status.cpu().tolist()
        TI._check_against_oracle(inst, pool_before, tables_before, sel, ki, budgets, d_order.cpu().numpy())
        return
    if form == "in place, begin + end":
        d_order = torch.full_like(d_sel, -9) if seed % 2 == 0 else None
        ws = torch.empty(B.actkv_compact_inplace_deferred_workspace_bytes(pd, len(lens), 1, max_keep) + 16,
                         dtype=torch.uint8, device=DEV)
        ws.fill_(0x5A)
        for l in range(NL):                               # layer by layer; the tables change with the last one
            rows = slice(l * Hkv, (l + 1) * Hkv)
            args = (pd, td, l, l + 1, d_sel[rows], stride, d_ki, d_bud, max_keep, None if d_order is None else d_order[rows],
                    ws, status)
            B.actkv_compact_inplace_begin(*args)
            B.actkv_compact_inplace_end(*args)
        torch.cuda.synchronize()
        assert status.cpu().tolist()[0] == 0, status.cpu().tolist()
        TI._check_against_oracle(inst, pool_before, tables_before, sel, ki, budgets,
                                 None if d_order is None else d_order.cpu().numpy())
        if d_order is not None:
            assert (d_order.cpu().numpy()[:, ki[-1]:] == -9).all()
        return
    want_pool, want_t = _fresh_page_oracle(inst, pool_before, tables_before, sel, ki, budgets, NL)
    if form == "one call":
        ws = torch.empty(B.actkv_compact_workspace_bytes(len(lens), td.max_pages) + 16, dtype=torch.uint8, device=DEV)
        B.actkv_compact(pd, td, 0, NL, d_sel, stride, d_ki, d_bud, max_keep, ws, status)
    else:
        ws = torch.empty(B.actkv_compact_deferred_workspace_bytes(pd, len(lens), td.max_pages, NL, max_keep) + 16,
                         dtype=torch.uint8, device=DEV)
        # layer by layer when there are several: the plan of the first call is reused by the later ones
        for l in range(NL):
            args = (pd, td, l, l + 1, d_sel[l * Hkv:(l + 1) * Hkv], stride, d_ki, d_bud, max_keep, ws, status)
            B.actkv_compact_begin(*args, reuse_plan=l > 0)
            B.actkv_compact_end(*args)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0, status.cpu().tolist()
    _check_fresh(inst, want_pool, want_t)
