"""actkv_compact_noalloc against actkv_compact, through the C ABI.

Some callers cannot allocate device memory for the compaction plan: an engine that gave all of
HBM to its KV pool, or a plain C host with no allocator.  The entry point under test keeps the
plan in a fixed array inside the library instead.  It must produce exactly what actkv_compact
produces (bytes of the pool, page tables, free list), also on a second call that finds the
array full of the first call's plan, and must refuse tables that do not fit the array.

Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import pytest
import torch

from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import harness as H
from paper_2609_31395_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _scored_and_selected(wl):
    """Instance plus a Compressor that has run score and select (not compact)."""
    inst = synth.generate(wl, DEV)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads,
                        H.sizes_of(inst))
    B.actkv_keep_indptr(inst.seq_len, inst.budget, wl.n_req, comp.keep_indptr)
    comp.run_score(inst.q, inst.win_indptr, inst.tok_indptr, wl.sm_scale, wl.causal)
    comp.run_select(inst.tok_indptr, inst.budget, wl.n_layers)
    return inst, comp


def _same(a, b):
    # compaction is a byte copy: the tolerance of the other compaction tests is exact equality
    assert torch.equal(a.pool.view(torch.int16), b.pool.view(torch.int16))
    assert torch.equal(a.page_table, b.page_table) and torch.equal(a.seq_len, b.seq_len)
    assert torch.equal(a.free_list, b.free_list) and torch.equal(a.free_count, b.free_count)


def _one_round(wl):
    ref, comp_ref = _scored_and_selected(wl)
    new, comp_new = _scored_and_selected(wl)
    assert torch.equal(comp_ref.sel_idx, comp_new.sel_idx)
    comp_ref.run_compact(ref.budget)                                   # existing entry point, caller's workspace
    B.actkv_compact_noalloc(comp_new.pd, comp_new.td, 0, wl.n_layers, comp_new.sel_idx, comp_new.sz.sel_stride,
                            comp_new.keep_indptr, new.budget, comp_new.sz.max_keep, comp_new.status)
    torch.cuda.synchronize()
    assert comp_ref.status.cpu().tolist()[0] == 0 and comp_new.status.cpu().tolist()[0] == 0
    assert ref.seq_len.cpu().tolist() == [min(b, L) for b, L in zip(wl.budgets, wl.seq_lens)]
    _same(ref, new)


def test_noalloc_matches_compact_on_two_calls_in_a_row():
    first = synth.Workload("na1", 2, 2, 4, [900, 333, 130], [8, 5, 16], [250, 100, 130],
                           table_style="fragmented", seed=21, poison_tail=True)
    second = synth.Workload("na2", 1, 4, 2, [70, 2000, 45, 512, 300], [4, 8, 4, 8, 8], [16, 700, 45, 100, 0],
                            table_style="permutation", seed=22)
    _one_round(first)
    _one_round(second)          # different request count and table width: the array holds a stale plan


def test_noalloc_refuses_tables_beyond_its_array():
    assert B.actkv_compact_noalloc_max_bytes() == 1 << 20
    wl = synth.Workload("na3", 1, 1, 2, [64, 64], [4, 4], [16, 16], table_style="permutation", seed=23)
    inst, comp = _scored_and_selected(wl)
    wide = torch.full((2, 200000), -1, dtype=torch.int32, device=DEV)      # 2 x 200000 entries > 1 MiB of plan
    wide[:, : inst.page_table.shape[1]] = inst.page_table
    td = B.tables_desc(wide, inst.seq_len, inst.free_list, inst.free_count)
    before = inst.pool.clone()
    with pytest.raises(B.ActKVError) as e:
        B.actkv_compact_noalloc(comp.pd, td, 0, 1, comp.sel_idx, comp.sz.sel_stride, comp.keep_indptr, inst.budget,
                                comp.sz.max_keep, comp.status)
    assert e.value.code == B.E_TOOBIG
    torch.cuda.synchronize()
    assert torch.equal(before.view(torch.int16), inst.pool.view(torch.int16))
    assert inst.seq_len.cpu().tolist() == [64, 64]
