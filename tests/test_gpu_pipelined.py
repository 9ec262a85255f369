"""The compaction of a layer group hidden under the score kernels of the next group
(actkv_compact_begin / actkv_score_overlap / actkv_compact_end): the copies are taken from a work
queue by spare warps of the tensor-core score kernels and by a drain kernel.  Whoever executes an
item, the result must be exactly what actkv_compact gives, which the other tests hold against the
oracle; here the one-call step is checked against the oracle first and the pipelined step against
it bit for bit.
"""
import numpy as np
import pytest
import torch

from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import harness as H
from paper_2609_31395_b200 import synth

import parity_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _same_state(a, b):
    assert torch.equal(a.pool.view(torch.int16), b.pool.view(torch.int16))
    assert torch.equal(a.page_table, b.page_table) and torch.equal(a.seq_len, b.seq_len)
    assert torch.equal(a.free_list, b.free_list) and torch.equal(a.free_count, b.free_count)


def _reference(wl):
    """One-call step, checked against the oracle (scores, index lists, every byte of the pool, tables)."""
    a = synth.generate(wl, DEV)
    pool_before, tables_before = U.bits(a.pool), U.oracle_tables(a)
    comp = U.run_step(a)
    comp.check_status()
    want, lse, tok, err = U.check_scores(a, comp, pool_before, tables_before)
    sel, ki = comp.sel_idx.cpu().numpy(), comp.keep_indptr.cpu().numpy()
    U.check_select_exact(comp.score.cpu().numpy().reshape(-1, want.shape[-1]), tok, wl.budgets, sel, ki)
    U.check_compaction(a, pool_before, tables_before, sel, ki, wl.budgets)
    return a, comp


def _pipelined(wl, lpc, groups=None, lse_in=None, lse_lpc=None):
    b = synth.generate(wl, DEV)
    comp = H.Compressor(b.pool, b.page_table, b.seq_len, b.free_list, b.free_count, wl.n_q_heads, H.sizes_of(b),
                        layers_per_call=lpc, want_lse=True, lse_layers_per_call=lse_lpc)
    comp.step_pipelined(b.q, b.win_indptr, b.tok_indptr, b.budget, wl.sm_scale, wl.causal, lse_in=lse_in, groups=groups)
    torch.cuda.synchronize()
    comp.check_status()
    return b, comp


@pytest.mark.parametrize("causal", [False, True])
def test_pipelined_step_equals_the_one_call_step(causal):
    # 7 layers in groups of 2, 2, 2, 1; 256 window rows (tensor-core path), ragged last pages, one request that
    # keeps everything (B >= L) and one that is emptied (B = 0)
    wl = synth.Workload("pipe", 7, 2, 8, [1500, 333, 700, 90, 260], [32, 16, 24, 8, 32], [400, 100, 200, 90, 0],
                        table_style="fragmented", causal=causal, seed=51, poison_tail=True)
    a, comp_a = _reference(wl)
    b, comp_b = _pipelined(wl, 2)
    _same_state(a, b)
    # (the LSE pass cuts the keys into chunks by the size of the launch, so its last bits depend on the grouping)
    assert torch.allclose(comp_a.lse, comp_b.lse, rtol=0, atol=1e-5)
    # with the LSE supplied (no LSE kernel: all copies ride on the pooled-score kernel or the drain)
    c, _ = _pipelined(wl, 2, lse_in=comp_a.lse)
    _same_state(a, c)
    # the LSE pass of all layers first, in one call of its own, then the groups
    d, comp_d = _pipelined(wl, 2, lse_lpc=7)
    _same_state(a, d)
    assert torch.equal(comp_a.lse, comp_d.lse)


def test_uneven_groups_and_other_shapes():
    # head_dim 64 (8 vectors per row), 4 heads x pages of 32 tokens = 128 (slot, head) pairs per page
    wl = synth.Workload("pipe64", 5, 4, 4, [1100, 257, 64], [32, 16, 16], [300, 64, 10], head_dim=64, page_size=32,
                        table_style="permutation", seed=52, poison_tail=True)
    a, _ = _reference(wl)
    b, _ = _pipelined(wl, 3, groups=[(0, 3), (3, 4), (4, 5)])
    _same_state(a, b)
    # a window below 64 rows: the FMA score kernels, which carry no copy role: the drain kernel copies everything
    wl2 = synth.Workload("pipefma", 4, 2, 2, [500, 130], [8, 4], [120, 40], table_style="fragmented", seed=53,
                         poison_tail=True)
    a2, _ = _reference(wl2)
    b2, _ = _pipelined(wl2, 1)
    _same_state(a2, b2)


def test_begin_plus_end_is_compact_and_errors_leave_everything_untouched():
    wl = synth.Workload("be", 2, 2, 4, [900, 333, 130], [16, 8, 16], [250, 100, 130], table_style="fragmented", seed=54,
                        poison_tail=True)
    a, comp_a = _reference(wl)
    b = synth.generate(wl, DEV)
    comp = H.Compressor(b.pool, b.page_table, b.seq_len, b.free_list, b.free_count, wl.n_q_heads, H.sizes_of(b))
    B.actkv_keep_indptr(b.seq_len, b.budget, wl.n_req, comp.keep_indptr)
    comp.run_score(b.q, b.win_indptr, b.tok_indptr, wl.sm_scale, wl.causal)
    comp.run_select(b.tok_indptr, b.budget, wl.n_layers)
    args = (comp.pd, comp.td, 0, wl.n_layers, comp.sel_idx, comp.sz.sel_stride, comp.keep_indptr, b.budget,
            comp.sz.max_keep, comp.ws_compact, comp.status)
    assert comp.ws_compact.numel() >= B.actkv_compact_deferred_workspace_bytes(comp.pd, wl.n_req, comp.td.max_pages,
                                                                                wl.n_layers, comp.sz.max_keep)
    # a free list that is too short: reported by the plan, nothing is copied by anyone, tables stay
    snap = [U.bits(b.pool).copy()] + [t.clone() for t in (b.page_table, b.seq_len, b.free_list, b.free_count)]
    fc = b.free_count.clone()
    b.free_count.fill_(3)
    snap[4] = b.free_count.clone()
    B.actkv_compact_begin(*args)
    B.actkv_compact_end(*args)
    torch.cuda.synchronize()
    assert comp.status.cpu().tolist()[0] == B.E_NOFREE
    assert np.array_equal(U.bits(b.pool), snap[0])
    for t, s0 in zip((b.page_table, b.seq_len, b.free_list, b.free_count), snap[1:]):
        assert torch.equal(t, s0)
    # the real thing
    b.free_count.copy_(fc)
    comp.status.zero_()
    B.actkv_compact_begin(*args)
    B.actkv_compact_end(*args)
    torch.cuda.synchronize()
    comp.check_status()
    _same_state(a, b)


@pytest.mark.parametrize("deferred", [False, True])
def test_a_bad_page_id_in_a_table_stops_the_compaction_before_anything_is_modified(deferred):
    """A page id outside the pool in a page table (of a page that holds evicted tokens only, so that no copy would
    ever read it): reported by the plan, which checks every page it would push on the free list; pool, tables and
    free list stay as they were."""
    wl = synth.Workload("badpage", 2, 2, 4, [900, 333], [16, 8], [250, 100], table_style="fragmented", seed=55,
                        poison_tail=True)
    b = synth.generate(wl, DEV)
    comp = H.Compressor(b.pool, b.page_table, b.seq_len, b.free_list, b.free_count, wl.n_q_heads, H.sizes_of(b))
    B.actkv_keep_indptr(b.seq_len, b.budget, wl.n_req, comp.keep_indptr)
    comp.run_score(b.q, b.win_indptr, b.tok_indptr, wl.sm_scale, wl.causal)
    comp.run_select(b.tok_indptr, b.budget, wl.n_layers)
    torch.cuda.synchronize()
    comp.check_status()
    b.page_table[1, 3] = b.pool.shape[2] + 5                       # out of range
    snap = [U.bits(b.pool).copy()] + [t.clone() for t in (b.page_table, b.seq_len, b.free_list, b.free_count)]
    args = (comp.pd, comp.td, 0, wl.n_layers, comp.sel_idx, comp.sz.sel_stride, comp.keep_indptr, b.budget,
            comp.sz.max_keep, comp.ws_compact, comp.status)
    if deferred:
        B.actkv_compact_begin(*args)
        B.actkv_compact_end(*args)
    else:
        B.actkv_compact(*args)
    torch.cuda.synchronize()
    st = comp.status.cpu().tolist()
    assert st[0] == B.E_BADPAGE and st[1] == 1 and st[2] == b.pool.shape[2] + 5
    assert np.array_equal(U.bits(b.pool), snap[0])
    for t, s0 in zip((b.page_table, b.seq_len, b.free_list, b.free_count), snap[1:]):
        assert torch.equal(t, s0)


def test_reusing_a_plan_that_is_not_there_is_reported_and_nothing_moves():
    """actkv_compact_begin with reuse_plan on a workspace that holds no plan of these tables (never written, or
    written for another pool): reported as an invalid call; neither begin + end nor a following score call with the
    workspace as its pending compaction copies anything or touches the tables."""
    wl = synth.Workload("noplan", 2, 2, 8, [900, 333], [16, 8], [250, 100], table_style="fragmented", seed=56,
                        poison_tail=True)
    b = synth.generate(wl, DEV)
    comp = H.Compressor(b.pool, b.page_table, b.seq_len, b.free_list, b.free_count, wl.n_q_heads, H.sizes_of(b))
    B.actkv_keep_indptr(b.seq_len, b.budget, wl.n_req, comp.keep_indptr)
    comp.run_score(b.q, b.win_indptr, b.tok_indptr, wl.sm_scale, wl.causal)
    comp.run_select(b.tok_indptr, b.budget, wl.n_layers)
    torch.cuda.synchronize()
    comp.check_status()
    snap = [U.bits(b.pool).copy()] + [t.clone() for t in (b.page_table, b.seq_len, b.free_list, b.free_count)]
    args = (comp.pd, comp.td, 0, wl.n_layers, comp.sel_idx, comp.sz.sel_stride, comp.keep_indptr, b.budget,
            comp.sz.max_keep, comp.ws_compact, comp.status)
    for fill in (0, 0x5A):
        comp.ws_compact.fill_(fill)
        comp.status.zero_()
        B.actkv_compact_begin(*args, reuse_plan=True)
        s = comp.sz
        B.actkv_score_overlap(comp.pd, comp.td, 0, wl.n_layers, b.q, b.win_indptr, wl.n_q_heads, None, wl.sm_scale, wl.causal,
                              b.tok_indptr, comp.score, None, s.sum_win, s.max_win, s.sum_tok, s.max_tok, comp.ws_score,
                              comp.ws_compact, comp.status)
        B.actkv_compact_end(*args)
        torch.cuda.synchronize()
        assert comp.status.cpu().tolist()[0] == B.E_INVALID
        assert np.array_equal(U.bits(b.pool), snap[0])
        for t, s0 in zip((b.page_table, b.seq_len, b.free_list, b.free_count), snap[1:]):
            assert torch.equal(t, s0)
    # a plan of another instance's tables in the workspace is refused as well
    c = synth.generate(wl, DEV)
    comp_c = H.Compressor(c.pool, c.page_table, c.seq_len, c.free_list, c.free_count, wl.n_q_heads, H.sizes_of(c))
    comp.status.zero_()
    B.actkv_compact_begin(comp_c.pd, comp_c.td, 0, wl.n_layers, comp.sel_idx, comp.sz.sel_stride, comp.keep_indptr, b.budget,
                          comp.sz.max_keep, comp.ws_compact, comp.status)
    B.actkv_compact_begin(*args, reuse_plan=True)
    B.actkv_compact_end(*args)
    torch.cuda.synchronize()
    assert comp.status.cpu().tolist()[0] == B.E_INVALID
    assert np.array_equal(U.bits(b.pool), snap[0])
    for t, s0 in zip((b.page_table, b.seq_len, b.free_list, b.free_count), snap[1:]):
        assert torch.equal(t, s0)


@pytest.mark.parametrize("causal", [False, True])
def test_pipelined_in_place_step_equals_the_one_call_in_place_step(causal):
    """Algorithm 4's in-place compaction with the moves of a layer group executed inside the pooled-score kernel of
    the next group (actkv_compact_inplace_begin / actkv_score_overlap / actkv_compact_inplace_end): pool, tables and
    free list bit for bit those of the one-call in-place step, which tests/test_gpu_compact_inplace.py holds
    against the oracle."""
    wl = synth.Workload("pipe-ip", 7, 2, 8, [1500, 333, 700, 90, 260], [32, 16, 24, 8, 32], [400, 100, 200, 90, 0],
                        table_style="fragmented", causal=causal, seed=57, poison_tail=True)
    a = synth.generate(wl, DEV)
    comp_a = H.Compressor(a.pool, a.page_table, a.seq_len, a.free_list, a.free_count, wl.n_q_heads, H.sizes_of(a),
                          want_lse=True)
    comp_a.step(a.q, a.win_indptr, a.tok_indptr, a.budget, wl.sm_scale, wl.causal, inplace=True)
    torch.cuda.synchronize()
    comp_a.check_status()
    for lpc, lse_in in ((2, None), (3, comp_a.lse)):
        b = synth.generate(wl, DEV)
        comp_b = H.Compressor(b.pool, b.page_table, b.seq_len, b.free_list, b.free_count, wl.n_q_heads, H.sizes_of(b),
                              layers_per_call=lpc, want_lse=True)
        stats = torch.zeros((8, 2), dtype=torch.int32, device=DEV)
        comp_b.step_pipelined(b.q, b.win_indptr, b.tok_indptr, b.budget, wl.sm_scale, wl.causal, lse_in=lse_in, inplace=True,
                              stats=stats)
        torch.cuda.synchronize()
        comp_b.check_status()
        _same_state(a, b)
        st = stats.cpu().numpy()
        assert st[0, 0] > 0 and (st[:, 1] <= st[:, 0]).all()          # a queue was published for the first group


def test_pipelined_step_with_the_lrfu_policy_equals_the_one_call_form():
    """Ranking by the LRFU keep-score (Section 5.1) in the pipelined step: pool, tables, persistent keep-scores and
    the survivors' keep-scores bit for bit those of the one-call form (held against the oracle in
    tests/test_gpu_keepscore.py)."""
    wl = synth.Workload("pipe-lrfu", 5, 2, 8, [1500, 333, 700, 90], [32, 16, 24, 8], [400, 100, 200, 90],
                        table_style="fragmented", seed=58, poison_tail=True)
    out = []
    for lpc in (None, 2):
        a = synth.generate(wl, DEV)
        sz = H.sizes_of(a)
        comp = H.Compressor(a.pool, a.page_table, a.seq_len, a.free_list, a.free_count, wl.n_q_heads, sz, layers_per_call=lpc)
        lrfu = H.LrfuState(wl.n_layers * wl.n_kv_heads, sz, DEV, 0.9, 0.5,
                           torch.tensor([4, 0, 300, 7], dtype=torch.int32, device=DEV), want_hits=True)
        lrfu.keep_score.uniform_(0.0, 1e-3, generator=torch.Generator(device=DEV).manual_seed(3))
        if lpc is None:
            comp.step(a.q, a.win_indptr, a.tok_indptr, a.budget, wl.sm_scale, wl.causal, lrfu=lrfu)
        else:
            comp.step_pipelined(a.q, a.win_indptr, a.tok_indptr, a.budget, wl.sm_scale, wl.causal, lrfu=lrfu)
        torch.cuda.synchronize()
        comp.check_status()
        out.append((a, lrfu))
    (a, la), (b, lb) = out
    _same_state(a, b)
    assert torch.equal(la.keep_score.view(torch.int32), lb.keep_score.view(torch.int32))
    assert torch.equal(la.hit_mask, lb.hit_mask)
    n_keep = sum(min(x, L) for x, L in zip(wl.budgets, wl.seq_lens))
    assert torch.equal(la.kept[:, :n_keep].view(torch.int32), lb.kept[:, :n_keep].view(torch.int32))
