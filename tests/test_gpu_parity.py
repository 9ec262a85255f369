"""GPU parity: every step of the CUDA path, called through the C ABI, against the CPU oracle."""
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


def _small(causal=False, head_dim=128, page=16, G=4, seed=0, **kw):
    """Several tiles and ragged tails: lengths not multiples of the page, the 64-key FMA tile or
    the 128-key tensor tile; ragged windows."""
    return synth.Workload("small", 2, 2, G, [1000, 333, 130, 17], [8, 5, 16, 3], [250, 100, 130, 4],
                          head_dim=head_dim, page_size=page, causal=causal, table_style="fragmented",
                          seed=seed, poison_tail=True, **kw)


def _full_check(inst, lse_in=None, layers_per_call=None):
    wl = inst.wl
    pool_before = U.bits(inst.pool)
    tables_before = U.oracle_tables(inst)
    comp = U.run_step(inst, lse_in=lse_in, layers_per_call=layers_per_call)
    comp.check_status()
    keep_indptr = comp.keep_indptr.cpu().numpy()
    sel_idx = comp.sel_idx.cpu().numpy()
    want_keep = np.concatenate([[0], np.cumsum([min(b, L) for b, L in zip(wl.budgets, wl.seq_lens)])])
    assert np.array_equal(keep_indptr, want_keep)
    out = {}
    if layers_per_call is None:
        lse_np = None if lse_in is None else lse_in.cpu().numpy().astype(np.float64)
        want, lse, tok, err = U.check_scores(inst, comp, pool_before, tables_before, lse_in=lse_np)
        if lse_in is None:
            got_lse = comp.lse.cpu().numpy()
            m = ~np.isnan(lse)
            assert np.abs(got_lse[m] - lse[m]).max() < 1e-4
        score_gpu = comp.score.cpu().numpy().reshape(-1, comp.score.shape[-1])
        U.check_select_exact(score_gpu, tok, wl.budgets, sel_idx, keep_indptr)
        out["ties"] = U.check_select_vs_oracle_scores(want.reshape(-1, want.shape[-1]), tok, wl.budgets, sel_idx,
                                                      keep_indptr)
        out["lse"] = lse
        out["err"] = err
        U.check_compaction(inst, pool_before, tables_before, sel_idx, keep_indptr, wl.budgets)
    out["comp"] = comp
    return out


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("head_dim,page,G", [(128, 16, 4), (64, 8, 2), (128, 16, 8)])
def test_pipeline_small(causal, head_dim, page, G):
    wl = _small(causal=causal, head_dim=head_dim, page=page, G=G)
    if causal:
        wl.windows = [min(w, L) for w, L in zip(wl.windows, wl.seq_lens)]
    inst = synth.generate(wl, DEV)
    _full_check(inst)


def test_pipeline_supplied_lse_matches_internal():
    inst = synth.generate(_small(), DEV)
    r1 = _full_check(inst)
    lse = r1["comp"].lse.clone()
    score_internal = r1["comp"].score.clone()
    inst2 = synth.generate(_small(), DEV)
    r2 = _full_check(inst2, lse_in=lse)
    # the same LSE values give the same scores bit for bit
    assert torch.equal(score_internal, r2["comp"].score)


def test_layer_sub_ranges_give_the_same_result():
    a = synth.generate(_small(), DEV)
    b = synth.generate(_small(), DEV)
    _full_check(a)
    _full_check(b, layers_per_call=1)
    assert torch.equal(a.pool.view(torch.int16), b.pool.view(torch.int16))
    assert torch.equal(a.page_table, b.page_table) and torch.equal(a.seq_len, b.seq_len)
    assert torch.equal(a.free_list, b.free_list) and torch.equal(a.free_count, b.free_count)


def test_overlapped_step_gives_the_same_result():
    """select + compact of layer group g on a second stream under the score of group g+1."""
    wl = synth.Workload("ovl", 5, 2, 8, [1200, 333, 700], [32, 16, 64], [300, 100, 200],
                        table_style="fragmented", seed=12, poison_tail=True)
    a = synth.generate(wl, DEV)
    b = synth.generate(wl, DEV)
    _full_check(a)
    sz = H.sizes_of(b)
    comp = H.Compressor(b.pool, b.page_table, b.seq_len, b.free_list, b.free_count, wl.n_q_heads, sz,
                        layers_per_call=2)
    comp.step_overlapped(b.q, b.win_indptr, b.tok_indptr, b.budget, wl.sm_scale, wl.causal)
    torch.cuda.synchronize()
    comp.check_status()
    assert torch.equal(a.pool.view(torch.int16), b.pool.view(torch.int16))
    assert torch.equal(a.page_table, b.page_table) and torch.equal(a.seq_len, b.seq_len)
    assert torch.equal(a.free_list, b.free_list) and torch.equal(a.free_count, b.free_count)


def test_step_host_matches_device_step():
    """actkv_step_host (host buffers in, host results out) gives what the per-stage calls give."""
    wl = synth.Workload("host", 3, 2, 4, [900, 333, 500], [16, 8, 32], [250, 100, 125],
                        table_style="fragmented", seed=14, poison_tail=True)
    a = synth.generate(wl, DEV)
    b = synth.generate(wl, DEV)
    _full_check(a)
    comp = H.Compressor(b.pool, b.page_table, b.seq_len, b.free_list, b.free_count, wl.n_q_heads, H.sizes_of(b),
                        layers_per_call=2)
    runner = H.HostStepRunner(comp, b.q, b.win_indptr, b.tok_indptr, b.budget, wl.sm_scale, wl.causal)
    # scribble over the device copies: the call must bring everything from the host buffers
    b.page_table.fill_(-7)
    b.seq_len.zero_()
    out = runner.run()
    assert out["st"].tolist()[0] == 0
    assert torch.equal(out["pt"], a.page_table.cpu()) and torch.equal(out["sl"], a.seq_len.cpu())
    assert int(out["fc"]) == int(a.free_count.cpu())
    fc = int(out["fc"])
    assert torch.equal(out["fl"][:fc], a.free_list.cpu()[:fc])
    assert out["bud"].tolist() == wl.budgets
    assert torch.equal(a.pool.view(torch.int16), b.pool.view(torch.int16))
    assert runner.h2d_bytes > b.q.numel() * 2 and runner.d2h_bytes > 0


def test_config1_all_units_and_planted_keys():
    inst = synth.generate(synth.config1(), DEV)
    res = _full_check(inst)
    comp = res["comp"]
    sel = comp.sel_idx.cpu().numpy()
    planted = set(inst.planted[0].tolist())
    assert len(planted) == 82
    for o in range(sel.shape[0]):
        assert planted <= set(sel[o, :1024].tolist())


def test_window_rows_at_tensor_tile_sizes():
    """window x group = 128 .. 512 rows (multiples and non-multiples of the 128-row tile)."""
    for W, G in [(32, 4), (64, 8), (33, 4), (96, 4), (20, 8)]:
        wl = synth.Workload("rows", 1, 2, G, [700, 257], [W, max(1, W // 2)], [200, 64], table_style="permutation",
                            seed=W * 10 + G, poison_tail=True)
        _full_check(synth.generate(wl, DEV))


@pytest.mark.parametrize("causal", [False, True])
def test_row_counts_at_every_column_group_boundary(causal):
    """The pooled-score epilogue reads an accumulator in 32-column groups, 64 and 128 at a time, and its two
    warpgroups take alternate jobs: one more row than every multiple of 32 between 128 and 512 (G = 1, so
    the window is the row count), a first request with an even and a second with an odd number of key
    tiles, ragged last tiles."""
    for W in [129, 161, 193, 225, 257, 289, 321, 353, 385, 417, 449, 481]:
        wl = synth.Workload("cg", 1, 2, 1, [128 * 10 + 37, 128 * 5 - 20], [W, W - 64], [300, 150], table_style="permutation",
                            causal=causal, seed=W, poison_tail=True)
        _full_check(synth.generate(wl, DEV))


@pytest.mark.parametrize("causal", [False, True])
def test_window_rows_above_one_cta(causal):
    """window x group above 512 rows: the score kernels take the rows in groups of 512 (whole action
    tokens); second group full, partial, and absent for the request with the short window."""
    for W, G in [(64, 16), (100, 8), (130, 4), (40, 32)]:
        wl = synth.Workload("rows+", 1, 2, G, [900, 300], [W, max(1, W // 3)], [300, 80], table_style="permutation",
                            causal=causal, seed=W * 7 + G, poison_tail=True)
        _full_check(synth.generate(wl, DEV))


@pytest.mark.parametrize("causal", [False, True])
def test_head_dim_64_on_the_tensor_core_path(causal):
    """head_dim 64 with 16-token pages: a K tile is one 64-dim half, four MMAs per accumulator."""
    for W, G in [(32, 4), (64, 8), (33, 2), (40, 16)]:
        wl = synth.Workload("d64", 2, 2, G, [1000, 300], [W, max(1, W // 2)], [260, 90], head_dim=64,
                            table_style="fragmented", causal=causal, seed=W * 3 + G, poison_tail=True)
        _full_check(synth.generate(wl, DEV))


@pytest.mark.parametrize("page", [32, 64, 128])
def test_larger_pages_on_the_tensor_core_path(page):
    """Pages of 32, 64 and 128 tokens: a key tile is 4, 2 or 1 TMA boxes per 64-dim half."""
    for head_dim, causal in [(128, False), (64, True)]:
        wl = synth.Workload("pages", 2, 2, 4, [1000, 333, 130], [32, 16, 20], [250, 100, 40], head_dim=head_dim,
                            page_size=page, table_style="fragmented", causal=causal, seed=page + head_dim,
                            poison_tail=True)
        _full_check(synth.generate(wl, DEV))


@pytest.mark.parametrize("causal", [False, True])
def test_group_sizes_that_are_not_powers_of_two(causal):
    """G = 3, 5, 6, 7 query heads per KV head on the tensor-core path: the pooled-score pass pads a group to
    the next power of two with rows that drop out of the max; the last group's padding reads past the last
    query head."""
    for W, G in [(32, 3), (24, 5), (100, 6), (40, 7)]:
        wl = synth.Workload("odd-g", 2, 2, G, [900, 300], [W, max(1, W // 3)], [300, 80], table_style="fragmented",
                            causal=causal, seed=W * 5 + G, poison_tail=True)
        _full_check(synth.generate(wl, DEV))


def test_new_shapes_really_take_the_tensor_core_path():
    """The library picks the path by itself and says which (actkv_score_path): the shapes that are meant to
    run on tensor cores do, shapes outside them (head_dim 96, pages of 8 tokens, fewer than 64 rows) take the
    FMA kernels."""
    from paper_2609_31395_b200 import binding as B
    shapes = [(dict(G=7), 1), (dict(G=4, head_dim=64), 1), (dict(G=4, page_size=64), 1), (dict(G=16, windows=[64, 20]), 1),
              (dict(G=4, head_dim=96), 0), (dict(G=4, page_size=8), 0), (dict(G=2, windows=[16, 8]), 0)]
    for kw, want in shapes:
        G = kw.pop("G")
        windows = kw.pop("windows", [32, 16])
        wl = synth.Workload("path", 1, 2, G, [700, 257], windows, [200, 64], table_style="permutation", seed=31,
                            poison_tail=True, **kw)
        inst = synth.generate(wl, DEV)
        got = B.actkv_score_path(B.pool_desc(inst.pool), wl.n_q_heads, max(windows), wl.sm_scale, inst.q)
        assert got == want, (kw, G, windows, got)
        _full_check(inst)


def test_head_major_pool_layout():
    """A pool stored [layer][K/V][page][head][slot][dim] (HND pages), described to the library by its
    strides alone: score (FMA path and tensor-core path), select and compaction give the same results as
    for the oracle's logical view."""
    small = _small(G=4, seed=21, head_dim=64, page=8)                 # FMA path
    rows = synth.Workload("hnd", 2, 2, 8, [1100, 257], [48, 17], [300, 64], table_style="fragmented", seed=22,
                          poison_tail=True)                          # tensor-core path (384 rows)
    for wl in (small, rows):
        inst = synth.generate(wl, DEV)
        hnd = inst.pool.permute(0, 1, 2, 4, 3, 5).contiguous()      # physical [NL, 2, pages, Hkv, P, D]
        inst.pool = hnd.permute(0, 1, 2, 4, 3, 5)                    # logical [NL, 2, pages, P, Hkv, D], HND strides
        assert inst.pool.stride(4) == wl.page_size * wl.head_dim and inst.pool.stride(3) == wl.head_dim
        _full_check(inst)


def test_every_other_layer_as_a_strided_view():
    """A model that interleaves sliding-window layers (bounded caches the method leaves alone) with
    full-attention layers: the full-attention layers of one allocation are described to the library as a
    pool whose layer stride skips the others.  Results match the oracle's logical view and the skipped
    layers keep every bit."""
    for wl in (synth.Workload("gptoss", 3, 2, 8, [1500, 300], [16, 9], [400, 80], head_dim=64,
                              table_style="fragmented", seed=31, poison_tail=True),
               _small(G=4, seed=32)):
        inst = synth.generate(wl, DEV)
        shape = list(inst.pool.shape)
        shape[0] *= 2
        g = torch.Generator(device=DEV).manual_seed(99)
        big = torch.randn(shape, generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
        big[0::2] = inst.pool
        inst.pool = big[0::2]
        assert inst.pool.stride(0) == 2 * big[0].numel()
        others = big[1::2].clone()
        _full_check(inst)
        assert torch.equal(big[1::2].view(torch.int16), others.view(torch.int16))


def test_long_request_many_chunks():
    """More keys than one LSE chunk and several key tiles per CTA; ragged last page."""
    wl = synth.Workload("long", 1, 1, 4, [9000 + 7], [32], [2300], table_style="fragmented", seed=5, poison_tail=True)
    _full_check(synth.generate(wl, DEV))


def test_workspace_sized_for_a_layer_range_serves_calls_on_fewer_layers():
    """The LSE pass cuts a request into more chunks when a call has fewer units; the workspace of the
    whole range must hold those partials too, and the scores do not depend on the cut."""
    wl = synth.Workload("ws", 3, 1, 4, [20000 + 13], [32], [5000], table_style="fragmented", seed=6)
    inst = synth.generate(wl, DEV)
    sz = H.sizes_of(inst)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads, sz,
                        want_lse=True)
    comp.run_score(inst.q, inst.win_indptr, inst.tok_indptr, wl.sm_scale, wl.causal)
    torch.cuda.synchronize()
    whole, whole_lse = comp.score.clone(), comp.lse.clone()
    for l in range(3):
        comp.run_score(inst.q, inst.win_indptr, inst.tok_indptr, wl.sm_scale, wl.causal, l0=l, l1=l + 1)
        torch.cuda.synchronize()
        comp.check_status()
        assert (comp.lse[l] - whole_lse[l]).abs().max().item() < 1e-5
        assert torch.allclose(comp.score[0], whole[l], rtol=1e-4, atol=1e-9)


def test_logits_that_keep_growing_move_the_lse_reference():
    """Keys arranged so that every row's logits climb by hundreds of log2 units along the request: the
    LSE pass keeps no running maximum, so its reference must be moved again and again (and 2^x saturates
    in between).  Scores of the early keys underflow, the late ones carry the mass."""
    wl = synth.Workload("climb", 1, 2, 4, [3000, 700], [32, 32], [600, 200], table_style="fragmented", seed=11,
                        poison_tail=True)
    inst = synth.generate(wl, DEV)
    P, G = wl.page_size, wl.group
    win = inst.win_indptr.cpu().numpy()
    for r, L in enumerate(wl.seq_lens):
        pages = inst.page_table[r, : -(-L // P)].long()
        alpha = torch.linspace(-5.0, 40.0, L, device=DEV)
        for h in range(wl.n_kv_heads):
            qbar = inst.q[0, win[r]:win[r + 1], h * G:(h + 1) * G].float().mean(dim=(0, 1))       # [D]
            rows = (alpha[:, None] * qbar[None, :]).to(torch.bfloat16)                             # [L, D]
            pad = torch.zeros((len(pages) * P - L, rows.shape[1]), dtype=torch.bfloat16, device=DEV)
            inst.pool[0, 0, pages, :, h, :] = torch.cat([rows, pad]).view(len(pages), P, -1)
    out = _full_check(inst)
    lse = out["lse"]
    assert np.nanmax(lse) > 100.0                      # the rows really reached large logits


def test_duplicate_keys_make_exact_ties():
    """Duplicated key rows give bit-equal scores; the lower index must win at the threshold."""
    wl = synth.Workload("dups", 1, 2, 4, [512], [16], [100], table_style="permutation", seed=9, plant_frac=0.0)
    inst = synth.generate(wl, DEV)
    P = wl.page_size
    kflat = inst.pool[0, 0].view(-1, wl.n_kv_heads, wl.head_dim)
    pt = inst.page_table[0].to(torch.int64)
    j = torch.arange(512, device=DEV)
    slots = pt[j // P] * P + j % P
    kflat[slots[256:]] = kflat[slots[:256]]            # second half duplicates the first
    res = _full_check(inst)
    comp = res["comp"]
    ties = comp.ties.cpu().numpy().reshape(-1, 4)
    score = comp.score.cpu().numpy().reshape(-1, 512)
    assert np.array_equal(score[:, :256], score[:, 256:])
    # every unit: threshold value appears at j and j+256; only consistent counts are possible
    for u in range(ties.shape[0]):
        thr = ties[u, 0:1].view(np.float32)[0]
        assert ties[u, 3] == 100
        assert ties[u, 2] == int((score[u] == thr).sum()) and ties[u, 2] >= 2
        assert 1 <= ties[u, 1] <= ties[u, 2]


def test_budget_covers_length_is_noop_and_budget_zero_empties():
    wl = _small()
    wl.budgets = [5000, 333, 0, 17]
    inst = synth.generate(wl, DEV)
    before = inst.pool.clone()
    pt_before = inst.page_table.clone()
    fc_before = int(inst.free_count.cpu())
    res = _full_check(inst)
    assert torch.equal(before.view(torch.int16), inst.pool.view(torch.int16))      # nothing copied at all
    assert torch.equal(inst.page_table[0], pt_before[0]) and torch.equal(inst.page_table[1], pt_before[1])
    assert inst.seq_len.cpu().tolist() == [1000, 333, 0, 17]
    assert (inst.page_table[2] == -1).all()
    assert int(inst.free_count.cpu()) == fc_before + -(-130 // 16)


def test_free_list_short_modifies_nothing():
    inst = synth.generate(_small(), DEV)
    inst.free_count.fill_(3)
    before = inst.pool.clone()
    pt, sl, fl = inst.page_table.clone(), inst.seq_len.clone(), inst.free_list.clone()
    comp = U.run_step(inst)
    st = comp.status.cpu().tolist()
    assert st[0] == B.E_NOFREE
    assert torch.equal(before.view(torch.int16), inst.pool.view(torch.int16))
    assert torch.equal(pt, inst.page_table) and torch.equal(sl, inst.seq_len) and torch.equal(fl, inst.free_list)
    assert int(inst.free_count.cpu()) == 3


def test_bad_page_id_is_reported_not_trapped():
    inst = synth.generate(_small(), DEV)
    inst.page_table[1, 2] = 10**6
    before_pt = inst.page_table.clone()
    comp = U.run_step(inst)
    st = comp.status.cpu().tolist()
    assert st[0] == B.E_BADPAGE and st[1] == 1 and st[2] == 10**6
    assert torch.equal(before_pt, inst.page_table)           # compaction refused to run
    # the context is still usable
    assert torch.ones(4, device=DEV).sum().item() == 4.0


def test_host_argument_errors():
    inst = synth.generate(_small(), DEV)
    sz = H.sizes_of(inst)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count,
                        inst.wl.n_q_heads, sz)
    tiny = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.ActKVError) as e:
        B.actkv_score(comp.pd, comp.td, 0, 2, inst.q, inst.win_indptr, inst.wl.n_q_heads, None, 0.1, 0,
                      inst.tok_indptr, comp.score, None, sz.sum_win, sz.max_win, sz.sum_tok, sz.max_tok, tiny,
                      comp.status)
    assert e.value.code == B.E_WORKSPACE
    with pytest.raises(B.ActKVError) as e:
        B.actkv_score(comp.pd, comp.td, 0, 3, inst.q, inst.win_indptr, inst.wl.n_q_heads, None, 0.1, 0,
                      inst.tok_indptr, comp.score, None, sz.sum_win, sz.max_win, sz.sum_tok, sz.max_tok,
                      comp.ws_score, comp.status)
    assert e.value.code == B.E_INVALID
    with pytest.raises(B.ActKVError) as e:                   # 7 q-heads do not divide over 2 KV heads
        B.actkv_score(comp.pd, comp.td, 0, 2, inst.q, inst.win_indptr, 7, None, 0.1, 0,
                      inst.tok_indptr, comp.score, None, sz.sum_win, sz.max_win, sz.sum_tok, sz.max_tok,
                      comp.ws_score, comp.status)
    assert e.value.code == B.E_INVALID


def test_zero_window_is_reported():
    wl = _small()
    wl.windows = [8, 0, 16, 3]
    inst = synth.generate(wl, DEV)
    comp = U.run_step(inst)
    st = comp.status.cpu().tolist()
    assert st[0] == B.E_INVALID and st[1] == 1


def test_empty_request_is_skipped():
    wl = synth.Workload("empty", 1, 2, 4, [300, 0, 64], [8, 4, 8], [100, 10, 10], table_style="fragmented", seed=4)
    inst = synth.generate(wl, DEV)
    _full_check(inst)


def test_keep_mask_bitmap():
    inst = synth.generate(_small(), DEV)
    wl = inst.wl
    sz = H.sizes_of(inst)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads, sz,
                        want_mask=True)
    B.actkv_keep_indptr(inst.seq_len, inst.budget, wl.n_req, comp.keep_indptr)
    comp.run_score(inst.q, inst.win_indptr, inst.tok_indptr, wl.sm_scale, False)
    comp.run_select(inst.tok_indptr, inst.budget, wl.n_layers)
    torch.cuda.synchronize()
    mask = comp.mask.cpu().numpy().view(np.uint32)
    sel = comp.sel_idx.cpu().numpy()
    ki = comp.keep_indptr.cpu().numpy()
    tok = inst.tok_indptr.cpu().numpy()
    for o in range(mask.shape[0]):
        bitsv = np.unpackbits(mask[o].view(np.uint8), bitorder="little")[: tok[-1]]
        want = np.zeros(tok[-1], dtype=np.uint8)
        for r in range(wl.n_req):
            want[tok[r] + sel[o, ki[r]:ki[r + 1]]] = 1
        assert np.array_equal(bitsv, want)


def test_select_reports_a_budget_beyond_the_index_buffer_and_stores_nothing_past_it():
    """The budgets are device data (they may come straight from actkv_budget, which can scale them up); the host
    sized the index buffer from what it knew.  A unit whose list would pass the end of its row is reported as
    ACTKV_E_INVALID before anything is stored, and the guard words behind the buffer keep their pattern."""
    rng = np.random.default_rng(3)
    lens, R, n_outer = [300, 500], 2, 3
    tok = np.array([0, 300, 800], dtype=np.int32)
    sc = torch.from_numpy(rng.random((n_outer, 800)).astype(np.float32)).to(DEV)
    sized_for = [100, 120]                                   # what the host sized the buffer for
    actual = [100, 333]                                      # what the device-side budgets say
    sel_stride = sum(sized_for)
    buf = torch.full((n_outer * sel_stride + 64,), -99, dtype=torch.int32, device=DEV)
    d_budget = torch.tensor(actual, dtype=torch.int32, device=DEV)
    d_len = torch.tensor(lens, dtype=torch.int32, device=DEV)
    ki = torch.zeros(R + 1, dtype=torch.int32, device=DEV)
    status = torch.zeros(4, dtype=torch.int32, device=DEV)
    B.actkv_keep_indptr(d_len, d_budget, R, ki)
    ws = torch.empty(256, dtype=torch.uint8, device=DEV)
    B.actkv_select(sc, torch.from_numpy(tok).to(DEV), 800, d_budget, n_outer, R, ki, buf[: n_outer * sel_stride].view(n_outer, sel_stride),
                   sel_stride, None, None, ws, status)
    torch.cuda.synchronize()
    st = status.cpu().tolist()
    assert st[0] == B.E_INVALID and st[1] == 1 and st[2] == 333
    assert bool((buf[n_outer * sel_stride:] == -99).all())
    # the request that fits was either written whole or, once the error was seen, not at all; never past its row
    rows = buf[: n_outer * sel_stride].view(n_outer, sel_stride).cpu().numpy()
    assert (rows[:, 100:] == -99).all()


@pytest.mark.parametrize("lse_supplied", [False, True])
def test_step_device_is_the_step_in_one_call(lse_supplied):
    """actkv_step_device (inputs already in device memory, one asynchronous call) against the per-stage calls, with the
    budgets coming from the confidence monitor inside the call."""
    wl = synth.Workload("onecall", 5, 2, 8, [1500, 333, 700, 90], [32, 16, 24, 8], [400, 100, 200, 90],
                        table_style="fragmented", seed=15, poison_tail=True)
    R, T, V = wl.n_req, 70, 2048
    logits, ltok = synth.confidence_logits(R, T, V, seed=9, device=DEV)
    p = B.BudgetParams.paper_defaults()
    # reference: monitor, then the step with those budgets, stage by stage
    a = synth.generate(wl, DEV)
    hist, hlen = torch.zeros((R, 256), dtype=torch.float32, device=DEV), torch.zeros(R, dtype=torch.int32, device=DEV)
    bud_a = torch.zeros(R, dtype=torch.int32, device=DEV)
    st = torch.zeros(4, dtype=torch.int32, device=DEV)
    ws = torch.empty(B.actkv_budget_workspace_bytes(R * T, R, 256) + 256, dtype=torch.uint8, device=DEV)
    B.actkv_budget(logits, ltok, R * T, V, hist, hlen, 256, p, a.seq_len, a.budget, bud_a, None, R, ws, st)
    torch.cuda.synchronize()
    budgets = bud_a.cpu().tolist()
    sz = H.StepSizes(R, sum(wl.windows), max(wl.windows), sum(wl.seq_lens), max(wl.seq_lens),
                     sum(min(b, L) for b, L in zip(budgets, wl.seq_lens)), max(min(b, L) for b, L in zip(budgets, wl.seq_lens)))
    comp_a = H.Compressor(a.pool, a.page_table, a.seq_len, a.free_list, a.free_count, wl.n_q_heads, sz, want_lse=True)
    comp_a.step(a.q, a.win_indptr, a.tok_indptr, bud_a, wl.sm_scale, wl.causal)
    torch.cuda.synchronize()
    comp_a.check_status()
    # the same in one call, layer groups of two
    b = synth.generate(wl, DEV)
    comp_b = H.Compressor(b.pool, b.page_table, b.seq_len, b.free_list, b.free_count, wl.n_q_heads, sz, layers_per_call=2,
                          want_lse=True, lse_layers_per_call=wl.n_layers)
    runner = H.HostStepRunner(comp_b, b.q, b.win_indptr, b.tok_indptr, b.budget, wl.sm_scale, wl.causal, logits=logits,
                              logit_indptr=ltok, hist_cap=256, params=p)
    runner.stage_inputs()
    if lse_supplied:
        comp_b.lse.copy_(comp_a.lse)
    runner.run_device(lse_supplied=lse_supplied)
    torch.cuda.synchronize()
    comp_b.check_status()
    assert runner.d["bud"].cpu().tolist() == budgets
    assert torch.equal(a.pool.view(torch.int16), b.pool.view(torch.int16))
    assert torch.equal(a.page_table, b.page_table) and torch.equal(a.seq_len, b.seq_len)
    assert torch.equal(a.free_list, b.free_list) and torch.equal(a.free_count, b.free_count)
    assert torch.equal(comp_a.lse, comp_b.lse)
