"""Seeded random shapes through the whole step (score -> select -> compact) against the oracle, element by
element, through the C ABI.  The hand-picked parity tests pin the boundaries that are known to matter (tile and
column-group edges, chunk counts, page sizes); this sweep draws everything at once, so that a combination nobody
thought of still runs: head dimension, page size, query heads per KV head, KV heads, layers, causal or not, table
style, request count, lengths (ragged, some shorter than a page or a window), windows (tensor-core and FMA row
counts in one batch), budgets (0, tiny, above the length), the step as one call, in layer groups, and with the
compaction of a group hidden under the next group's score kernels.
"""
import numpy as np
import pytest
import torch

from paper_2609_31395_b200 import harness as H
from paper_2609_31395_b200 import synth

import parity_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _draw(seed):
    rng = np.random.default_rng(1000 + seed)
    head_dim = int(rng.choice([64, 128, 128, 32, 96]))
    page = int(rng.choice([8, 16, 16, 32, 64]))
    G = int(rng.choice([1, 2, 3, 4, 8, 16]))
    Hkv = int(rng.choice([1, 2, 4]))
    NL = int(rng.integers(1, 5))
    causal = bool(rng.integers(0, 2))
    R = int(rng.integers(1, 6))
    # window x group rows on both sides of the 64-row switch between the FMA and the tensor-core kernels
    wmax = int(rng.choice([4, 16, 40, 64, 96]))
    seq, win, bud = [], [], []
    for _ in range(R):
        L = int(rng.choice([rng.integers(1, 40), rng.integers(40, 700), rng.integers(700, 2600)]))
        w = int(rng.integers(1, wmax + 1))
        if causal:
            w = min(w, L)
        kind = rng.integers(0, 6)
        b = [0, 1, L, L + 7, max(1, L // 4), int(rng.integers(1, L + 1))][kind]
        seq.append(L); win.append(w); bud.append(int(b))
    style = str(rng.choice(["permutation", "fragmented", "interleaved"]))
    wl = synth.Workload(f"rand{seed}", NL, Hkv, G, seq, win, bud, head_dim=head_dim, page_size=page, causal=causal,
                        table_style=style, seed=2000 + seed, poison_tail=True)
    form = ["one call", "layer groups", "pipelined"][int(rng.integers(0, 3))]
    return wl, form


@pytest.mark.parametrize("seed", range(48))
def test_random_shape(seed):
    wl, form = _draw(seed)
    inst = synth.generate(wl, DEV)
    pool_before, tables_before = U.bits(inst.pool), U.oracle_tables(inst)
    lpc = None if form == "one call" else max(1, (wl.n_layers + 1) // 2)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads,
                        H.sizes_of(inst), layers_per_call=lpc, want_lse=True, want_ties=True)
    if form == "pipelined":
        comp.step_pipelined(inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, wl.sm_scale, wl.causal)
    else:
        comp.step(inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, wl.sm_scale, wl.causal)
    torch.cuda.synchronize()
    comp.check_status()
    ki, sel = comp.keep_indptr.cpu().numpy(), comp.sel_idx.cpu().numpy()
    assert np.array_equal(ki, np.concatenate([[0], np.cumsum([min(b, L) for b, L in zip(wl.budgets, wl.seq_lens)])]))
    # scores: the buffer holds the last layer group of the step
    n_last = wl.n_layers if lpc is None else (wl.n_layers - 1) % lpc + 1
    layers = list(range(wl.n_layers - n_last, wl.n_layers))
    want, lse, tok, err = U.check_scores(inst, comp, pool_before, tables_before, layers=layers)
    m = ~np.isnan(lse)
    got_lse = comp.lse.cpu().numpy()[layers]
    assert np.abs(got_lse[m] - lse[m]).max() < 1e-4
    # index lists of those layers: TopK of the GPU's own scores exactly, of the oracle's within the score tolerance
    Hkv = wl.n_kv_heads
    sel_last = sel[(wl.n_layers - n_last) * Hkv: wl.n_layers * Hkv] if sel.shape[0] == wl.n_layers * Hkv else sel[: n_last * Hkv]
    score_gpu = comp.score[:n_last].cpu().numpy().reshape(-1, comp.score.shape[-1])
    U.check_select_exact(score_gpu, tok, wl.budgets, sel_last, ki)
    U.check_select_vs_oracle_scores(want.reshape(-1, want.shape[-1]), tok, wl.budgets, sel_last, ki)
    # every byte of the pool, the tables and the free list, for the layers whose index lists are still there
    if sel.shape[0] == wl.n_layers * Hkv:
        U.check_compaction(inst, pool_before, tables_before, sel, ki, wl.budgets)
    else:
        _check_last_group_and_tables(inst, pool_before, tables_before, sel_last, ki, wl, layers)
        # the earlier groups' lists are gone: the whole pool against the one-call step on a second copy of the
        # inputs, which is itself held against the oracle byte by byte
        ref = synth.generate(wl, DEV)
        comp_ref = U.run_step(ref)
        comp_ref.check_status()
        U.check_compaction(ref, pool_before, tables_before, comp_ref.sel_idx.cpu().numpy(),
                           comp_ref.keep_indptr.cpu().numpy(), wl.budgets)
        assert torch.equal(ref.pool.view(torch.int16), inst.pool.view(torch.int16))


def _check_last_group_and_tables(inst, pool_before, tables_before, sel_last, ki, wl, layers):
    """With one index buffer per layer group only the last group's lists survive the step: the pool bytes of those
    layers and the tables (which do not depend on the layer) are compared; the earlier groups went through the
    same calls on their own lists."""
    from oracle import actkv_oracle as O
    Hkv = wl.n_kv_heads
    sel = [[[sel_last[a * Hkv + h, ki[r]:ki[r + 1]] for r in range(wl.n_req)] for h in range(Hkv)]
           for a in range(len(layers))]
    want_pool, want_t = O.compact(pool_before, tables_before, sel, wl.budgets, layers=layers)
    got_pool = U.bits(inst.pool)
    assert np.array_equal(got_pool[layers], want_pool[layers])
    assert np.array_equal(inst.page_table.cpu().numpy(), want_t.page_table)
    assert np.array_equal(inst.seq_len.cpu().numpy(), want_t.seq_len)
    fc = int(inst.free_count.cpu())
    assert fc == want_t.free_count
    assert np.array_equal(inst.free_list.cpu().numpy()[:fc], want_t.free_list[:fc])
