"""Comparators shared by the GPU parity tests: CUDA path (through the C ABI) vs CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import actkv_oracle as O
from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import harness as H

SCORE_RTOL = 2e-3        # max relative error of a pooled score (fp32 accumulation from bf16 inputs)
SCORE_ATOL = 1e-30


def bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def oracle_tables(inst) -> O.Tables:
    return O.Tables(inst.page_table.cpu().numpy().copy(), inst.seq_len.cpu().numpy().copy(),
                    inst.free_list.cpu().numpy().copy(), int(inst.free_count.cpu()))


def max_rel(got: np.ndarray, want: np.ndarray) -> float:
    got = got.astype(np.float64)
    want = want.astype(np.float64)
    return float(np.max(np.abs(got - want) / np.maximum(np.abs(want), SCORE_ATOL))) if got.size else 0.0


def check_scores(inst, comp: H.Compressor, pool_before: np.ndarray, tables_before: O.Tables, units=None,
                 layers=None, lse_in=None):
    """GPU scores (comp.score, first slabs) against the oracle on `units` (default: all), on the
    pool and tables as they were BEFORE the step (compaction rewrites the tables)."""
    wl = inst.wl
    pool_b = pool_before
    q_b = bits(inst.q if layers is None else inst.q[layers])
    want, lse, tok = O.score(pool_b, tables_before.page_table, tables_before.seq_len, q_b,
                             inst.win_indptr.cpu().numpy(), wl.n_q_heads, wl.sm_scale, wl.causal,
                             layers=layers, lse_in=lse_in, units=units)
    got = comp.score[: want.shape[0]].cpu().numpy()
    mask = ~np.isnan(want)
    assert mask.any()
    assert np.isfinite(got[mask]).all()
    err = max_rel(got[mask], want[mask])
    assert err <= SCORE_RTOL, f"score max-rel {err:.3e}"
    return want, lse, tok, err


def check_select_exact(score_gpu: np.ndarray, tok, budgets, sel_idx: np.ndarray, keep_indptr: np.ndarray):
    """The GPU's index lists equal TopK of the GPU's own float32 scores (bit-exact rule: larger
    score first, lower index on ties, ascending output)."""
    n_outer = score_gpu.shape[0]
    for o in range(n_outer):
        for r in range(len(budgets)):
            want = O.select_unit(score_gpu[o, tok[r]:tok[r + 1]], budgets[r])
            got = sel_idx[o, keep_indptr[r]:keep_indptr[r + 1]]
            assert np.array_equal(got, want), f"unit ({o},{r})"


def check_select_vs_oracle_scores(score_oracle: np.ndarray, tok, budgets, sel_idx, keep_indptr, rtol=2 * SCORE_RTOL):
    """Index sets against TopK of the ORACLE's scores: identical except for entries whose oracle
    score lies within `rtol` of the oracle's n-th score; those are counted and returned."""
    n_ties = 0
    for o in range(score_oracle.shape[0]):
        for r in range(len(budgets)):
            sc = score_oracle[o, tok[r]:tok[r + 1]]
            if np.isnan(sc).any():
                continue
            want = set(O.select_unit(sc, budgets[r]).tolist())
            got = set(sel_idx[o, keep_indptr[r]:keep_indptr[r + 1]].tolist())
            if want == got:
                continue
            n = len(want)
            thr = np.sort(sc.astype(np.float64))[::-1][n - 1]
            for i in want ^ got:
                assert abs(sc[i] - thr) <= rtol * thr, f"unit ({o},{r}) index {i}: {sc[i]} vs n-th {thr}"
            n_ties += len(want ^ got)
    return n_ties


def check_compaction(inst, pool_before: np.ndarray, tables_before: O.Tables, sel_idx: np.ndarray,
                     keep_indptr: np.ndarray, budgets, layers=None):
    """Pool and tables after the GPU compaction against the oracle's compaction of the GPU's index
    lists: valid slots bit-exact, every byte outside the destination slots unchanged, tables,
    free list and free count bit-exact."""
    wl = inst.wl
    NL = pool_before.shape[0]
    Hkv, P = wl.n_kv_heads, wl.page_size
    layers = list(range(NL)) if layers is None else layers
    sel = [[[sel_idx[a * Hkv + h, keep_indptr[r]:keep_indptr[r + 1]] for r in range(wl.n_req)]
            for h in range(Hkv)] for a in range(len(layers))]
    want_pool, want_t = O.compact(pool_before, tables_before, sel, budgets, layers=layers)
    got_pool = bits(inst.pool)
    got_pt = inst.page_table.cpu().numpy()
    got_sl = inst.seq_len.cpu().numpy()
    got_fl = inst.free_list.cpu().numpy()
    got_fc = int(inst.free_count.cpu())
    assert np.array_equal(got_pt, want_t.page_table)
    assert np.array_equal(got_sl, want_t.seq_len)
    assert got_fc == want_t.free_count
    assert np.array_equal(got_fl[:got_fc], want_t.free_list[:got_fc])
    # the oracle writes exactly the destination slots and nothing else, so whole-pool equality
    # checks both "valid slots equal" and "nothing else changed"
    assert np.array_equal(got_pool, want_pool)
    return want_pool, want_t


def run_step(inst, lse_in=None, layers_per_call=None, sel_stride=None, want_lse=True):
    wl = inst.wl
    sz = H.sizes_of(inst, sel_stride)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads, sz,
                        layers_per_call=layers_per_call, want_lse=want_lse, want_ties=True)
    comp.step(inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, wl.sm_scale, wl.causal, lse_in=lse_in)
    torch.cuda.synchronize()
    return comp
