"""Torch-side owner of the buffers one compression step needs, and the step itself.

`Compressor` allocates (once) the score / index / scratch buffers for a pool and its tables and
runs  [budget ->] score -> select -> compact  by calling the C-ABI entry points in order on one
stream.  All arithmetic of the path happens inside those calls; this file only sizes buffers
and passes pointers.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import torch

from . import binding as B


def _ws(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(256, int(nbytes)), dtype=torch.uint8, device=device)


@dataclass
class StepSizes:
    n_req: int
    sum_win: int
    max_win: int
    sum_tok: int
    max_tok: int
    sel_stride: int
    max_keep: int


class Compressor:
    """Buffers and call sequence of one score -> select -> compact step over a paged pool."""

    def __init__(self, pool: torch.Tensor, page_table, seq_len, free_list, free_count, n_q_heads: int,
                 sizes: StepSizes, layers_per_call: Optional[int] = None, want_lse: bool = False,
                 want_ties: bool = False, want_mask: bool = False):
        B.load()
        self.dev = pool.device
        self.pool = pool
        self.page_table, self.seq_len, self.free_list, self.free_count = page_table, seq_len, free_list, free_count
        self.pd = B.pool_desc(pool)
        self.td = B.tables_desc(page_table, seq_len, free_list, free_count)
        self.n_q_heads = n_q_heads
        self.sz = sizes
        NL, Hkv = self.pd.n_layers, self.pd.n_kv_heads
        self.lpc = NL if layers_per_call is None else max(1, min(NL, layers_per_call))
        s = sizes
        self.score = torch.empty((self.lpc, Hkv, s.sum_tok), dtype=torch.float32, device=self.dev)
        self.sel_idx = torch.empty((self.lpc * Hkv, s.sel_stride), dtype=torch.int32, device=self.dev)
        self.keep_indptr = torch.zeros(s.n_req + 1, dtype=torch.int32, device=self.dev)
        self.status = torch.zeros(4, dtype=torch.int32, device=self.dev)
        self.lse = torch.empty((NL, s.sum_win, n_q_heads), dtype=torch.float32, device=self.dev) if want_lse else None
        self.ties = torch.zeros((self.lpc * Hkv * s.n_req, 4), dtype=torch.int32, device=self.dev) if want_ties else None
        self.mask = (torch.zeros((self.lpc * Hkv, (s.sum_tok + 31) // 32), dtype=torch.int32, device=self.dev)
                     if want_mask else None)
        self.ws_score = _ws(B.actkv_score_workspace_bytes(self.pd, s.n_req, self.lpc, n_q_heads, s.sum_win, s.max_win,
                                                          s.max_tok), self.dev)
        self.ws_select = _ws(B.actkv_select_workspace_bytes(self.lpc * Hkv, s.n_req, s.max_tok), self.dev)
        self.ws_compact = _ws(B.actkv_compact_workspace_bytes(s.n_req, self.td.max_pages), self.dev)

    # -- single stages (whole layer range unless given) ------------------------------------------
    def run_score(self, q, win_indptr, tok_indptr, sm_scale, causal, l0=0, l1=None, lse_in=None, stream=None):
        l1 = self.pd.n_layers if l1 is None else l1
        s = self.sz
        assert l1 - l0 <= self.lpc
        lse_out = None if self.lse is None else self.lse[l0:l1]
        B.actkv_score(self.pd, self.td, l0, l1, q[l0:l1], win_indptr, self.n_q_heads,
                      None if lse_in is None else lse_in[l0:l1], sm_scale, causal, tok_indptr,
                      self.score[: l1 - l0], lse_out, s.sum_win, s.max_win, s.sum_tok, s.max_tok,
                      self.ws_score, self.status, stream)

    def run_select(self, tok_indptr, budget, n_layers_sub, stream=None):
        s = self.sz
        Hkv = self.pd.n_kv_heads
        B.actkv_select(self.score, tok_indptr, s.sum_tok, budget, n_layers_sub * Hkv, s.n_req, self.keep_indptr,
                       self.sel_idx, s.sel_stride, self.mask, self.ties, self.ws_select, self.status, stream)

    def run_compact(self, budget, l0=0, l1=None, stream=None):
        l1 = self.pd.n_layers if l1 is None else l1
        B.actkv_compact(self.pd, self.td, l0, l1, self.sel_idx, self.sz.sel_stride, self.keep_indptr, budget,
                        self.sz.max_keep, self.ws_compact, self.status, stream)

    # -- the whole step ---------------------------------------------------------------------------
    def run_lse(self, q, win_indptr, tok_indptr, sm_scale, causal, l0, l1, lse_out, stream=None):
        s = self.sz
        B.actkv_score_lse(self.pd, self.td, l0, l1, q[l0:l1], win_indptr, self.n_q_heads, sm_scale, causal,
                          tok_indptr, lse_out, s.sum_win, s.max_win, s.sum_tok, s.max_tok, self.ws_score,
                          self.status, stream)

    def step(self, q, win_indptr, tok_indptr, budget, sm_scale, causal, lse_in=None, stream=None, marks=None):
        """score -> select -> compact over all layers, `layers_per_call` layers at a time.
        Tables are rewritten by the last compact call; earlier calls see the old tables.
        `marks`: optional callable(name) invoked between stages (the benchmark records CUDA events
        there); with it the LSE pass and the pooled-score pass run as two calls so that each can be
        timed on its own.  Returns the number of kernels launched."""
        NL = self.pd.n_layers
        mark = marks if marks is not None else (lambda name: None)
        B.actkv_keep_indptr(self.seq_len, budget, self.sz.n_req, self.keep_indptr, stream)
        launches = 1
        for l0 in range(0, NL, self.lpc):
            l1 = min(NL, l0 + self.lpc)
            mark("begin")
            if marks is not None and lse_in is None:
                if self.lse is None:
                    self.lse = torch.empty((NL, self.sz.sum_win, self.n_q_heads), dtype=torch.float32, device=self.dev)
                self.run_lse(q, win_indptr, tok_indptr, sm_scale, causal, l0, l1, self.lse[l0:l1], stream)
                mark("lse")
                self.run_score(q, win_indptr, tok_indptr, sm_scale, causal, l0, l1, self.lse, stream)
            else:
                self.run_score(q, win_indptr, tok_indptr, sm_scale, causal, l0, l1, lse_in, stream)
            mark("score")
            self.run_select(tok_indptr, budget, l1 - l0, stream)
            mark("select")
            self.run_compact(budget, l0, l1, stream)
            mark("compact")
            launches += (3 if lse_in is None else 1) + 1 + 2 + (1 if l1 == NL else 0)
        return launches

    def check_status(self):
        st = self.status.cpu().tolist()
        if st[0] != 0:
            raise B.ActKVError(f"device status {st}", st[0])


def sizes_of(inst, sel_stride: Optional[int] = None) -> StepSizes:
    """StepSizes for a synth.Instance (host-known lengths)."""
    wl = inst.wl
    keep = [min(b, L) for b, L in zip(wl.budgets, wl.seq_lens)]
    return StepSizes(wl.n_req, sum(wl.windows), max(wl.windows), sum(wl.seq_lens), max(wl.seq_lens),
                     max(1, sum(keep)) if sel_stride is None else sel_stride, max(keep + [0]))
