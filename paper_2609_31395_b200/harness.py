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
                 want_ties: bool = False, want_mask: bool = False, lse_layers_per_call: Optional[int] = None):
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
        # layers per call of an LSE pass of its own (step_pipelined): it needs no score or index buffer, so it may
        # cover more layers than the other passes
        self.lse_lpc = self.lpc if lse_layers_per_call is None else max(self.lpc, min(NL, lse_layers_per_call))
        s = sizes
        self.score = torch.empty((self.lpc, Hkv, s.sum_tok), dtype=torch.float32, device=self.dev)
        self.sel_idx = torch.empty((self.lpc * Hkv, s.sel_stride), dtype=torch.int32, device=self.dev)
        self.keep_indptr = torch.zeros(s.n_req + 1, dtype=torch.int32, device=self.dev)
        self.status = torch.zeros(4, dtype=torch.int32, device=self.dev)
        self.lse = torch.empty((NL, s.sum_win, n_q_heads), dtype=torch.float32, device=self.dev) if want_lse else None
        self.ties = torch.zeros((self.lpc * Hkv * s.n_req, 4), dtype=torch.int32, device=self.dev) if want_ties else None
        self.mask = (torch.zeros((self.lpc * Hkv, (s.sum_tok + 31) // 32), dtype=torch.int32, device=self.dev)
                     if want_mask else None)
        self.ws_score = _ws(B.actkv_score_workspace_bytes(self.pd, s.n_req, self.lse_lpc, n_q_heads, s.sum_win, s.max_win,
                                                          s.max_tok), self.dev)
        self.ws_select = _ws(B.actkv_select_workspace_bytes(self.lpc * Hkv, s.n_req, s.max_tok), self.dev)
        # (sized for the pipelined step as well: room for the resolved sources of one layer group)
        self.ws_compact = _ws(max(B.actkv_compact_workspace_bytes(s.n_req, self.td.max_pages),
                                  B.actkv_compact_deferred_workspace_bytes(self.pd, s.n_req, self.td.max_pages, self.lpc,
                                                                           s.max_keep),
                                  B.actkv_compact_inplace_deferred_workspace_bytes(self.pd, s.n_req, self.lpc, s.max_keep)),
                              self.dev)

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

    def run_keepscore(self, lrfu: "LrfuState", tok_indptr, l0, l1, stream=None):
        """Turns the pooled scores of layers [l0, l1) into ranking keys (keep-scores, protected prefix
        lifted) and updates the persistent keep-scores of those layers."""
        Hkv, s = self.pd.n_kv_heads, self.sz
        hit = None if lrfu.hit_mask is None else lrfu.hit_mask[l0 * Hkv:l1 * Hkv]
        B.actkv_keepscore(self.score[: l1 - l0], tok_indptr, s.sum_tok, (l1 - l0) * Hkv, s.n_req, lrfu.top_p, lrfu.lam,
                          lrfu.n_protect, lrfu.keep_score[l0 * Hkv:l1 * Hkv], hit, self.status, stream)

    def run_keepscore_select(self, lrfu: "LrfuState", tok_indptr, budget, l0, l1, stream=None):
        """Keep-score update and TopK of layers [l0, l1) in one launch (actkv_keepscore_select)."""
        Hkv, s = self.pd.n_kv_heads, self.sz
        hit = None if lrfu.hit_mask is None else lrfu.hit_mask[l0 * Hkv:l1 * Hkv]
        B.actkv_keepscore_select(self.score[: l1 - l0], tok_indptr, s.sum_tok, s.max_tok, (l1 - l0) * Hkv, s.n_req,
                                 lrfu.top_p, lrfu.lam, lrfu.n_protect, lrfu.keep_score[l0 * Hkv:l1 * Hkv], hit, budget,
                                 self.keep_indptr, self.sel_idx, s.sel_stride, self.mask, self.ties, self.status, stream)

    def run_gather_ks(self, lrfu: "LrfuState", tok_indptr, l0, l1, stream=None, idx=None):
        """Keep-scores of the survivors of layers [l0, l1), packed like the index lists (`idx`: the
        lists to follow, default the ascending ones; after an in-place compaction its new order)."""
        Hkv, s = self.pd.n_kv_heads, self.sz
        B.actkv_gather_f32(lrfu.keep_score[l0 * Hkv:l1 * Hkv], s.sum_tok, tok_indptr,
                           self.sel_idx if idx is None else idx, s.sel_stride,
                           self.keep_indptr, (l1 - l0) * Hkv, s.n_req, s.sel_stride,
                           lrfu.kept[l0 * Hkv:l1 * Hkv], s.sel_stride, stream)

    def run_compact_inplace(self, budget, l0=0, l1=None, stream=None, want_order=True):
        """In-place tail compaction (Algorithm 4) of layers [l0, l1); `self.new_order` then holds, per
        unit, the original token index at every new logical slot."""
        l1 = self.pd.n_layers if l1 is None else l1
        if want_order and getattr(self, "new_order", None) is None:
            self.new_order = torch.empty_like(self.sel_idx)
        B.actkv_compact_inplace(self.pd, self.td, l0, l1, self.sel_idx, self.sz.sel_stride, self.keep_indptr, budget,
                                self.sz.max_keep, self.new_order if want_order else None, self.status, stream)

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

    def step(self, q, win_indptr, tok_indptr, budget, sm_scale, causal, lse_in=None, stream=None, marks=None,
             lrfu: Optional["LrfuState"] = None, inplace: bool = False, fused_lrfu: bool = True):
        """score -> select -> compact over all layers, `layers_per_call` layers at a time.
        Tables are rewritten by the last compact call; earlier calls see the old tables.
        `lrfu`: rank by the attention-aware LRFU keep-score instead of the raw pooled score
        (score -> keepscore + select in one launch, or as two with fused_lrfu=False -> gather keep-scores -> compact).
        `inplace`: compact into the tail blocks of each request (Algorithm 4) instead of fresh pages.
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
            if lrfu is not None and fused_lrfu:
                self.run_keepscore_select(lrfu, tok_indptr, budget, l0, l1, stream)
                mark("keepscore")
            else:
                if lrfu is not None:
                    self.run_keepscore(lrfu, tok_indptr, l0, l1, stream)
                    mark("keepscore")
                self.run_select(tok_indptr, budget, l1 - l0, stream)
            if lrfu is not None and not inplace:
                self.run_gather_ks(lrfu, tok_indptr, l0, l1, stream)
            mark("select")
            if inplace:
                self.run_compact_inplace(budget, l0, l1, stream, want_order=lrfu is not None)
                if lrfu is not None:
                    self.run_gather_ks(lrfu, tok_indptr, l0, l1, stream, idx=self.new_order)
            else:
                self.run_compact(budget, l0, l1, stream)
            mark("compact")
            launches += (3 if lse_in is None else 1) + 1 + (1 if inplace else 2) + (1 if l1 == NL else 0)
            launches += 2 if lrfu is not None else 0
        return launches

    def step_pipelined(self, q, win_indptr, tok_indptr, budget, sm_scale, causal, lse_in=None, stream=None, marks=None,
                       groups=None, stats=None, inplace=False, lrfu: Optional["LrfuState"] = None):
        """score -> select -> compact over all layers with the copies of layer group g running inside the
        score kernels of group g+1 (actkv_compact_begin / actkv_score_overlap / actkv_compact_end), all on one
        stream.  `groups`: list of (l0, l1) layer ranges, each at most `layers_per_call` long (default: equal
        groups of `layers_per_call`); the copies of the last group are not hidden, so a short last group
        exposes less.  Results are those of step().  inplace: Algorithm 4's in-place compaction instead of fresh
        pages (actkv_compact_inplace_begin / _end).  lrfu (fresh-page form only): rank by the LRFU keep-score, as
        step() does.  Returns the number of kernels launched."""
        assert lrfu is None or not inplace
        NL, Hkv, s = self.pd.n_layers, self.pd.n_kv_heads, self.sz
        if groups is None:
            groups = [(l0, min(NL, l0 + self.lpc)) for l0 in range(0, NL, self.lpc)]
        assert groups[0][0] == 0 and groups[-1][1] == NL and all(a[1] == b[0] for a, b in zip(groups, groups[1:]))
        assert all(0 < l1 - l0 <= self.lpc for l0, l1 in groups)
        mark = marks if marks is not None else (lambda name: None)
        B.actkv_keep_indptr(self.seq_len, budget, s.n_req, self.keep_indptr, stream)
        launches = 1
        prev = None
        done = []               # groups whose statistics have been written to `stats` ([n_groups, 2] int32, optional)
        if lse_in is None and (marks is not None or self.lse_lpc > self.lpc):
            # the LSE pass of all layers first, in calls of its own (as long as the workspace allows: fewer, larger
            # launches), then the pooled-score passes, which carry the copies
            if self.lse is None:
                self.lse = torch.empty((NL, s.sum_win, self.n_q_heads), dtype=torch.float32, device=self.dev)
            for l0 in range(0, NL, self.lse_lpc):
                l1 = min(NL, l0 + self.lse_lpc)
                mark("begin")
                self.run_lse(q, win_indptr, tok_indptr, sm_scale, causal, l0, l1, self.lse[l0:l1], stream)
                mark("lse")
                launches += 2
            lse_in = self.lse
        for l0, l1 in groups:
            mark("begin")
            lse_g = None if lse_in is None else lse_in[l0:l1]
            lse_out = None if (self.lse is None or lse_in is self.lse) else self.lse[l0:l1]
            B.actkv_score_overlap(self.pd, self.td, l0, l1, q[l0:l1], win_indptr, self.n_q_heads, lse_g, sm_scale, causal,
                                  tok_indptr, self.score[: l1 - l0], lse_out, s.sum_win, s.max_win, s.sum_tok, s.max_tok,
                                  self.ws_score, None if prev is None else self.ws_compact, self.status, stream)
            mark("score")
            if prev is not None:
                if stats is not None:
                    B.actkv_compact_stats(self.ws_compact, stats[len(done)], stream)
                    done.append(prev)
                    launches += 1
                launches += 1                       # the drain kernel
                if inplace:
                    B.actkv_compact_inplace_end(self.pd, self.td, prev[0], prev[1], self.sel_idx, s.sel_stride,
                                                self.keep_indptr, budget, s.max_keep, None, self.ws_compact, self.status,
                                                stream)
                else:
                    B.actkv_compact_end(self.pd, self.td, prev[0], prev[1], self.sel_idx, s.sel_stride, self.keep_indptr,
                                        budget, s.max_keep, self.ws_compact, self.status, stream)
                mark("compact")
            if lrfu is not None:
                self.run_keepscore_select(lrfu, tok_indptr, budget, l0, l1, stream)
                mark("keepscore")
                self.run_gather_ks(lrfu, tok_indptr, l0, l1, stream)
                launches += 1
            else:
                self.run_select(tok_indptr, budget, l1 - l0, stream)
            mark("select")
            launches += (3 if lse_in is None else 1) + 1      # score kernels, select
            if l1 == NL:
                # nothing follows the last group that could carry its copies: the one-launch copy of actkv_compact
                # (a CTA per destination page) is a little faster than draining a queue
                if inplace:
                    B.actkv_compact_inplace(self.pd, self.td, l0, l1, self.sel_idx, s.sel_stride, self.keep_indptr, budget,
                                            s.max_keep, None, self.status, stream)
                    mark("compact")
                    return launches + 2             # copy, finalize
                self.run_compact(budget, l0, l1, stream)
                mark("compact")
                return launches + 3                 # plan, copy, finalize
            launches += 2                           # plan (or the job record when the plan is reused), resolve
            if inplace:
                B.actkv_compact_inplace_begin(self.pd, self.td, l0, l1, self.sel_idx, s.sel_stride, self.keep_indptr,
                                              budget, s.max_keep, None, self.ws_compact, self.status, stream)
                prev = (l0, l1)
                continue
            B.actkv_compact_begin(self.pd, self.td, l0, l1, self.sel_idx, s.sel_stride, self.keep_indptr, budget,
                                  s.max_keep, self.ws_compact, self.status, stream, reuse_plan=prev is not None)
            prev = (l0, l1)
        return launches

    def step_overlapped(self, q, win_indptr, tok_indptr, budget, sm_scale, causal, lse_in=None, marks=None):
        """The same step with select + compact of layer group g running on a second stream while
        the score kernels of group g+1 run on the current one (the score kernels are bound by the
        tensor / MUFU pipes, compaction by HBM).  Score and index buffers are double-buffered by
        group parity.  Tables are still rewritten only by the last compact call, so every score
        call reads the old tables; compaction writes fresh pages only.
        `marks`: optional callable(name, stream).  Returns the number of kernels launched."""
        NL, Hkv, s = self.pd.n_layers, self.pd.n_kv_heads, self.sz
        cur = torch.cuda.current_stream()
        if not hasattr(self, "_aux"):
            # The score kernels run on a high-priority stream, select + compact on a low-priority one: a
            # score CTA is placed whenever it fits, the others only ever take what a score CTA leaves over
            # on its SM (registers, shared memory), so they run beside the score kernels instead of in turns.
            self._main = torch.cuda.Stream(device=self.dev, priority=-1)
            self._aux = torch.cuda.Stream(device=self.dev, priority=0)
            self._score2 = [self.score, torch.empty_like(self.score)]
            self._sel2 = [self.sel_idx, torch.empty_like(self.sel_idx)]
            self._ev_score = [torch.cuda.Event(), torch.cuda.Event()]
            self._ev_sel = [torch.cuda.Event(), torch.cuda.Event()]
            self._ev_done = torch.cuda.Event()
            if self.lse is None and lse_in is None:
                self.lse = torch.empty((NL, s.sum_win, self.n_q_heads), dtype=torch.float32, device=self.dev)
        aux, main = self._aux, self._main
        main.wait_stream(cur)
        mark = marks if marks is not None else (lambda name, stream: None)
        B.actkv_keep_indptr(self.seq_len, budget, s.n_req, self.keep_indptr, main)
        launches = 1
        for gi, l0 in enumerate(range(0, NL, self.lpc)):
            l1 = min(NL, l0 + self.lpc)
            buf = gi & 1
            score, sel = self._score2[buf], self._sel2[buf]
            if gi >= 2:
                main.wait_event(self._ev_sel[buf])          # select of group gi-2 has read this score buffer
            mark("begin", main)
            if lse_in is None:
                self.run_lse(q, win_indptr, tok_indptr, sm_scale, causal, l0, l1, self.lse[l0:l1], main)
                mark("lse", main)
                lse = self.lse
            else:
                lse = lse_in
            B.actkv_score(self.pd, self.td, l0, l1, q[l0:l1], win_indptr, self.n_q_heads, lse[l0:l1], sm_scale,
                          causal, tok_indptr, score[: l1 - l0], None, s.sum_win, s.max_win, s.sum_tok, s.max_tok,
                          self.ws_score, self.status, main)
            mark("score", main)
            self._ev_score[buf].record(main)
            aux.wait_event(self._ev_score[buf])
            mark("begin_aux", aux)
            B.actkv_select(score, tok_indptr, s.sum_tok, budget, (l1 - l0) * Hkv, s.n_req, self.keep_indptr, sel,
                           s.sel_stride, None, None, self.ws_select, self.status, aux)
            self._ev_sel[buf].record(aux)
            mark("select", aux)
            B.actkv_compact(self.pd, self.td, l0, l1, sel, s.sel_stride, self.keep_indptr, budget, s.max_keep,
                            self.ws_compact, self.status, aux)
            mark("compact", aux)
            launches += (3 if lse_in is None else 1) + 1 + 2 + (1 if l1 == NL else 0)
        self._ev_done.record(aux)
        main.wait_event(self._ev_done)
        cur.wait_stream(main)
        return launches

    def check_status(self):
        st = self.status.cpu().tolist()
        if st[0] != 0:
            raise B.ActKVError(f"device status {st}", st[0])


class LrfuState:
    """Device buffers of the attention-aware LRFU policy (Section 5.1) for one pool: the persistent
    keep-scores KS [layers * KV heads, sum_tok] in the score layout, the survivors' keep-scores
    `kept` [layers * KV heads, sel_stride] in the index-list layout, and the policy constants."""

    def __init__(self, n_outer: int, sizes: StepSizes, device, top_p: float = 0.9, lam: float = 0.9,
                 n_protect: Optional[torch.Tensor] = None, want_hits: bool = False):
        self.top_p, self.lam, self.n_protect = float(top_p), float(lam), n_protect
        self.keep_score = torch.zeros((n_outer, sizes.sum_tok), dtype=torch.float32, device=device)
        self.kept = torch.zeros((n_outer, sizes.sel_stride), dtype=torch.float32, device=device)
        self.hit_mask = (torch.zeros((n_outer, (sizes.sum_tok + 31) // 32), dtype=torch.int32, device=device)
                         if want_hits else None)


def extend_keep_scores(ks_compact: torch.Tensor, keep_counts, new_seq_lens) -> torch.Tensor:
    """Keep-score array for the next round: per request the survivors' keep-scores (as gathered by
    actkv_gather_f32, packed by keep_indptr) followed by zeros for the tokens appended since
    (Algorithm 1 step 2: new entries enter with keep-score 0).  Buffer bookkeeping only."""
    n_outer = ks_compact.shape[0]
    out = torch.zeros((n_outer, int(sum(new_seq_lens))), dtype=torch.float32, device=ks_compact.device)
    src = dst = 0
    for n, L in zip(keep_counts, new_seq_lens):
        out[:, dst:dst + n] = ks_compact[:, src:src + n]
        src += n
        dst += L
    return out


class HostStepRunner:
    """Pinned host buffers + device staging for actkv_step_host, the host-buffer form of the step.

    `comp` supplies the device scratch (score, index lists, workspaces, status); this class adds the
    host side: pinned copies of the per-step inputs and pinned result buffers."""

    def __init__(self, comp: Compressor, q: torch.Tensor, win_indptr, tok_indptr, budget_in, sm_scale: float,
                 causal: bool, logits: Optional[torch.Tensor] = None, logit_indptr=None, hist_cap: int = 4096,
                 params: Optional[B.BudgetParams] = None):
        self.comp, self.params = comp, params
        dev, s, R = comp.dev, comp.sz, comp.sz.n_req
        pin = lambda t: t.detach().cpu().contiguous().pin_memory()
        self.h_in = {"q": pin(q), "win": pin(win_indptr), "tok": pin(tok_indptr), "bud": pin(budget_in),
                     "pt": pin(comp.page_table), "sl": pin(comp.seq_len), "fl": pin(comp.free_list),
                     "fc": pin(comp.free_count)}
        self.h_out = {"pt": torch.empty_like(self.h_in["pt"]).pin_memory(),
                      "sl": torch.empty_like(self.h_in["sl"]).pin_memory(),
                      "fl": torch.empty_like(self.h_in["fl"]).pin_memory(),
                      "fc": torch.empty(1, dtype=torch.int32).pin_memory(),
                      "bud": torch.empty(R, dtype=torch.int32).pin_memory(),
                      "st": torch.empty(4, dtype=torch.int32).pin_memory()}
        self.d = {"q": torch.empty_like(q), "win": torch.empty_like(win_indptr), "tok": torch.empty_like(tok_indptr),
                  "bud": torch.empty(R, dtype=torch.int32, device=dev)}
        if comp.lse is None:
            comp.lse = torch.empty((comp.pd.n_layers, s.sum_win, comp.n_q_heads), dtype=torch.float32, device=dev)
        n_rows = vocab = 0
        if logits is not None:
            n_rows, vocab = logits.shape
            self.h_in["lg"], self.h_in["lgi"] = pin(logits), pin(logit_indptr)
            self.d["lg"], self.d["lgi"] = torch.empty_like(logits), torch.empty_like(logit_indptr)
            self.d["hist"] = torch.zeros((R, hist_cap), dtype=torch.float32, device=dev)
            self.d["hlen"] = torch.zeros(R, dtype=torch.int32, device=dev)
            self.d["wsb"] = _ws(B.actkv_budget_workspace_bytes(n_rows, R, hist_cap), dev)
        io = B.HostStep()
        hp = lambda k: self.h_in[k].data_ptr() if k in self.h_in else None
        io.q_host, io.logits_host, io.win_indptr_host, io.tok_indptr_host = hp("q"), hp("lg"), hp("win"), hp("tok")
        io.logit_indptr_host, io.budget_in_host, io.page_table_host = hp("lgi"), hp("bud"), hp("pt")
        io.seq_len_host, io.free_list_host, io.free_count_host = hp("sl"), hp("fl"), hp("fc")
        io.page_table_out_host, io.seq_len_out_host = self.h_out["pt"].data_ptr(), self.h_out["sl"].data_ptr()
        io.free_list_out_host, io.free_count_out_host = self.h_out["fl"].data_ptr(), self.h_out["fc"].data_ptr()
        io.budget_out_host, io.status_out_host = self.h_out["bud"].data_ptr(), self.h_out["st"].data_ptr()
        io.n_q_heads, io.sum_win, io.max_win, io.sum_tok, io.max_tok = comp.n_q_heads, s.sum_win, s.max_win, s.sum_tok, s.max_tok
        io.n_rows, io.vocab, io.hist_cap, io.max_keep = n_rows, vocab, hist_cap, s.max_keep
        io.causal, io.layers_per_call, io.sm_scale, io.sel_stride = int(bool(causal)), comp.lpc, float(sm_scale), s.sel_stride
        dp = lambda k: self.d[k].data_ptr() if k in self.d else None
        io.q_dev, io.logits_dev, io.win_indptr_dev, io.tok_indptr_dev = dp("q"), dp("lg"), dp("win"), dp("tok")
        io.logit_indptr_dev, io.budget_dev, io.keep_indptr_dev = dp("lgi"), dp("bud"), comp.keep_indptr.data_ptr()
        io.conf_hist_dev, io.hist_len_dev, io.lse_dev = dp("hist"), dp("hlen"), comp.lse.data_ptr()
        io.score_dev, io.sel_idx_dev = comp.score.data_ptr(), comp.sel_idx.data_ptr()
        io.ws_budget, io.ws_budget_bytes = dp("wsb"), (self.d["wsb"].numel() if "wsb" in self.d else 0)
        io.ws_score, io.ws_score_bytes = comp.ws_score.data_ptr(), comp.ws_score.numel()
        io.ws_compact, io.ws_compact_bytes = comp.ws_compact.data_ptr(), comp.ws_compact.numel()
        io.status_dev = comp.status.data_ptr()
        self.io = io
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in self.h_in.values())
        self.d2h_bytes = sum(t.numel() * t.element_size() for t in self.h_out.values())

    def run(self, stream=None):
        if "hlen" in self.d:
            self.d["hlen"].zero_()
        B.actkv_step_host(self.comp.pd, self.comp.td, self.params, self.io, stream)
        return self.h_out

    def stage_inputs(self):
        """Puts the step's inputs into the device staging buffers (for run_device; tables are the caller's)."""
        for k in ("q", "win", "tok", "bud", "lg", "lgi"):
            if k in self.d:
                self.d[k].copy_(self.h_in[k], non_blocking=True)

    def run_device(self, lse_supplied=False, stream=None):
        """The whole step as ONE call on inputs already in device memory (actkv_step_device): asynchronous, no
        copies; results are in the caller's pool, tables, free list and `self.d["bud"]`."""
        B.actkv_step_device(self.comp.pd, self.comp.td, self.params, self.io, lse_supplied, stream)


def sizes_of(inst, sel_stride: Optional[int] = None) -> StepSizes:
    """StepSizes for a synth.Instance (host-known lengths)."""
    wl = inst.wl
    keep = [min(b, L) for b, L in zip(wl.budgets, wl.seq_lens)]
    return StepSizes(wl.n_req, sum(wl.windows), max(wl.windows), sum(wl.seq_lens), max(wl.seq_lens),
                     max(1, sum(keep)) if sel_stride is None else sel_stride, max(keep + [0]))
