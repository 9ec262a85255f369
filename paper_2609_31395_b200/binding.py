"""ctypes binding of libactkv.so: the same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors (torch is used for device memory and streams, nothing else);
each wrapper checks dtype / device / contiguity, passes raw pointers and raises `ActKVError`
on a non-zero return code.  There is no fallback: a missing or unloadable library is an error.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libactkv.so")

OK, E_INVALID, E_WORKSPACE, E_CUDA, E_BADPAGE, E_NOFREE, E_BADINDEX, E_TIMEOUT = 0, -1, -2, -3, -4, -5, -6, -7
E_TOOBIG = -8
ERROR_NAMES = {E_INVALID: "ACTKV_E_INVALID", E_WORKSPACE: "ACTKV_E_WORKSPACE", E_CUDA: "ACTKV_E_CUDA",
               E_BADPAGE: "ACTKV_E_BADPAGE", E_NOFREE: "ACTKV_E_NOFREE", E_BADINDEX: "ACTKV_E_BADINDEX",
               E_TIMEOUT: "ACTKV_E_TIMEOUT", E_TOOBIG: "ACTKV_E_TOOBIG"}

EXPORTS = ["actkv_budget_workspace_bytes", "actkv_budget", "actkv_score_workspace_bytes", "actkv_score",
           "actkv_score_lse", "actkv_score_accumulate",
           "actkv_keep_indptr", "actkv_select_workspace_bytes", "actkv_select",
           "actkv_compact_workspace_bytes", "actkv_compact", "actkv_compact_noalloc",
           "actkv_compact_noalloc_max_bytes", "actkv_step_host", "actkv_step_device", "actkv_keepscore", "actkv_gather_f32",
           "actkv_compact_inplace", "actkv_score_path", "actkv_debug_inject_stall", "actkv_score_sliding", "actkv_keepscore_select",
           "actkv_compact_deferred_workspace_bytes", "actkv_compact_begin", "actkv_compact_end", "actkv_score_overlap", "actkv_compact_stats",
           "actkv_compact_inplace_deferred_workspace_bytes", "actkv_compact_inplace_begin", "actkv_compact_inplace_end",
           "actkv_version"]


class ActKVError(RuntimeError):
    def __init__(self, fn: str, code: int):
        super().__init__(f"{fn} returned {code} ({ERROR_NAMES.get(code, 'unknown')})")
        self.code = code


class PoolDesc(C.Structure):
    _fields_ = [("base", C.c_void_p), ("n_layers", C.c_int32), ("n_pages", C.c_int32), ("page_size", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("stride_layer", C.c_int64),
                ("stride_kv", C.c_int64), ("stride_page", C.c_int64), ("stride_slot", C.c_int64),
                ("stride_head", C.c_int64)]


class TablesDesc(C.Structure):
    _fields_ = [("n_req", C.c_int32), ("max_pages", C.c_int32), ("page_table", C.c_void_p),
                ("seq_len", C.c_void_p), ("free_list", C.c_void_p), ("free_count", C.c_void_p)]


class BudgetParams(C.Structure):
    _fields_ = [("k", C.c_int32), ("w", C.c_int32), ("s", C.c_int32), ("b_percent", C.c_double),
                ("scale_up", C.c_double), ("B_upper", C.c_int32), ("clamp_lo_ppm", C.c_int32),
                ("clamp_hi_ppm", C.c_int32)]

    @classmethod
    def paper_defaults(cls, clamp_lo_ppm: int = 0, clamp_hi_ppm: int = 0):
        return cls(20, 64, 8, 10.0, 1.75, 30000, clamp_lo_ppm, clamp_hi_ppm)


class TieReport(C.Structure):
    _fields_ = [("threshold", C.c_float), ("n_equal_kept", C.c_int32), ("n_equal_total", C.c_int32),
                ("n_keep", C.c_int32)]


class HostStep(C.Structure):
    """actkv_host_step_t: host inputs / outputs, sizes, device staging and scratch of actkv_step_host."""
    _fields_ = ([(n, C.c_void_p) for n in
                 ("q_host", "logits_host", "win_indptr_host", "tok_indptr_host", "logit_indptr_host", "budget_in_host",
                  "page_table_host", "seq_len_host", "free_list_host", "free_count_host",
                  "page_table_out_host", "seq_len_out_host", "free_list_out_host", "free_count_out_host",
                  "budget_out_host", "status_out_host")] +
                [(n, C.c_int32) for n in
                 ("n_q_heads", "sum_win", "max_win", "sum_tok", "max_tok", "n_rows", "vocab", "hist_cap", "max_keep",
                  "causal", "layers_per_call")] +
                [("sm_scale", C.c_float), ("sel_stride", C.c_int64)] +
                [(n, C.c_void_p) for n in
                 ("q_dev", "logits_dev", "win_indptr_dev", "tok_indptr_dev", "logit_indptr_dev", "budget_dev",
                  "keep_indptr_dev", "conf_hist_dev", "hist_len_dev", "lse_dev", "score_dev", "sel_idx_dev")] +
                [("ws_budget", C.c_void_p), ("ws_budget_bytes", C.c_size_t), ("ws_score", C.c_void_p),
                 ("ws_score_bytes", C.c_size_t), ("ws_compact", C.c_void_p), ("ws_compact_bytes", C.c_size_t),
                 ("status_dev", C.c_void_p)])


_lib = None


def load():
    """Open libactkv.so (building it first when nvcc is present and the sources are newer)."""
    global _lib
    if _lib is not None:
        return _lib
    try:
        from . import build as _build
        if os.path.exists(os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")):
            _build.build()
    except Exception:
        if not os.path.exists(LIB_PATH):
            raise
    if not os.path.exists(LIB_PATH):
        raise ActKVError("load: libactkv.so is missing; run __graft_entry__.build()", E_CUDA)
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t, C.c_float
    lib.actkv_version.restype = C.c_char_p
    lib.actkv_budget_workspace_bytes.restype = sz
    lib.actkv_budget_workspace_bytes.argtypes = [i32, i32, i32]
    lib.actkv_budget.restype = i32
    lib.actkv_budget.argtypes = [vp, vp, i32, i32, vp, vp, i32, C.POINTER(BudgetParams), vp, vp, vp, vp, i32,
                                 vp, sz, vp, vp]
    lib.actkv_score_workspace_bytes.restype = sz
    lib.actkv_score_workspace_bytes.argtypes = [C.POINTER(PoolDesc), i32, i32, i32, i32, i32, i32]
    lib.actkv_score.restype = i32
    lib.actkv_score.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, vp, i32, vp, f32, i32,
                                vp, vp, vp, i32, i32, i32, i32, vp, sz, vp, vp]
    lib.actkv_score_lse.restype = i32
    lib.actkv_score_lse.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, vp, i32, f32, i32,
                                    vp, vp, i32, i32, i32, i32, vp, sz, vp, vp]
    lib.actkv_score_accumulate.restype = i32
    lib.actkv_score_accumulate.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, vp, i32, vp, f32,
                                           i32, vp, vp, vp, i32, i32, i32, i32, vp, sz, vp, vp]
    lib.actkv_keep_indptr.restype = i32
    lib.actkv_keep_indptr.argtypes = [vp, vp, i32, vp, vp]
    lib.actkv_select_workspace_bytes.restype = sz
    lib.actkv_select_workspace_bytes.argtypes = [i32, i32, i32]
    lib.actkv_select.restype = i32
    lib.actkv_select.argtypes = [vp, vp, i32, vp, i32, i32, vp, vp, i64, vp, vp, vp, sz, vp, vp]
    lib.actkv_compact_workspace_bytes.restype = sz
    lib.actkv_compact_workspace_bytes.argtypes = [i32, i32]
    lib.actkv_compact.restype = i32
    lib.actkv_compact.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, i64, vp, vp, i32,
                                  vp, sz, vp, vp]
    lib.actkv_keepscore.restype = i32
    lib.actkv_keepscore.argtypes = [vp, vp, i32, i32, i32, f32, f32, vp, vp, vp, vp, vp]
    lib.actkv_compact_inplace.restype = i32
    lib.actkv_compact_inplace.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, i64, vp, vp, i32,
                                          vp, vp, vp]
    lib.actkv_compact_inplace_deferred_workspace_bytes.restype = sz
    lib.actkv_compact_inplace_deferred_workspace_bytes.argtypes = [C.POINTER(PoolDesc), i32, i32, i32]
    for fn in (lib.actkv_compact_inplace_begin, lib.actkv_compact_inplace_end):
        fn.restype = i32
        fn.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, i64, vp, vp, i32, vp, vp, sz, vp, vp]
    lib.actkv_gather_f32.restype = i32
    lib.actkv_gather_f32.argtypes = [vp, i64, vp, vp, i64, vp, i32, i32, i32, vp, i64, vp]
    lib.actkv_step_device.restype = i32
    lib.actkv_step_device.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), C.POINTER(BudgetParams),
                                      C.POINTER(HostStep), i32, vp]
    lib.actkv_step_host.restype = i32
    lib.actkv_step_host.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), C.POINTER(BudgetParams),
                                    C.POINTER(HostStep), vp]
    lib.actkv_compact_noalloc_max_bytes.restype = sz
    lib.actkv_compact_noalloc_max_bytes.argtypes = []
    lib.actkv_compact_noalloc.restype = i32
    lib.actkv_compact_noalloc.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, i64, vp, vp, i32,
                                          vp, vp]
    lib.actkv_compact_begin.restype = i32
    lib.actkv_compact_begin.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, i64, vp, vp, i32, i32, vp,
                                        sz, vp, vp]
    lib.actkv_compact_end.restype = i32
    lib.actkv_compact_end.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, i64, vp, vp, i32, vp, sz,
                                      vp, vp]
    lib.actkv_score_overlap.restype = i32
    lib.actkv_score_overlap.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, vp, i32, vp, f32, i32,
                                        vp, vp, vp, i32, i32, i32, i32, vp, sz, vp, vp, vp]
    lib.actkv_compact_deferred_workspace_bytes.restype = sz
    lib.actkv_compact_deferred_workspace_bytes.argtypes = [C.POINTER(PoolDesc), i32, i32, i32, i32]
    lib.actkv_compact_stats.restype = i32
    lib.actkv_compact_stats.argtypes = [vp, vp, vp]
    lib.actkv_keepscore_select.restype = i32
    lib.actkv_keepscore_select.argtypes = [vp, vp, i32, i32, i32, i32, f32, f32, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp, vp]
    lib.actkv_score_sliding.restype = i32
    lib.actkv_score_sliding.argtypes = [C.POINTER(PoolDesc), C.POINTER(TablesDesc), i32, i32, vp, vp, i32, vp, f32, i32,
                                        i32, vp, vp, vp, i32, i32, i32, i32, vp, sz, vp, vp]
    lib.actkv_score_path.restype = i32
    lib.actkv_score_path.argtypes = [C.POINTER(PoolDesc), i32, i32, f32, vp, i32]
    lib.actkv_debug_inject_stall.restype = i32
    lib.actkv_debug_inject_stall.argtypes = [i32, i32]
    _lib = lib
    return lib


# ---------------------------------------------------------------------------------------------
# marshalling helpers


def _ptr(t: Optional[torch.Tensor], dtype=None, name: str = "tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError(f"{name}: expected a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous tensor")
    return t.data_ptr()


def _stream(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _check(fn: str, rc: int):
    if rc != 0:
        raise ActKVError(fn, rc)


def pool_desc(pool: torch.Tensor) -> PoolDesc:
    """Descriptor of a bf16 pool tensor [n_layers, 2, n_pages, page_size, n_kv_heads, head_dim]
    (any strides with a contiguous head dimension)."""
    if pool.dtype != torch.bfloat16 or pool.dim() != 6 or pool.shape[1] != 2 or pool.stride(5) != 1:
        raise TypeError("pool: expected bf16 [NL, 2, n_pages, P, Hkv, D] with contiguous D")
    NL, _, n_pages, P, H, D = pool.shape
    st = pool.stride()
    return PoolDesc(pool.data_ptr(), NL, n_pages, P, H, D, st[0], st[1], st[2], st[3], st[4])


def tables_desc(page_table, seq_len, free_list, free_count) -> TablesDesc:
    R, max_pages = page_table.shape
    return TablesDesc(R, max_pages, _ptr(page_table, torch.int32, "page_table"), _ptr(seq_len, torch.int32, "seq_len"),
                      _ptr(free_list, torch.int32, "free_list"), _ptr(free_count, torch.int32, "free_count"))


# ---------------------------------------------------------------------------------------------
# the entry points


def actkv_version() -> str:
    return load().actkv_version().decode()


def actkv_budget_workspace_bytes(n_rows: int, n_req: int, hist_cap: int) -> int:
    return load().actkv_budget_workspace_bytes(n_rows, n_req, hist_cap)


def actkv_budget(logits, tok_indptr, n_rows, vocab, conf_hist, hist_len, hist_cap, params: BudgetParams,
                 seq_len, budget_in, budget_out, slope_out, n_req, ws, status, stream=None):
    rc = load().actkv_budget(_ptr(logits, torch.float32, "logits"), _ptr(tok_indptr, torch.int32, "tok_indptr"),
                             n_rows, vocab, _ptr(conf_hist, torch.float32, "conf_hist"),
                             _ptr(hist_len, torch.int32, "hist_len"), hist_cap, C.byref(params),
                             _ptr(seq_len, torch.int32, "seq_len"), _ptr(budget_in, torch.int32, "budget_in"),
                             _ptr(budget_out, torch.int32, "budget_out"), _ptr(slope_out, torch.float64, "slope_out"),
                             n_req, _ptr(ws, None, "ws"), ws.numel() * ws.element_size(),
                             _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_budget", rc)


def actkv_score_workspace_bytes(pool: PoolDesc, n_req, n_layers_sub, n_q_heads, sum_win, max_win, max_tok) -> int:
    return load().actkv_score_workspace_bytes(C.byref(pool), n_req, n_layers_sub, n_q_heads, sum_win, max_win, max_tok)


def actkv_score(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, q, win_indptr, n_q_heads, lse_in,
                sm_scale, causal, tok_indptr, score_out, lse_out, sum_win, max_win, sum_tok, max_tok, ws, status,
                stream=None):
    rc = load().actkv_score(C.byref(pool), C.byref(tables), layer_begin, layer_end, _ptr(q, torch.bfloat16, "q"),
                            _ptr(win_indptr, torch.int32, "win_indptr"), n_q_heads,
                            _ptr(lse_in, torch.float32, "lse_in"), float(sm_scale), int(bool(causal)),
                            _ptr(tok_indptr, torch.int32, "tok_indptr"), _ptr(score_out, torch.float32, "score_out"),
                            _ptr(lse_out, torch.float32, "lse_out"), sum_win, max_win, sum_tok, max_tok,
                            _ptr(ws, None, "ws"), ws.numel() * ws.element_size(),
                            _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_score", rc)


def actkv_score_overlap(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, q, win_indptr, n_q_heads, lse_in,
                        sm_scale, causal, tok_indptr, score_out, lse_out, sum_win, max_win, sum_tok, max_tok, ws,
                        pending_compact_ws, status, stream=None):
    rc = load().actkv_score_overlap(C.byref(pool), C.byref(tables), layer_begin, layer_end, _ptr(q, torch.bfloat16, "q"),
                                    _ptr(win_indptr, torch.int32, "win_indptr"), n_q_heads,
                                    _ptr(lse_in, torch.float32, "lse_in"), float(sm_scale), int(bool(causal)),
                                    _ptr(tok_indptr, torch.int32, "tok_indptr"),
                                    _ptr(score_out, torch.float32, "score_out"), _ptr(lse_out, torch.float32, "lse_out"),
                                    sum_win, max_win, sum_tok, max_tok, _ptr(ws, None, "ws"),
                                    ws.numel() * ws.element_size(), _ptr(pending_compact_ws, None, "pending_compact_ws"),
                                    _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_score_overlap", rc)


def actkv_compact_begin(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr,
                        budget, max_keep, ws, status, stream=None, reuse_plan=False):
    rc = load().actkv_compact_begin(C.byref(pool), C.byref(tables), layer_begin, layer_end,
                                    _ptr(sel_idx, torch.int32, "sel_idx"), sel_stride,
                                    _ptr(keep_indptr, torch.int32, "keep_indptr"), _ptr(budget, torch.int32, "budget"),
                                    max_keep, int(bool(reuse_plan)), _ptr(ws, None, "ws"), ws.numel() * ws.element_size(),
                                    _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_compact_begin", rc)


def actkv_compact_end(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr,
                      budget, max_keep, ws, status, stream=None):
    rc = load().actkv_compact_end(C.byref(pool), C.byref(tables), layer_begin, layer_end,
                                  _ptr(sel_idx, torch.int32, "sel_idx"), sel_stride,
                                  _ptr(keep_indptr, torch.int32, "keep_indptr"), _ptr(budget, torch.int32, "budget"),
                                  max_keep, _ptr(ws, None, "ws"), ws.numel() * ws.element_size(),
                                  _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_compact_end", rc)


def actkv_compact_deferred_workspace_bytes(pool: PoolDesc, n_req, max_pages, n_layers_sub, max_keep) -> int:
    return load().actkv_compact_deferred_workspace_bytes(C.byref(pool), n_req, max_pages, n_layers_sub, max_keep)


def actkv_compact_stats(ws, stats, stream=None):
    _check("actkv_compact_stats", load().actkv_compact_stats(_ptr(ws, None, "ws"), _ptr(stats, torch.int32, "stats"),
                                                             _stream(stream)))


def actkv_keepscore_select(score, tok_indptr, sum_tok, max_tok, n_outer, n_req, top_p, lam, n_protect, keep_score,
                           hit_mask, budget, keep_indptr, sel_idx, sel_stride, keep_mask, tie_report, status, stream=None):
    rc = load().actkv_keepscore_select(_ptr(score, torch.float32, "score"), _ptr(tok_indptr, torch.int32, "tok_indptr"),
                                       sum_tok, max_tok, n_outer, n_req, float(top_p), float(lam),
                                       _ptr(n_protect, torch.int32, "n_protect"),
                                       _ptr(keep_score, torch.float32, "keep_score"), _ptr(hit_mask, None, "hit_mask"),
                                       _ptr(budget, torch.int32, "budget"), _ptr(keep_indptr, torch.int32, "keep_indptr"),
                                       _ptr(sel_idx, torch.int32, "sel_idx"), sel_stride, _ptr(keep_mask, None, "keep_mask"),
                                       _ptr(tie_report, None, "tie_report"), _ptr(status, torch.int32, "status"),
                                       _stream(stream))
    _check("actkv_keepscore_select", rc)


def actkv_score_sliding(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, q, win_indptr, n_q_heads, lse_in,
                        sm_scale, causal, window_left, tok_indptr, score_out, lse_out, sum_win, max_win, sum_tok, max_tok,
                        ws, status, stream=None):
    rc = load().actkv_score_sliding(C.byref(pool), C.byref(tables), layer_begin, layer_end, _ptr(q, torch.bfloat16, "q"),
                                    _ptr(win_indptr, torch.int32, "win_indptr"), n_q_heads,
                                    _ptr(lse_in, torch.float32, "lse_in"), float(sm_scale), int(bool(causal)),
                                    int(window_left), _ptr(tok_indptr, torch.int32, "tok_indptr"),
                                    _ptr(score_out, torch.float32, "score_out"), _ptr(lse_out, torch.float32, "lse_out"),
                                    sum_win, max_win, sum_tok, max_tok, _ptr(ws, None, "ws"),
                                    ws.numel() * ws.element_size(), _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_score_sliding", rc)


def actkv_score_path(pool: PoolDesc, n_q_heads, max_win, sm_scale, q, streaming=False) -> int:
    """1: the tensor-core kernels would run, 0: the FMA kernels."""
    rc = load().actkv_score_path(C.byref(pool), n_q_heads, max_win, float(sm_scale), _ptr(q, torch.bfloat16, "q"),
                                 int(bool(streaming)))
    if rc < 0:
        raise ActKVError("actkv_score_path", rc)
    return rc


def actkv_debug_inject_stall(after_tile: int, wait_limit_us: int = 0):
    _check("actkv_debug_inject_stall", load().actkv_debug_inject_stall(int(after_tile), int(wait_limit_us)))


def actkv_score_lse(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, q, win_indptr, n_q_heads, sm_scale,
                    causal, tok_indptr, lse_out, sum_win, max_win, sum_tok, max_tok, ws, status, stream=None):
    rc = load().actkv_score_lse(C.byref(pool), C.byref(tables), layer_begin, layer_end, _ptr(q, torch.bfloat16, "q"),
                                _ptr(win_indptr, torch.int32, "win_indptr"), n_q_heads, float(sm_scale),
                                int(bool(causal)), _ptr(tok_indptr, torch.int32, "tok_indptr"),
                                _ptr(lse_out, torch.float32, "lse_out"), sum_win, max_win, sum_tok, max_tok,
                                _ptr(ws, None, "ws"), ws.numel() * ws.element_size(),
                                _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_score_lse", rc)


def actkv_score_accumulate(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, q, win_indptr, n_q_heads, lse_in,
                           sm_scale, causal, tok_indptr, acc_steps, score_io, sum_win, max_win, sum_tok, max_tok, ws,
                           status, stream=None):
    rc = load().actkv_score_accumulate(C.byref(pool), C.byref(tables), layer_begin, layer_end,
                                       _ptr(q, torch.bfloat16, "q"), _ptr(win_indptr, torch.int32, "win_indptr"),
                                       n_q_heads, _ptr(lse_in, torch.float32, "lse_in"), float(sm_scale),
                                       int(bool(causal)), _ptr(tok_indptr, torch.int32, "tok_indptr"),
                                       _ptr(acc_steps, torch.int32, "acc_steps"),
                                       _ptr(score_io, torch.float32, "score_io"), sum_win, max_win, sum_tok, max_tok,
                                       _ptr(ws, None, "ws"), ws.numel() * ws.element_size(),
                                       _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_score_accumulate", rc)


def actkv_keep_indptr(seq_len, budget, n_req, keep_indptr, stream=None):
    rc = load().actkv_keep_indptr(_ptr(seq_len, torch.int32, "seq_len"), _ptr(budget, torch.int32, "budget"), n_req,
                                  _ptr(keep_indptr, torch.int32, "keep_indptr"), _stream(stream))
    _check("actkv_keep_indptr", rc)


def actkv_select_workspace_bytes(n_outer, n_req, max_tok) -> int:
    return load().actkv_select_workspace_bytes(n_outer, n_req, max_tok)


def actkv_select(score, tok_indptr, sum_tok, budget, n_outer, n_req, keep_indptr, sel_idx, sel_stride, keep_mask,
                 tie_report, ws, status, stream=None):
    rc = load().actkv_select(_ptr(score, torch.float32, "score"), _ptr(tok_indptr, torch.int32, "tok_indptr"), sum_tok,
                             _ptr(budget, torch.int32, "budget"), n_outer, n_req,
                             _ptr(keep_indptr, torch.int32, "keep_indptr"), _ptr(sel_idx, torch.int32, "sel_idx"),
                             sel_stride, _ptr(keep_mask, torch.int32, "keep_mask"),
                             _ptr(tie_report, torch.int32, "tie_report"),
                             _ptr(ws, None, "ws"), 0 if ws is None else ws.numel() * ws.element_size(),
                             _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_select", rc)


def actkv_compact_workspace_bytes(n_req, max_pages) -> int:
    return load().actkv_compact_workspace_bytes(n_req, max_pages)


def actkv_compact(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr,
                  budget, max_keep, ws, status, stream=None):
    rc = load().actkv_compact(C.byref(pool), C.byref(tables), layer_begin, layer_end,
                              _ptr(sel_idx, torch.int32, "sel_idx"), sel_stride,
                              _ptr(keep_indptr, torch.int32, "keep_indptr"), _ptr(budget, torch.int32, "budget"),
                              max_keep, _ptr(ws, None, "ws"), ws.numel() * ws.element_size(),
                              _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_compact", rc)


def actkv_compact_inplace(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr,
                          budget, max_keep, new_order, status, stream=None):
    rc = load().actkv_compact_inplace(C.byref(pool), C.byref(tables), layer_begin, layer_end,
                                      _ptr(sel_idx, torch.int32, "sel_idx"), sel_stride,
                                      _ptr(keep_indptr, torch.int32, "keep_indptr"),
                                      _ptr(budget, torch.int32, "budget"), max_keep,
                                      _ptr(new_order, torch.int32, "new_order"),
                                      _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_compact_inplace", rc)


def actkv_compact_inplace_deferred_workspace_bytes(pool: PoolDesc, n_req, n_layers_sub, max_keep) -> int:
    return load().actkv_compact_inplace_deferred_workspace_bytes(C.byref(pool), n_req, n_layers_sub, max_keep)


def _inplace_deferred(fn_name, pool, tables, layer_begin, layer_end, sel_idx, sel_stride, keep_indptr, budget, max_keep,
                      new_order, ws, status, stream):
    rc = getattr(load(), fn_name)(C.byref(pool), C.byref(tables), layer_begin, layer_end,
                                  _ptr(sel_idx, torch.int32, "sel_idx"), sel_stride,
                                  _ptr(keep_indptr, torch.int32, "keep_indptr"), _ptr(budget, torch.int32, "budget"),
                                  max_keep, _ptr(new_order, torch.int32, "new_order"), _ptr(ws, None, "ws"),
                                  ws.numel() * ws.element_size(), _ptr(status, torch.int32, "status"), _stream(stream))
    _check(fn_name, rc)


def actkv_compact_inplace_begin(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, sel_idx, sel_stride,
                                keep_indptr, budget, max_keep, new_order, ws, status, stream=None):
    _inplace_deferred("actkv_compact_inplace_begin", pool, tables, layer_begin, layer_end, sel_idx, sel_stride,
                      keep_indptr, budget, max_keep, new_order, ws, status, stream)


def actkv_compact_inplace_end(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, sel_idx, sel_stride,
                              keep_indptr, budget, max_keep, new_order, ws, status, stream=None):
    _inplace_deferred("actkv_compact_inplace_end", pool, tables, layer_begin, layer_end, sel_idx, sel_stride,
                      keep_indptr, budget, max_keep, new_order, ws, status, stream)


def actkv_keepscore(score, tok_indptr, sum_tok, n_outer, n_req, top_p, lam, n_protect, keep_score, hit_mask, status,
                    stream=None):
    rc = load().actkv_keepscore(_ptr(score, torch.float32, "score"), _ptr(tok_indptr, torch.int32, "tok_indptr"),
                                sum_tok, n_outer, n_req, float(top_p), float(lam),
                                _ptr(n_protect, torch.int32, "n_protect"), _ptr(keep_score, torch.float32, "keep_score"),
                                _ptr(hit_mask, torch.int32, "hit_mask"), _ptr(status, torch.int32, "status"),
                                _stream(stream))
    _check("actkv_keepscore", rc)


def actkv_gather_f32(src, src_stride, tok_indptr, sel_idx, sel_stride, keep_indptr, n_outer, n_req, max_total_keep,
                     dst, dst_stride, stream=None):
    rc = load().actkv_gather_f32(_ptr(src, torch.float32, "src"), src_stride, _ptr(tok_indptr, torch.int32, "tok_indptr"),
                                 _ptr(sel_idx, torch.int32, "sel_idx"), sel_stride,
                                 _ptr(keep_indptr, torch.int32, "keep_indptr"), n_outer, n_req, max_total_keep,
                                 _ptr(dst, torch.float32, "dst"), dst_stride, _stream(stream))
    _check("actkv_gather_f32", rc)


def actkv_step_device(pool: PoolDesc, tables: TablesDesc, params: Optional[BudgetParams], io: HostStep, lse_supplied: bool,
                      stream=None):
    rc = load().actkv_step_device(C.byref(pool), C.byref(tables), None if params is None else C.byref(params),
                                  C.byref(io), int(bool(lse_supplied)), _stream(stream))
    _check("actkv_step_device", rc)


def actkv_step_host(pool: PoolDesc, tables: TablesDesc, params: Optional[BudgetParams], io: HostStep, stream=None):
    """One whole step with host-resident per-step inputs and outputs (synchronises `stream`)."""
    rc = load().actkv_step_host(C.byref(pool), C.byref(tables), None if params is None else C.byref(params),
                                C.byref(io), _stream(stream))
    _check("actkv_step_host", rc)


def actkv_compact_noalloc_max_bytes() -> int:
    return load().actkv_compact_noalloc_max_bytes()


def actkv_compact_noalloc(pool: PoolDesc, tables: TablesDesc, layer_begin, layer_end, sel_idx, sel_stride,
                          keep_indptr, budget, max_keep, status, stream=None):
    """actkv_compact for callers that cannot allocate the plan scratch: a serving engine that has
    handed all of HBM to its KV pool (cudaMalloc may fail, and it stalls the device), or a host
    without an allocator of its own.  The scratch is a fixed 1 MiB array inside the library, shared
    by every call on the device, so calls that overlap on the GPU race; tables larger than the
    array are refused with ACTKV_E_TOOBIG."""
    rc = load().actkv_compact_noalloc(C.byref(pool), C.byref(tables), layer_begin, layer_end,
                                      _ptr(sel_idx, torch.int32, "sel_idx"), sel_stride,
                                      _ptr(keep_indptr, torch.int32, "keep_indptr"),
                                      _ptr(budget, torch.int32, "budget"), max_keep,
                                      _ptr(status, torch.int32, "status"), _stream(stream))
    _check("actkv_compact_noalloc", rc)
