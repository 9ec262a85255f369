"""GPU parity of the streaming score update (Algorithm 3 triggered per decode step, LSE supplied,
running mean restarted at region entry) through the C ABI, against the oracle's step-by-step form
and against the batch score of the whole window."""
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


def _oracle_stream_all(inst, pool_bits, lse_np):
    """Oracle running mean after every request's whole window, fed one query at a time."""
    wl = inst.wl
    pt, sl = inst.page_table.cpu().numpy(), np.asarray(wl.seq_lens)
    wi, ti = inst.win_indptr.cpu().numpy(), inst.tok_indptr.cpu().numpy()
    q_bits = U.bits(inst.q)
    G = wl.group
    want = np.zeros((wl.n_layers, wl.n_kv_heads, int(ti[-1])), dtype=np.float64)
    for a in range(wl.n_layers):
        for h in range(wl.n_kv_heads):
            for r in range(wl.n_req):
                L, W = int(sl[r]), int(wi[r + 1] - wi[r])
                if L == 0 or W == 0:
                    continue
                k = O.bf16_bits_to_f64(O.gather_rows(pool_bits, a, 0, h, O.slot_map(pt[r], L, wl.page_size)))
                q = O.bf16_bits_to_f64(q_bits[a, wi[r]:wi[r + 1], h * G:(h + 1) * G])
                lse = lse_np[a, wi[r]:wi[r + 1], h * G:(h + 1) * G].astype(np.float64)
                want[a, h, ti[r]:ti[r + 1]] = O.score_stream(q, k, wl.sm_scale, lse)
    return want


def _run_stream(inst, chunk=1, garbage=True):
    """Feeds every request's window `chunk` queries per call, the cache length growing with it."""
    wl = inst.wl
    NL, R, Hq = wl.n_layers, wl.n_req, wl.n_q_heads
    sz = H.sizes_of(inst)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, Hq, sz, want_lse=True)
    # the LSE the attention backend would hand over at each decode step (row w: keys j <= L - W + w)
    # (a request without a window is given length 0 for this call: with L > 0 it would be reported)
    len_lse = torch.tensor([L if W else 0 for L, W in zip(wl.seq_lens, wl.windows)], dtype=torch.int32, device=DEV)
    B.actkv_score_lse(comp.pd, B.tables_desc(inst.page_table, len_lse, inst.free_list, inst.free_count), 0, NL, inst.q,
                      inst.win_indptr, Hq, wl.sm_scale, True, inst.tok_indptr, comp.lse, sz.sum_win, sz.max_win,
                      sz.sum_tok, sz.max_tok, comp.ws_score, comp.status)
    torch.cuda.synchronize()
    comp.check_status()
    pd = comp.pd
    score_io = torch.zeros((NL, wl.n_kv_heads, sz.sum_tok), dtype=torch.float32, device=DEV)
    tok = inst.tok_indptr.cpu().tolist()
    if garbage:                                      # what an earlier region left behind in the keys cached at entry
        for r in range(R):
            n0 = wl.seq_lens[r] - wl.windows[r] + 1
            if n0 > 0 and wl.windows[r] > 0:
                score_io[:, :, tok[r]:tok[r] + n0] = 123.0
    win0 = inst.win_indptr.cpu().tolist()
    status = comp.status
    n_calls = 0
    for t0 in range(0, max(wl.windows), chunk):
        rows, w_step, steps, lens = [], [], [], []
        for r in range(R):
            W = wl.windows[r]
            n = max(0, min(chunk, W - t0))
            w_step.append(n)
            steps.append(t0 if n else 0)
            lens.append(wl.seq_lens[r] - W + t0 + n if n else wl.seq_lens[r])
            rows += list(range(win0[r] + t0, win0[r] + t0 + n))
        if not rows:
            break
        idx = torch.tensor(rows, dtype=torch.int64, device=DEV)
        q_step = inst.q[:, idx].contiguous()
        lse_step = comp.lse[:, idx].contiguous()
        win_indptr = torch.tensor([0] + np.cumsum(w_step).tolist(), dtype=torch.int32, device=DEV)
        seq_len = torch.tensor(lens, dtype=torch.int32, device=DEV)
        td = B.tables_desc(inst.page_table, seq_len, inst.free_list, inst.free_count)
        B.actkv_score_accumulate(pd, td, 0, NL, q_step, win_indptr, Hq, lse_step, wl.sm_scale, True, inst.tok_indptr,
                                 torch.tensor(steps, dtype=torch.int32, device=DEV), score_io, len(rows), max(w_step),
                                 sz.sum_tok, max(lens), comp.ws_score, status)
        n_calls += 1
    torch.cuda.synchronize()
    comp.check_status()
    return comp, score_io, n_calls


def _wl(head_dim=128, page=16, G=4, NL=4):
    return synth.Workload("stream", NL, 2, G, [1000, 333, 130, 17, 260, 64, 48, 500], [8, 5, 16, 3, 1, 0, 12, 7],
                          [250, 100, 130, 4, 60, 16, 12, 100], head_dim=head_dim, page_size=page, causal=True,
                          table_style="fragmented", seed=21, poison_tail=True)


@pytest.mark.parametrize("head_dim,page,G", [(128, 16, 4), (128, 16, 8), (64, 8, 2), (128, 16, 3), (64, 32, 7)])
def test_one_query_per_call_matches_oracle_and_batch(head_dim, page, G):
    """(., 16 or 32, .) runs the tensor-core pooled pass with G live rows (a group of 3 or 7 padded to 4 or 8),
    (64, 8, 2) the FMA path."""
    inst = synth.generate(_wl(head_dim, page, G), DEV)
    wl = inst.wl
    pool_bits = U.bits(inst.pool)
    comp, score_io, n_calls = _run_stream(inst, chunk=1)
    assert n_calls == max(wl.windows)
    got = score_io.cpu().numpy()
    want = _oracle_stream_all(inst, pool_bits, comp.lse.cpu().numpy())
    tok = inst.tok_indptr.cpu().tolist()
    for r in range(wl.n_req):
        seg = slice(tok[r], tok[r + 1])
        if wl.windows[r] == 0:                        # never inside an action region: untouched
            assert (got[:, :, seg] == 0).all()
            continue
        err = U.max_rel(got[:, :, seg], want[:, :, seg])
        assert err <= U.SCORE_RTOL, f"request {r}: max-rel {err:.3e}"
    # the batch definition of the same windows with the same LSE (one unit per request)
    keep = [r for r in range(wl.n_req) if wl.windows[r] > 0]
    batch, _, _ = O.score(pool_bits, inst.page_table.cpu().numpy(), np.asarray(wl.seq_lens), U.bits(inst.q),
                          inst.win_indptr.cpu().numpy(), wl.n_q_heads, wl.sm_scale, True,
                          lse_in=comp.lse.cpu().numpy().astype(np.float64),
                          units=[(0, 0, r) for r in keep])
    for r in keep:
        seg = slice(tok[r], tok[r + 1])
        assert U.max_rel(got[0, 0, seg], batch[0, 0, seg]) <= U.SCORE_RTOL


def test_chunks_of_queries_with_the_causal_rule():
    """Three queries per call (the last call of a request ragged): same state as one per call."""
    a = synth.generate(_wl(), DEV)
    b = synth.generate(_wl(), DEV)
    comp_a, one, _ = _run_stream(a, chunk=1)
    comp_b, three, n_calls = _run_stream(b, chunk=3)
    assert n_calls == -(-max(a.wl.windows) // 3)
    x, y = one.cpu().numpy(), three.cpu().numpy()
    assert np.allclose(x, y, rtol=2e-5, atol=1e-12)           # same sums, other rounding order of the running mean
    want = _oracle_stream_all(b, U.bits(b.pool), comp_b.lse.cpu().numpy())
    m = want > 0
    assert U.max_rel(y[m], want[m]) <= U.SCORE_RTOL


def test_region_entry_ignores_old_state_and_argument_errors():
    inst = synth.generate(_wl(NL=2), DEV)
    wl = inst.wl
    _, with_garbage, _ = _run_stream(inst, chunk=1, garbage=True)
    _, clean, _ = _run_stream(inst, chunk=1, garbage=False)
    assert torch.equal(with_garbage, clean)
    sz = H.sizes_of(inst)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads, sz,
                        want_lse=True)
    score_io = torch.zeros((2, wl.n_kv_heads, sz.sum_tok), dtype=torch.float32, device=DEV)
    steps = torch.zeros(wl.n_req, dtype=torch.int32, device=DEV)
    lse = torch.zeros((2, sz.sum_win, wl.n_q_heads), dtype=torch.float32, device=DEV)
    args = (inst.q, inst.win_indptr, wl.n_q_heads)
    with pytest.raises(B.ActKVError):                 # the LSE is required in this mode
        B.actkv_score_accumulate(comp.pd, comp.td, 0, 2, *args, None, wl.sm_scale, True, inst.tok_indptr, steps,
                                 score_io, sz.sum_win, sz.max_win, sz.sum_tok, sz.max_tok, comp.ws_score, comp.status)
    with pytest.raises(B.ActKVError):                 # so is the step count
        B.actkv_score_accumulate(comp.pd, comp.td, 0, 2, *args, lse, wl.sm_scale, True, inst.tok_indptr, None,
                                 score_io, sz.sum_win, sz.max_win, sz.sum_tok, sz.max_tok, comp.ws_score, comp.status)
    # no request inside an action region: nothing to do, not an error
    zero_win = torch.zeros(wl.n_req + 1, dtype=torch.int32, device=DEV)
    B.actkv_score_accumulate(comp.pd, comp.td, 0, 2, inst.q, zero_win, wl.n_q_heads, lse, wl.sm_scale, True,
                             inst.tok_indptr, steps, score_io, 0, 0, sz.sum_tok, sz.max_tok, comp.ws_score, comp.status)
    torch.cuda.synchronize()
    assert (score_io == 0).all() and comp.status.cpu().tolist()[0] == 0


def test_more_than_512_rows_per_call_on_the_tensor_core_path():
    """75 queries x 8 heads = 600 window rows per call: the pooled-score kernel takes them in row groups of 512, the
    first forming the running mean, the second adding its share with the same divisor; second call with 75 queries
    already folded in."""
    wl = synth.Workload("stream600", 2, 2, 8, [1500, 700, 333], [150, 75, 9], [400, 200, 100], causal=True,
                        table_style="fragmented", seed=23, poison_tail=True)
    inst = synth.generate(wl, DEV)
    pd = B.pool_desc(inst.pool)
    assert B.actkv_score_path(pd, wl.n_q_heads, 75, wl.sm_scale, inst.q, streaming=True) == 1
    comp, score_io, n_calls = _run_stream(inst, chunk=75)
    assert n_calls == 2
    got = score_io.cpu().numpy()
    want = _oracle_stream_all(inst, U.bits(inst.pool), comp.lse.cpu().numpy())
    m = want > 0
    assert U.max_rel(got[m], want[m]) <= U.SCORE_RTOL
    assert not got[want == 0].any()
