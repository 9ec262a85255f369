"""Every kernel and every memset of a call runs on the stream the call was given.

The step is queued on a non-blocking side stream behind a long sleep kernel, and the real inputs (queries,
sequence lengths, budgets, logits) are copied into place on that stream only after the sleep: a kernel
that the library launched on any other stream would start at once, read the zeroed placeholders and leave
results that differ from the reference run on the default stream.
"""
import pytest
import torch

from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import harness as H
from paper_2609_31395_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SLEEP_CYCLES = 800_000_000          # about 0.4 s: far longer than the host needs to queue a step


def _wl():
    return synth.Workload("streams", 5, 2, 8, [1500, 333, 700, 90], [32, 16, 24, 8], [400, 100, 200, 90],
                          table_style="fragmented", seed=71, poison_tail=True)


def _run(form, inst, comp, lrfu):
    wl = inst.wl
    args = (inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, wl.sm_scale, wl.causal)
    if form == "one call":
        comp.step(*args)
    elif form == "pipelined":
        comp.step_pipelined(*args)
    elif form == "in place":
        comp.step(*args, inplace=True)
    elif form == "pipelined in place":
        comp.step_pipelined(*args, inplace=True)
    elif form == "lrfu":
        comp.step(*args, lrfu=lrfu)
    elif form == "pipelined lrfu":
        comp.step_pipelined(*args, lrfu=lrfu)
    else:
        raise AssertionError(form)


def _make(form):
    wl = _wl()
    inst = synth.generate(wl, DEV)
    sz = H.sizes_of(inst)
    lpc = 2 if form.startswith("pipelined") else None
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads, sz,
                        layers_per_call=lpc, want_lse=True)
    lrfu = None
    if "lrfu" in form:
        lrfu = H.LrfuState(wl.n_layers * wl.n_kv_heads, sz, DEV, 0.9, 0.5, torch.tensor([4, 0, 300, 7], dtype=torch.int32,
                                                                                         device=DEV))
        lrfu.keep_score.uniform_(0.0, 1e-3, generator=torch.Generator(device=DEV).manual_seed(3))
    return inst, comp, lrfu


@pytest.mark.parametrize("form", ["one call", "pipelined", "in place", "pipelined in place", "lrfu", "pipelined lrfu"])
def test_the_step_runs_on_the_stream_it_is_given(form):
    a, comp_a, lrfu_a = _make(form)
    _run(form, a, comp_a, lrfu_a)
    torch.cuda.synchronize()
    comp_a.check_status()

    b, comp_b, lrfu_b = _make(form)
    live = [b.q, b.seq_len, b.budget, b.page_table]
    real = [t.clone() for t in live]
    for t in live:
        t.zero_()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        torch.cuda._sleep(SLEEP_CYCLES)
        for t, r in zip(live, real):
            t.copy_(r, non_blocking=True)
        _run(form, b, comp_b, lrfu_b)
    assert not side.query(), "the side stream should still be busy when the calls return"
    side.synchronize()
    torch.cuda.synchronize()
    comp_b.check_status()
    assert torch.equal(a.pool.view(torch.int16), b.pool.view(torch.int16))
    assert torch.equal(a.page_table, b.page_table) and torch.equal(a.seq_len, b.seq_len)
    assert torch.equal(a.free_list, b.free_list) and torch.equal(a.free_count, b.free_count)
    assert torch.equal(comp_a.lse, comp_b.lse)
    if lrfu_a is not None:
        assert torch.equal(lrfu_a.keep_score.view(torch.int32), lrfu_b.keep_score.view(torch.int32))


def test_the_monitor_and_the_streaming_update_run_on_the_stream_they_are_given():
    R, T, V = 3, 40, 4099
    logits, tok = synth.confidence_logits(R, T, V, seed=5, device=DEV)
    p = B.BudgetParams.paper_defaults()
    budget_in = torch.tensor([512, 896, 100], dtype=torch.int32, device=DEV)

    def monitor(lg):
        hist = torch.zeros((R, 256), dtype=torch.float32, device=DEV)
        hist_len = torch.zeros(R, dtype=torch.int32, device=DEV)
        out = torch.zeros(R, dtype=torch.int32, device=DEV)
        ws = torch.empty(B.actkv_budget_workspace_bytes(R * T, R, 256) + 256, dtype=torch.uint8, device=DEV)
        status = torch.zeros(4, dtype=torch.int32, device=DEV)
        B.actkv_budget(lg, tok, R * T, V, hist, hist_len, 256, p, None, budget_in, out, None, R, ws, status)
        return hist, hist_len, out, status, ws

    ref = monitor(logits)
    torch.cuda.synchronize()
    live = torch.zeros_like(logits)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        torch.cuda._sleep(SLEEP_CYCLES)
        live.copy_(logits, non_blocking=True)
        got = monitor(live)
    side.synchronize()
    torch.cuda.synchronize()
    assert got[3].cpu().tolist()[0] == 0
    for x, y in zip(ref[:3], got[:3]):
        assert torch.equal(x, y)

    # streaming update: one query per request per call
    wl = synth.Workload("streams2", 2, 2, 4, [900, 333], [4, 4], [200, 100], causal=True, table_style="fragmented", seed=72)
    inst = synth.generate(wl, DEV)
    sz = H.sizes_of(inst)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads, sz,
                        want_lse=True)
    B.actkv_score_lse(comp.pd, comp.td, 0, wl.n_layers, inst.q, inst.win_indptr, wl.n_q_heads, wl.sm_scale, True,
                      inst.tok_indptr, comp.lse, sz.sum_win, sz.max_win, sz.sum_tok, sz.max_tok, comp.ws_score, comp.status)
    first = inst.win_indptr[:-1].to(torch.int64)
    q1, lse1 = inst.q[:, first].contiguous(), comp.lse[:, first].contiguous()
    win1 = torch.arange(wl.n_req + 1, dtype=torch.int32, device=DEV)
    steps = torch.zeros(wl.n_req, dtype=torch.int32, device=DEV)
    lens = torch.tensor([L - W + 1 for L, W in zip(wl.seq_lens, wl.windows)], dtype=torch.int32, device=DEV)
    td = B.tables_desc(inst.page_table, lens, inst.free_list, inst.free_count)

    def update(q):
        io = torch.zeros((wl.n_layers, wl.n_kv_heads, sz.sum_tok), dtype=torch.float32, device=DEV)
        B.actkv_score_accumulate(comp.pd, td, 0, wl.n_layers, q, win1, wl.n_q_heads, lse1, wl.sm_scale, True,
                                 inst.tok_indptr, steps, io, wl.n_req, 1, sz.sum_tok, int(lens.max()), comp.ws_score,
                                 comp.status)
        return io

    torch.cuda.synchronize()
    ref_io = update(q1)
    torch.cuda.synchronize()
    q_live = torch.zeros_like(q1)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        torch.cuda._sleep(SLEEP_CYCLES)
        q_live.copy_(q1, non_blocking=True)
        got_io = update(q_live)
    side.synchronize()
    torch.cuda.synchronize()
    comp.check_status()
    assert torch.equal(ref_io, got_io)
