"""A bounded wait inside the tensor-core score kernels that runs out, without any GPU fault.

Every wait of those kernels (on a shared-memory barrier) has a limit.  The fault-injection hook
`actkv_debug_inject_stall` makes the K-tile producers stop issuing key tiles after a given tile
(nothing is left in flight) and shortens the limit to a few milliseconds, so the MMA and epilogue
roles run into it.  Expected: the call returns, status[0] == ACTKV_E_TIMEOUT, select and
compaction of the same step do nothing (index lists, pool, tables, free list untouched), and a
following normal step on the same context gives exactly the bits of a run that never stalled.
"""
import numpy as np
import pytest
import torch

from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import synth

import parity_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _workload(seed):
    # 2 layers x 2 KV heads x 2 requests, 8 x 32 = 256 window rows: both score kernels on the tensor-core path,
    # several key tiles per CTA
    return synth.Workload("stall", 2, 2, 8, [1500, 700], [32, 16], [400, 200], table_style="fragmented", seed=seed,
                          poison_tail=True)


def _snapshot(inst):
    return [U.bits(inst.pool).copy()] + [t.clone() for t in (inst.page_table, inst.seq_len, inst.free_list, inst.free_count)]


def _unchanged(inst, snap):
    assert np.array_equal(U.bits(inst.pool), snap[0])
    for t, s in zip((inst.page_table, inst.seq_len, inst.free_list, inst.free_count), snap[1:]):
        assert torch.equal(t, s)


@pytest.mark.parametrize("which", ["lse", "pooled"])
def test_a_wait_that_runs_out_is_reported_and_the_step_does_nothing(which):
    wl = _workload(41)
    # the reference: a run that never stalls
    ref = synth.generate(wl, DEV)
    assert B.actkv_score_path(B.pool_desc(ref.pool), wl.n_q_heads, max(wl.windows), wl.sm_scale, ref.q) == 1
    comp_ref = U.run_step(ref)
    comp_ref.check_status()
    lse_ref = comp_ref.lse.clone()

    inst = synth.generate(wl, DEV)
    snap = _snapshot(inst)
    # "pooled": the LSE comes from outside, so the first kernel to stall is the pooled-score kernel
    lse_in = lse_ref if which == "pooled" else None
    B.actkv_debug_inject_stall(1, 5000)            # tile 0 arrives, nothing after it; waits give up after ~5 ms
    try:
        from paper_2609_31395_b200 import harness as H
        comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads,
                            H.sizes_of(inst), want_lse=True, want_ties=True)
        comp.sel_idx.fill_(-12345)
        comp.step(inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, wl.sm_scale, wl.causal, lse_in=lse_in)
        torch.cuda.synchronize()                   # the call returns: the kernels left on their own
    finally:
        B.actkv_debug_inject_stall(-1)
    st = comp.status.cpu().tolist()
    assert st[0] == B.E_TIMEOUT, st
    assert bool((comp.sel_idx == -12345).all()), "select consumed the scores of a launch that gave up"
    _unchanged(inst, snap)                         # compaction did nothing: pool, tables and free list as before

    # the same context, the same buffers, a normal step: exactly the reference's bits
    comp.status.zero_()
    comp.step(inst.q, inst.win_indptr, inst.tok_indptr, inst.budget, wl.sm_scale, wl.causal, lse_in=lse_in)
    torch.cuda.synchronize()
    comp.check_status()
    assert torch.equal(comp.score, comp_ref.score)
    assert torch.equal(comp.sel_idx, comp_ref.sel_idx)
    assert torch.equal(comp.lse, comp_ref.lse) or which == "pooled"
    assert np.array_equal(U.bits(inst.pool), U.bits(ref.pool))
    for a, b in zip((inst.page_table, inst.seq_len, inst.free_list, inst.free_count),
                    (ref.page_table, ref.seq_len, ref.free_list, ref.free_count)):
        assert torch.equal(a, b)


def test_hook_rejects_a_stall_without_a_limit():
    with pytest.raises(B.ActKVError):
        B.actkv_debug_inject_stall(0, 0)
    B.actkv_debug_inject_stall(-1)
