"""actkv_score_sliding (sliding-window attention layers: a query at position p attends to keys
p - S < j <= p) against the oracle, element by element, through the C ABI: the tensor-core kernels
(with the key tiles no row sees skipped), the FMA kernels, the LSE computed by the library and
supplied, causal and not, and the sliding-window layers of an interleaved model handed over as a
pool view with a skipping layer stride.
"""
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


def _check(inst, S, want_path, lse_mode="internal"):
    wl = inst.wl
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads,
                        H.sizes_of(inst), want_lse=True)
    assert B.actkv_score_path(comp.pd, wl.n_q_heads, max(wl.windows), wl.sm_scale, inst.q) == want_path
    want, lse, tok = O.score(U.bits(inst.pool), inst.page_table.cpu().numpy(), inst.seq_len.cpu().numpy(), U.bits(inst.q),
                             inst.win_indptr.cpu().numpy(), wl.n_q_heads, wl.sm_scale, wl.causal, window_left=S)
    s = comp.sz
    lse_in = None
    if lse_mode == "supplied":
        lse_in = torch.from_numpy(np.nan_to_num(lse).astype(np.float32)).to(DEV)
    comp.score.fill_(float("nan"))
    B.actkv_score_sliding(comp.pd, comp.td, 0, wl.n_layers, inst.q, inst.win_indptr, wl.n_q_heads, lse_in, wl.sm_scale,
                          wl.causal, S, inst.tok_indptr, comp.score, comp.lse, s.sum_win, s.max_win, s.sum_tok, s.max_tok,
                          comp.ws_score, comp.status)
    torch.cuda.synchronize()
    comp.check_status()
    got = comp.score.cpu().numpy()
    assert np.isfinite(got).all()
    err = U.max_rel(got, want)
    assert err <= U.SCORE_RTOL, f"S = {S}: score max-rel {err:.3e}"
    assert not got[want == 0].any(), "a key no row sees must score exactly 0"
    m = ~np.isnan(lse)
    assert np.abs(comp.lse.cpu().numpy()[m] - lse[m]).max() < 1e-4
    return err


@pytest.mark.parametrize("causal", [False, True])
def test_sliding_window_on_the_tensor_core_path(causal):
    # 256 and 128 window rows; 3100 keys = 25 key tiles, most of them invisible for a short window
    wl = synth.Workload("sw", 2, 2, 8, [3100, 700], [32, 16], [800, 200], table_style="fragmented", causal=causal, seed=61,
                        poison_tail=True)
    inst = synth.generate(wl, DEV)
    for S in (128, 1, 17, 600, 3100, 5000):
        _check(inst, S, 1)
    _check(inst, 128, 1, lse_mode="supplied")


@pytest.mark.parametrize("causal", [False, True])
def test_sliding_window_with_many_rows_and_chunks(causal):
    # 512 window rows (four row blocks, two row chunks per key tile), 9000 keys over several CTAs per unit
    wl = synth.Workload("sw512", 1, 1, 8, [9000 + 7, 260], [64, 64], [2000, 100], table_style="permutation", causal=causal,
                        seed=62, poison_tail=True)
    inst = synth.generate(wl, DEV)
    for S in (128, 1000, 8900):
        _check(inst, S, 1)


@pytest.mark.parametrize("causal", [False, True])
def test_sliding_window_on_the_fma_path(causal):
    wl = synth.Workload("swfma", 2, 2, 2, [500, 130], [8, 4], [120, 40], head_dim=64, page_size=8, table_style="fragmented",
                        causal=causal, seed=63, poison_tail=True)
    inst = synth.generate(wl, DEV)
    for S in (1, 9, 128, 1000):
        _check(inst, S, 0)
    _check(inst, 9, 0, lse_mode="supplied")


def test_sliding_window_layers_of_an_interleaved_model():
    """head_dim 64, 8 query heads per KV head, every other layer a sliding-window layer (window 128): those
    layers are handed over as a pool view whose layer stride skips the full-attention ones."""
    wl = synth.Workload("gptoss-sw", 3, 2, 8, [1500, 300], [16, 9], [400, 80], head_dim=64, table_style="fragmented",
                        causal=True, seed=64, poison_tail=True)
    inst = synth.generate(wl, DEV)
    shape = list(inst.pool.shape)
    shape[0] *= 2
    g = torch.Generator(device=DEV).manual_seed(98)
    big = torch.randn(shape, generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    big[1::2] = inst.pool
    inst.pool = big[1::2]
    assert inst.pool.stride(0) == 2 * big[0].numel()
    before = big.clone()
    _check(inst, 128, 1)
    assert torch.equal(big.view(torch.int16), before.view(torch.int16))       # scoring writes nothing into the pool


def test_window_zero_is_the_plain_score():
    wl = synth.Workload("sw0", 1, 2, 4, [900, 333], [32, 16], [250, 100], table_style="fragmented", seed=65, poison_tail=True)
    inst = synth.generate(wl, DEV)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads,
                        H.sizes_of(inst), want_lse=True)
    comp.run_score(inst.q, inst.win_indptr, inst.tok_indptr, wl.sm_scale, wl.causal)
    torch.cuda.synchronize()
    plain = comp.score.clone()
    s = comp.sz
    B.actkv_score_sliding(comp.pd, comp.td, 0, 1, inst.q, inst.win_indptr, wl.n_q_heads, None, wl.sm_scale, wl.causal, 0,
                          inst.tok_indptr, comp.score, comp.lse, s.sum_win, s.max_win, s.sum_tok, s.max_tok, comp.ws_score,
                          comp.status)
    torch.cuda.synchronize()
    comp.check_status()
    assert torch.equal(plain, comp.score)
