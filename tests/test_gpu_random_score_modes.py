"""Seeded random shapes through the two other score entry points, against the oracle element by element:
actkv_score_sliding (sliding-window layers; the LSE computed by the library or supplied) and
actkv_score_accumulate (the streaming update, fed a random number of queries per call).  Shapes are drawn
across the switch between the FMA and the tensor-core kernels, pages of 8 to 64 tokens, groups that are not
powers of two, requests shorter than their window (non-causal) or than one key tile.
"""
import numpy as np
import pytest
import torch

from paper_2609_31395_b200 import binding as B
from paper_2609_31395_b200 import harness as H
from paper_2609_31395_b200 import synth

import parity_util as U
import test_gpu_sliding as TS
import test_gpu_stream as TR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _shape(rng, causal):
    head_dim = int(rng.choice([64, 128, 128, 32]))
    page = int(rng.choice([8, 16, 16, 32, 64]))
    G = int(rng.choice([1, 2, 3, 4, 7, 8, 16]))
    Hkv = int(rng.choice([1, 2, 4]))
    NL = int(rng.integers(1, 4))
    R = int(rng.integers(1, 6))
    wmax = int(rng.choice([4, 16, 40, 64, 96]))
    seq, win, bud = [], [], []
    for _ in range(R):
        L = int(rng.choice([rng.integers(1, 40), rng.integers(40, 700), rng.integers(700, 3000)]))
        w = int(rng.integers(1, wmax + 1))
        if causal:
            w = min(w, L)
        seq.append(L); win.append(w); bud.append(max(1, L // 4))
    style = str(rng.choice(["permutation", "fragmented", "interleaved"]))
    return dict(n_layers=NL, n_kv_heads=Hkv, group=G, seq_lens=seq, windows=win, budgets=bud, head_dim=head_dim,
                page_size=page, causal=causal, table_style=style, poison_tail=True)


@pytest.mark.parametrize("seed", range(24))
def test_random_sliding_window(seed):
    rng = np.random.default_rng(3000 + seed)
    kw = _shape(rng, causal=bool(rng.integers(0, 2)))
    wl = synth.Workload(f"rsw{seed}", seed=4000 + seed, **kw)
    inst = synth.generate(wl, DEV)
    comp = H.Compressor(inst.pool, inst.page_table, inst.seq_len, inst.free_list, inst.free_count, wl.n_q_heads,
                        H.sizes_of(inst), want_lse=True)
    path = B.actkv_score_path(comp.pd, wl.n_q_heads, max(wl.windows), wl.sm_scale, inst.q)
    Lmax = max(wl.seq_lens)
    for S in sorted({1, int(rng.integers(2, 200)), int(rng.integers(1, Lmax + 1)), Lmax + 5}):
        TS._check(inst, S, path, lse_mode="supplied" if rng.integers(0, 3) == 0 else "internal")


@pytest.mark.parametrize("seed", range(16))
def test_random_streaming_update(seed):
    rng = np.random.default_rng(5000 + seed)
    kw = _shape(rng, causal=True)
    # a request outside any action region (no window) now and then
    kw["windows"] = [0 if (rng.integers(0, 6) == 0 and len(kw["windows"]) > 1 and i > 0) else w
                     for i, w in enumerate(kw["windows"])]
    kw["windows"] = [min(w, 24) for w in kw["windows"]]          # one call per chunk of queries: keep the call count low
    if max(kw["windows"]) == 0:
        kw["windows"][0] = 1
    wl = synth.Workload(f"rst{seed}", seed=6000 + seed, **kw)
    inst = synth.generate(wl, DEV)
    pool_bits = U.bits(inst.pool)
    chunk = int(rng.integers(1, 6))
    comp, score_io, n_calls = TR._run_stream(inst, chunk=chunk)
    assert n_calls == -(-max(wl.windows) // chunk)
    got = score_io.cpu().numpy()
    want = TR._oracle_stream_all(inst, pool_bits, comp.lse.cpu().numpy())
    tok = inst.tok_indptr.cpu().tolist()
    for r in range(wl.n_req):
        seg = slice(tok[r], tok[r + 1])
        if wl.windows[r] == 0:
            assert (got[:, :, seg] == 0).all()
            continue
        err = U.max_rel(got[:, :, seg], want[:, :, seg])
        assert err <= U.SCORE_RTOL, f"request {r}: max-rel {err:.3e}"
