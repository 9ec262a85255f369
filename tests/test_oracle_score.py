"""Pins for the oracle's score path (CPU only): what the paper and the mathematics fix."""
import math

import numpy as np
import pytest
import torch

from oracle import actkv_oracle as O
from paper_2609_31395_b200 import synth

from conftest import read_golden


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def test_slot_map_printed_example():
    g = read_golden("slot_map_example.txt")
    got = O.slot_map(g["block_table"], g["seqused_k"][0], g["block_size"][0])
    assert got.tolist() == g["slot_map"]


def test_kv_footprint_of_benchmark_shape():
    g = read_golden("kv_footprint.txt")
    nbytes = g["tokens"][0] * g["layers"][0] * g["kv_heads"][0] * g["head_dim"][0] * g["bytes_per_elem"][0] * 2
    assert abs(nbytes / 2**30 - g["gib"][0]) < 0.005
    wl = synth.config3()
    assert (wl.n_layers, wl.n_kv_heads, wl.head_dim, wl.seq_lens[0]) == (48, 4, 128, 35000)


def test_kernel_table_mean_rederives():
    g = read_golden("kernel_table.txt")
    cells = g["row_1k_0p5k"] + g["row_2k_1p5k"] + g["row_6k_4k"]
    assert abs(sum(cells) / 12 - g["mean"][0]) < 0.005


def _rand_unit(rng, W, G, L, D):
    return rng.standard_normal((W, G, D)), rng.standard_normal((L, D))


def test_bf16_bits_roundtrip():
    x = torch.randn(1000, dtype=torch.float32).to(torch.bfloat16)
    assert np.array_equal(O.bf16_bits_to_f64(_bits(x)), x.double().numpy())


def test_rows_sum_to_one_and_lse_identity():
    """Section 7.1: exp(s - LSE) is the softmax row; its entries sum to 1."""
    rng = np.random.default_rng(0)
    q, k = _rand_unit(rng, 5, 3, 77, 16)
    scale = 0.25
    _, lse = O.score_unit(q, k, scale, causal=False)
    s = scale * np.einsum("wgd,jd->wgj", q, k)
    a = np.exp(s - lse[:, :, None])
    assert np.abs(a.sum(axis=2) - 1.0).max() < 1e-12
    direct = np.exp(s) / np.exp(s).sum(axis=2, keepdims=True)
    assert np.abs(a - direct).max() < 1e-14


def test_single_row_single_head_is_textbook_softmax():
    """G = W = 1: max and mean are identities, the score is softmax(scale * q K^T)."""
    rng = np.random.default_rng(1)
    q, k = _rand_unit(rng, 1, 1, 300, 32)
    scale = 1 / math.sqrt(32)
    sc, _ = O.score_unit(q, k, scale, causal=False)
    ref = torch.softmax(torch.from_numpy(scale * (k @ q[0, 0])), dim=0).numpy()
    assert np.abs(sc.astype(np.float64) - ref).max() < 1e-7 * ref.max() + 1e-12
    assert sc.dtype == np.float32


def _loops(q, k, scale, causal):
    """The definition by pure Python loops: softmax by exp/sum, max over g, mean over w."""
    W, G, D = q.shape
    L = k.shape[0]
    out = [0.0] * L
    for w in range(W):
        probs = []
        for g in range(G):
            vis = [j for j in range(L) if (not causal) or j <= L - W + w]
            e = {j: math.exp(scale * sum(q[w, g, d] * k[j, d] for d in range(D))) for j in vis}
            z = sum(e.values())
            probs.append({j: e[j] / z for j in vis})
        for j in range(L):
            out[j] += max(p.get(j, 0.0) for p in probs) / W
    return np.array(out)


@pytest.mark.parametrize("causal", [False, True])
def test_against_pure_python_loops(causal):
    rng = np.random.default_rng(2)
    q, k = _rand_unit(rng, 3, 2, 9, 4)
    sc, _ = O.score_unit(q, k, 0.5, causal=causal)
    ref = _loops(q, k, 0.5, causal)
    assert np.abs(sc - ref).max() < 1e-7


def test_causal_window_rule():
    """Row w of a W-row window at the end of L tokens sees keys 0..L-W+w, nothing later."""
    rng = np.random.default_rng(3)
    W, G, L, D = 4, 2, 12, 8
    q, k = _rand_unit(rng, W, G, L, D)
    sc, lse = O.score_unit(q, k, 0.3, causal=True)
    # the last key is visible to the last row only: its score is that row's max_g prob / W
    s_last = 0.3 * np.einsum("gd,jd->gj", q[W - 1], k)
    p_last = np.exp(s_last - lse[W - 1][:, None])
    assert abs(sc[L - 1] - p_last[:, L - 1].max() / W) < 1e-7
    # row 0 sees exactly L-W+1 keys: its lse is the logsumexp over them
    s0 = 0.3 * np.einsum("gd,jd->gj", q[0], k[: L - W + 1])
    assert np.abs(lse[0] - np.log(np.exp(s0).sum(axis=1))).max() < 1e-12


def test_score_mass_bounds_and_degenerate_group():
    rng = np.random.default_rng(4)
    W, G, L, D = 6, 4, 200, 16
    q, k = _rand_unit(rng, W, G, L, D)
    sc, _ = O.score_unit(q, k, 0.25, causal=False)
    total = float(sc.astype(np.float64).sum())
    assert 1.0 - 1e-6 <= total <= G + 1e-6
    # identical q-heads inside the group: the max is a no-op, the mass is exactly 1
    q_same = np.repeat(q[:, :1, :], G, axis=1)
    sc1, _ = O.score_unit(q_same, k, 0.25, causal=False)
    assert abs(float(sc1.astype(np.float64).sum()) - 1.0) < 1e-6


def test_score_permutation_invariances():
    rng = np.random.default_rng(5)
    W, G, L, D = 5, 3, 64, 8
    q, k = _rand_unit(rng, W, G, L, D)
    sc, _ = O.score_unit(q, k, 0.3, causal=False)
    sc_w, _ = O.score_unit(q[rng.permutation(W)], k, 0.3, causal=False)
    sc_g, _ = O.score_unit(q[:, rng.permutation(G)], k, 0.3, causal=False)
    assert np.abs(sc - sc_w).max() < 1e-7 and np.abs(sc - sc_g).max() < 1e-7
    perm = rng.permutation(L)
    sc_k, _ = O.score_unit(q, k[perm], 0.3, causal=False)
    assert np.abs(sc[perm] - sc_k).max() < 1e-7


def test_supplied_lse_reproduces_internal():
    rng = np.random.default_rng(6)
    q, k = _rand_unit(rng, 4, 2, 50, 8)
    sc, lse = O.score_unit(q, k, 0.4, causal=True)
    sc2, _ = O.score_unit(q, k, 0.4, causal=True, lse_in=lse)
    assert np.array_equal(sc, sc2)


def _tiny_instance(table_style="permutation", causal=False, seed=0):
    wl = synth.Workload("tiny", 2, 2, 2, [37, 20], [3, 2], [10, 8], head_dim=16, page_size=4,
                        table_style=table_style, causal=causal, seed=seed, plant_frac=0.0)
    return synth.generate(wl, "cpu")


def test_paged_score_matches_contiguous_and_page_relabeling():
    """Scoring through the block table equals scoring the gathered keys; relabeling physical
    pages together with their data changes nothing."""
    inst = _tiny_instance()
    wl = inst.wl
    pool = _bits(inst.pool)
    pt = inst.page_table.numpy()
    sl = inst.seq_len.numpy()
    out, lse, tok = O.score(pool, pt, sl, _bits(inst.q), inst.win_indptr.numpy(), wl.n_q_heads, wl.sm_scale, False)
    assert not np.isnan(out).any()
    # by hand for one unit
    l, h, r = 1, 1, 0
    slots = [pt[r][j // 4] * 4 + j % 4 for j in range(sl[r])]
    kk = O.bf16_bits_to_f64(pool[l, 0].reshape(-1, 2, 16)[slots, h])
    qq = O.bf16_bits_to_f64(_bits(inst.q)[l, 0:3, h * 2:(h + 1) * 2])
    ref, _ = O.score_unit(qq, kk, wl.sm_scale, False)
    assert np.array_equal(out[l, h, tok[r]:tok[r + 1]], ref)
    # relabel pages
    n_pages = pool.shape[2]
    perm = np.random.default_rng(0).permutation(n_pages)       # new id of old page p is perm[p]
    pool2 = np.empty_like(pool)
    pool2[:, :, perm] = pool
    pt2 = np.where(pt >= 0, perm[np.clip(pt, 0, None)], -1)
    out2, _, _ = O.score(pool2, pt2, sl, _bits(inst.q), inst.win_indptr.numpy(), wl.n_q_heads, wl.sm_scale, False)
    assert np.array_equal(out, out2)


def test_planted_keys_are_retained_config1():
    """With the generator's shared-direction action queries every planted key survives TopK."""
    wl = synth.config1()
    wl.n_kv_heads = 2          # two heads are enough for the pin and keep the CPU suite short
    inst = synth.generate(wl, "cpu")
    out, _, tok = O.score(_bits(inst.pool), inst.page_table.numpy(), inst.seq_len.numpy(), _bits(inst.q),
                          inst.win_indptr.numpy(), wl.n_q_heads, wl.sm_scale, False)
    planted = set(inst.planted[0].tolist())
    assert len(planted) == 82
    for h in range(wl.n_kv_heads):
        kept = set(O.select_unit(out[0, h], wl.budgets[0]).tolist())
        assert planted <= kept


# ---- sliding-window layers (window_left = S: a query at position p attends to keys p - S < j <= p) ----


def _loops_windowed(q, k, scale, causal, S):
    """The definition in pure-Python loops."""
    W, G, D = q.shape
    L = k.shape[0]
    out = [0.0] * L
    for w in range(W):
        p = L - W + w if causal else L - 1
        best = [0.0] * L
        for g in range(G):
            vis = [j for j in range(L) if j <= p and (S <= 0 or j > p - S)]
            logit = {j: scale * sum(q[w, g, d] * k[j, d] for d in range(D)) for j in vis}
            z = sum(math.exp(v) for v in logit.values())
            for j in vis:
                best[j] = max(best[j], math.exp(logit[j]) / z)
        for j in range(L):
            out[j] += best[j] / W
    return np.array(out)


@pytest.mark.parametrize("causal", [False, True])
def test_sliding_window_against_python_loops(causal):
    rng = np.random.default_rng(3)
    q, k = _rand_unit(rng, 4, 2, 23, 5)
    for S in (0, 1, 3, 7, 22, 23, 100):
        got, lse = O.score_unit(q, k, 0.4, causal, window_left=S)
        assert np.abs(got.astype(np.float64) - _loops_windowed(q, k, 0.4, causal, S)).max() < 1e-7
        assert np.isfinite(lse).all()


def test_sliding_window_closed_forms():
    rng = np.random.default_rng(4)
    W, G, L = 6, 3, 40
    q, k = _rand_unit(rng, W, G, L, 8)
    # S = 1, causal: a row sees its own key only, with probability 1 in every head -> each window position
    # scores 1/W, every other key 0, and the LSE is the row's own logit
    got, lse = O.score_unit(q, k, 0.3, True, window_left=1)
    want = np.zeros(L)
    want[L - W:] = 1.0 / W
    assert np.abs(got - want).max() < 1e-7
    own = 0.3 * np.einsum("wgd,wd->wg", q, k[L - W:])
    assert np.abs(lse - own).max() < 1e-12
    # a window at least as long as the cache changes nothing
    for causal in (False, True):
        full, lse_f = O.score_unit(q, k, 0.3, causal)
        same, lse_s = O.score_unit(q, k, 0.3, causal, window_left=L + 5)
        assert np.array_equal(full, same) and np.array_equal(lse_f, lse_s)
    # not causal, one row, one head: the textbook softmax over the last S keys, 0 before them
    S = 9
    got, _ = O.score_unit(q[:1, :1], k, 0.3, False, window_left=S)
    ref = torch.softmax(torch.from_numpy(0.3 * (k[L - S:] @ q[0, 0])), dim=0).numpy()
    assert np.abs(got[L - S:] - ref).max() < 1e-7 and not got[:L - S].any()
    # visible probabilities of a row sum to 1, so the unit's mass stays in [1, G]
    got, _ = O.score_unit(q, k, 0.3, True, window_left=5)
    assert 1.0 - 1e-6 <= got.sum() <= G + 1e-6 and not got[:L - W - 4].any()
