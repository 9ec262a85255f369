"""CPU oracle for the ActKV hot path.  TEST INFRASTRUCTURE ONLY.

This file is the plain, slow, float64 statement of what the path computes, written from the
paper's equations and algorithms.  It is imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark, and by nothing else: the product path is the CUDA library
and shares no code with this file (only the seeded input generators serve both sides).

Every function cites the passage it follows.  There is no blocking, fusion or reordering
beyond what the definition states; numpy's matmul, sort and exp/log are used as library
steps.  bf16 tensors arrive as numpy uint16 arrays holding the raw bits.

Pins (tests/test_oracle_*.py): the printed slot-map example of Section 2.5; rows of
exp(s - LSE) summing to 1 and equalling a direct softmax (Section 7.1); G = W = 1 reducing to
torch.softmax; a pure-Python triple loop of the definition on tiny inputs; bounds
1 <= sum(score) <= G; invariance under permutations of window rows, group heads and physical
pages; brute-force O(L^2) rank counting and numpy's stable argsort for TopK; a hand-worked
compaction example and byte-permutation / conservation properties; closed forms for the
confidence monitor (uniform logits -> log V, two-point slope, numpy.polyfit, the budget chain
from the Section 8.1 constants).

Parity unpinned (conventions the paper leaves open, fixed by this build): the causal reading of
the action window, per-KV-head selection, ascending survivor order, fresh-page allocation order and free-list discipline, nearest-rank percentile
and the x-axis of the line fit.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

# --------------------------------------------------------------------------------------------
# helpers that are not part of the method


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Raw bf16 bit patterns (uint16) -> float64 values (exact)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------------------------
# Section 2.5 — paged pool addressing


def slot_map(block_table, seqused_k: int, block_size: int) -> np.ndarray:
    """Physical slot of every occupied logical position (Section 2.5).

    Logical token j lives in physical block block_table[j // BS], slot j % BS of it, i.e. in
    physical slot block_table[j // BS] * BS + j % BS.
    """
    block_table = np.asarray(block_table, dtype=np.int64)
    j = np.arange(int(seqused_k), dtype=np.int64)
    return block_table[j // block_size] * block_size + j % block_size


def gather_rows(pool_bits: np.ndarray, layer: int, kv: int, head: int, slots: np.ndarray) -> np.ndarray:
    """Rows (raw bf16 bits) of one head at the given physical slots.

    pool_bits: uint16 [n_layers, 2, n_pages, page_size, n_kv_heads, head_dim]
    (PagedKVCache[2, B, BS, H, D] of Section 2.5 with a leading layer axis).
    """
    n_pages, page_size = pool_bits.shape[2], pool_bits.shape[3]
    flat = pool_bits[layer, kv].reshape(n_pages * page_size, pool_bits.shape[4], pool_bits.shape[5])
    return flat[np.asarray(slots, dtype=np.int64), head, :]


# --------------------------------------------------------------------------------------------
# Sections 2.3 and 7.1, Algorithm 3 — action-region attention score


def score_unit(q_unit: np.ndarray, k_unit: np.ndarray, sm_scale: float, causal: bool,
               lse_in: np.ndarray | None = None, window_left: int = 0):
    """Pooled action-region score of one (layer, request, KV head) unit.

    q_unit float64 [W, G, D]: the action-window queries of the G q-heads that share this KV
    head.  k_unit float64 [L, D]: the cached keys in logical order.

    Steps, in the paper's order:
      s_{w,g,j}  = sm_scale * q_{w,g} . k_j                     (Section 7.1, logit s_ij)
      LSE_{w,g}  = log sum_{j visible} exp(s_{w,g,j})           (Section 7.1, LSE equation)
      A_{w,g,j}  = exp(s_{w,g,j} - LSE_{w,g})                   (Section 7.1, recovery identity)
      AttnScore_{w,j} = max_g A_{w,g,j}                         (Algorithm 3, step 4)
      Out_j      = mean over the W action tokens of AttnScore   (Algorithm 3, step 5)
    Visibility: causal=False, every key; causal=True, the window is the last W cached tokens
    and row w sees j <= L - W + w (a decode step attends to the keys before it and itself
    being already cached); an invisible pair adds 0 and the divisor stays W, which is the
    running mean started from zero of Section 7.1's last paragraph.
    window_left = S > 0: a sliding-window attention layer (Section 8.2 names such layers; the paper does
    not say how they are scored): a query at cache position p attends to the S keys p - S < j <= p only.
    With causal=True row w sits at p = L - W + w; with causal=False every row is taken to sit at the end of
    the cache, p = L - 1.  The LSE runs over the same visible set, so a row's visible probabilities sum to 1.

    Returns (score float32 [L], lse float64 [W, G]).
    """
    W, G, D = q_unit.shape
    L = k_unit.shape[0]
    s = sm_scale * np.einsum("wgd,jd->wgj", q_unit, k_unit)          # [W, G, L]
    j = np.arange(L)[None, None, :]
    pos = (L - W + np.arange(W))[:, None, None] if causal else np.full((W, 1, 1), L - 1)    # position of each row
    visible = j <= pos
    if window_left > 0:
        visible = visible & (j > pos - window_left)
    visible = np.broadcast_to(visible, s.shape)
    if lse_in is None:
        s_masked = np.where(visible, s, -np.inf)
        m = s_masked.max(axis=2, keepdims=True)
        lse = (m + np.log(np.exp(s_masked - m).sum(axis=2, keepdims=True)))[:, :, 0]
    else:
        lse = np.asarray(lse_in, dtype=np.float64).reshape(W, G)
    a = np.where(visible, np.exp(s - lse[:, :, None]), 0.0)          # [W, G, L]
    attn = a.max(axis=1)                                              # max over the GQA group
    out = attn.sum(axis=0) / W                                        # mean over action tokens
    return out.astype(np.float32), lse


def score(pool_bits, page_table, seq_len, q_bits, win_indptr, n_q_heads, sm_scale, causal,
          layers=None, lse_in=None, units=None, window_left=0):
    """actkv_score over whole tensors (or over the listed units only).

    q_bits uint16 [NLs, sum_win, n_q_heads, D]; page_table int [R, max_pages]; seq_len [R];
    win_indptr [R+1].  `layers`: absolute pool layer of each q slab (default 0..NLs-1).
    `units`: optional iterable of (slab, head, request); others are left as NaN.
    GQA mapping: q-head qh serves KV head qh // G (contiguous groups).
    Returns (score float32 [NLs, Hkv, sum_tok], lse float64 [NLs, sum_win, n_q_heads],
    tok_indptr).
    """
    NLs = q_bits.shape[0]
    Hkv, D, P = pool_bits.shape[4], pool_bits.shape[5], pool_bits.shape[3]
    G = n_q_heads // Hkv
    R = len(seq_len)
    layers = list(range(NLs)) if layers is None else list(layers)
    tok_indptr = np.concatenate([[0], np.cumsum(np.asarray(seq_len, dtype=np.int64))])
    out = np.full((NLs, Hkv, int(tok_indptr[-1])), np.nan, dtype=np.float32)
    lse = np.full((NLs, q_bits.shape[1], n_q_heads), np.nan, dtype=np.float64)
    todo = units if units is not None else [(a, h, r) for a in range(NLs) for h in range(Hkv) for r in range(R)]
    for (a, h, r) in todo:
        L = int(seq_len[r])
        w0, w1 = int(win_indptr[r]), int(win_indptr[r + 1])
        if L == 0 or w1 == w0:
            continue
        slots = slot_map(page_table[r], L, P)
        k_unit = bf16_bits_to_f64(gather_rows(pool_bits, layers[a], 0, h, slots))
        q_unit = bf16_bits_to_f64(q_bits[a, w0:w1, h * G:(h + 1) * G, :])
        li = None if lse_in is None else lse_in[a, w0:w1, h * G:(h + 1) * G]
        sc, ls = score_unit(q_unit, k_unit, sm_scale, causal, li, window_left)
        out[a, h, tok_indptr[r]:tok_indptr[r + 1]] = sc
        lse[a, w0:w1, h * G:(h + 1) * G] = ls
    return out, lse, tok_indptr


def score_stream_step(out_prev: np.ndarray, n_prev: int, q_tok: np.ndarray, k_unit: np.ndarray,
                      lse_tok: np.ndarray, sm_scale: float) -> np.ndarray:
    """Algorithm 3 steps 3-5 for ONE current action query of one (request, KV head): the form in which
    the kernel is triggered at every decode step of an action region, with the LSE handed over by the
    attention backend (Section 7.1).

    q_tok float64 [G, D]: the current query of the G q-heads of the group.  k_unit float64 [L, D]:
    the keys cached at this step (the current token's own key included).  lse_tok float64 [G].
    out_prev float64 [<= L]: running mean after the n_prev earlier action queries of this region
    (entries appended since are taken as 0; n_prev = 0 at region entry: the state starts from zero).

      for every q-head of the group: Logits = Q_head . K^T (scaled), Attn = exp(Logits - LSE)   (step 3)
      AttnScore = max over the group of Attn                                                    (step 4)
      Out <- running mean over the action queries seen so far                                   (step 5)
    Returns the new running mean, float64 [L].
    """
    G = q_tok.shape[0]
    L = k_unit.shape[0]
    attn_score = np.zeros(L, dtype=np.float64)
    for g in range(G):
        logits = sm_scale * (k_unit @ q_tok[g])
        attn = np.exp(logits - float(lse_tok[g]))
        attn_score = np.maximum(attn_score, attn)
    out = np.zeros(L, dtype=np.float64)
    out[: out_prev.shape[0]] = out_prev
    return (n_prev * out + attn_score) / (n_prev + 1)


def score_stream(q_unit: np.ndarray, k_unit: np.ndarray, sm_scale: float, lse: np.ndarray,
                 out_prev: np.ndarray | None = None, n_prev: int = 0) -> np.ndarray:
    """`score_stream_step` over the W queries of q_unit [W, G, D] in decoding order: query w is issued
    when the cache holds the first L - W + w + 1 keys of k_unit [L, D].  lse float64 [W, G].
    Returns float64 [L] (the running mean after n_prev + W action queries)."""
    W = q_unit.shape[0]
    L = k_unit.shape[0]
    out = np.zeros(0, dtype=np.float64) if out_prev is None else np.asarray(out_prev, dtype=np.float64)
    for w in range(W):
        out = score_stream_step(out, n_prev + w, q_unit[w], k_unit[: L - W + w + 1], lse[w], sm_scale)
    return out


# --------------------------------------------------------------------------------------------
# Algorithm 1, step 5 — TopK(score, k = B)


def select_unit(score_f32: np.ndarray, budget: int) -> np.ndarray:
    """Indices of the min(B, L) largest float32 scores, ties to the lower index, ascending.

    Written as the definition: order by (score descending, index ascending), take the first
    n, report them in ascending index order (Algorithm 1 step 5 keeps the B highest scores).
    """
    score_f32 = np.asarray(score_f32, dtype=np.float32)
    L = score_f32.shape[0]
    n = min(int(budget), L)
    order = np.lexsort((np.arange(L), -score_f32.astype(np.float64)))   # last key is primary
    return np.sort(np.asarray(order[:n], dtype=np.int64)).astype(np.int32)


# --------------------------------------------------------------------------------------------
# Section 7.2 / Algorithm 4 — compaction (fresh-page form)


# --------------------------------------------------------------------------------------------
# Section 5.1, Algorithm 1 steps 2-5 — attention-aware LRFU keep-score


MASS_BITS = 32            # scores are weighed in units of 2^-32 so that masses add exactly
P_DENOM = 10000           # top-p is taken to 1/10000


def hit_mask_unit(score_f32: np.ndarray, top_p: float) -> np.ndarray:
    """GetHitMask(AttnScore, p): an entry is hit if its score falls within the top-p set
    (Section 5.1; p = 90% in Section 8.1).

    The top-p set is the shortest prefix of the entries ordered by (score descending, index
    ascending) whose mass reaches p of the unit's total mass; the entry that crosses the mark
    is in.  Mass is counted in exact integers: m_i = floor(score_i * 2^32), mark =
    ceil(p_q * sum(m) / 10000) with p_q = round(p * 10000) — so the set does not depend on a
    summation order.  Entries of zero mass are never needed and are not hits.
    """
    s = np.asarray(score_f32, dtype=np.float32)
    L = s.shape[0]
    # scores are pooled probabilities in [0, 1]; anything outside [0, 256] is clipped so that masses of
    # up to 2^16 entries still add up in 64 bits
    mass = [int(math.floor(min(max(float(x), 0.0), 256.0) * (1 << MASS_BITS))) for x in s]
    total = sum(mass)
    p_q = int(round(top_p * P_DENOM))
    mark = -(-(p_q * total) // P_DENOM)
    order = np.lexsort((np.arange(L), -s.astype(np.float64)))
    hit = np.zeros(L, dtype=bool)
    acc = 0
    for i in order:
        if acc >= mark:
            break
        hit[i] = True
        acc += mass[i]
    return hit


def keep_score_update(ks_f32: np.ndarray, score_f32: np.ndarray, hit: np.ndarray, lam: float) -> np.ndarray:
    """KS_t = lambda * KS_{t-1} + AttnScore_t * [hit at t]   (Section 5.1 equation; Algorithm 1 step 4),
    in float32 with one rounding per operation (product, then sum).  New entries of the round
    enter with KS = 0 (Algorithm 1 step 2)."""
    ks = np.asarray(ks_f32, dtype=np.float32)
    s = np.asarray(score_f32, dtype=np.float32)
    decayed = (np.float32(lam) * ks).astype(np.float32)
    return np.where(hit, (decayed + s).astype(np.float32), decayed).astype(np.float32)


def rank_keys(ks_f32: np.ndarray, n_protect: int) -> np.ndarray:
    """What TopK ranks (Algorithm 1 step 5): the keep-score, with the first n_protect entries (system
    prompt and task description, Section 8.1) lifted to +inf so that they are always retained."""
    out = np.array(ks_f32, dtype=np.float32, copy=True)
    out[: int(n_protect)] = np.inf
    return out


@dataclass
class Tables:
    page_table: np.ndarray   # int32 [R, max_pages], unused -1
    seq_len: np.ndarray      # int32 [R]
    free_list: np.ndarray    # int32 [n_pages]
    free_count: int


def compact(pool_bits: np.ndarray, tables: Tables, sel, budget, layers=None):
    """Pack the survivors of every compacting request into fresh pages; free the old pages.

    What Algorithm 4 achieves (Section 7.2: the retained entries end up packed in contiguous
    logical slots by pure copies with disjoint sources and destinations, freed blocks go back
    to the serving system), with the destination taken from the free list:
      requests r ascending with B_r < L_r:  n = B_r, X = ceil(n / BS), Y = ceil(L_r / BS),
      new_page[i] = free_list[free_count - 1 - (off + i)], i < X, off = pages taken by earlier
      requests; for every layer, head, i < n: K and V row of token sel[layer][head][r][i]
      -> logical slot i of the new pages (survivors keep ascending original order).
      Then page_table[r] = new pages ++ -1.., seq_len[r] = n, free_count -= total X, and for r
      ascending, i = 0..Y-1 ascending, the old pages are pushed back.
    sel[a][h][r]: ascending token indices of pool layer layers[a].  Tables are updated in all
    cases (the call covers every layer the caller passes).  Raises if the free list is short.
    Returns (new pool_bits copy, new Tables).
    """
    P, Hkv = pool_bits.shape[3], pool_bits.shape[4]
    n_pages = pool_bits.shape[2]
    layers = list(range(pool_bits.shape[0])) if layers is None else list(layers)
    new_pool = pool_bits.copy()
    pt = tables.page_table.copy()
    sl = tables.seq_len.copy()
    fl = tables.free_list.copy()
    fc = int(tables.free_count)
    R = len(sl)
    compacting = [r for r in range(R) if int(budget[r]) < int(sl[r])]
    need = sum(-(-int(budget[r]) // P) for r in compacting)
    if need > fc:
        raise RuntimeError("free list short")
    off = 0
    old_pages = {}
    for r in compacting:
        L, n = int(sl[r]), int(budget[r])
        X, Y = -(-n // P), -(-L // P)
        new_page = [int(fl[fc - 1 - (off + i)]) for i in range(X)]
        off += X
        old = [int(x) for x in tables.page_table[r, :Y]]
        old_pages[r] = old
        src_slot_of = slot_map(old, L, P)
        for a, layer in enumerate(layers):
            src = pool_bits[layer].reshape(2, n_pages * P, Hkv, -1)
            dst = new_pool[layer].reshape(2, n_pages * P, Hkv, -1)
            for h in range(Hkv):
                idx = np.asarray(sel[a][h][r], dtype=np.int64)
                assert idx.shape[0] == n
                # survivor i (token idx[i]) goes to logical slot i of the new pages; the same
                # copy for every i at once (sources and destinations are disjoint pages)
                i = np.arange(n)
                d = np.asarray(new_page, dtype=np.int64)[i // P] * P + i % P
                sslot = src_slot_of[idx]
                dst[0, d, h, :] = src[0, sslot, h, :]
                dst[1, d, h, :] = src[1, sslot, h, :]
        pt[r, :] = -1
        pt[r, :X] = new_page
        sl[r] = n
    fc -= off
    for r in compacting:
        for p in old_pages[r]:
            fl[fc] = p
            fc += 1
    return new_pool, Tables(pt, sl, fl, fc)


def tail_region(L: int, B: int, P: int):
    """Section 7.2 target-region equations / Algorithm 4 step 1: Y = ceil(L/BS), X = ceil(B/BS),
    Start = (Y - X) * BS, End = Start + B.  Returns (Y, X, Start, End)."""
    Y = -(-int(L) // P)
    X = -(-int(B) // P)
    start = (Y - X) * P
    return Y, X, start, start + int(B)


def copy_pairs_unit(kept, L: int, B: int, P: int):
    """Algorithm 4 steps 1-5 for one keep mask, in logical slots: returns (src, dst), ascending, zipped
    pairwise.  The mask spans every allocated slot (Y * BS of them: the region may reach past L
    into the unused slots of the last block, which are holes)."""
    Y, X, start, end = tail_region(L, B, P)
    keep_mask = np.zeros(Y * P, dtype=bool)
    keep_mask[np.asarray(kept, dtype=np.int64)] = True
    dst_mask = np.zeros(Y * P, dtype=bool)
    dst_mask[start:end] = ~keep_mask[start:end]                    # step 2
    keep_mask[start:end] = False                                   # step 3
    src_mask = keep_mask
    dst = np.nonzero(dst_mask)[0]
    src = np.nonzero(src_mask)[0]
    assert src.shape[0] == dst.shape[0], "as many survivors outside the region as holes inside"
    return src, dst                                                # step 5: Zip(src, dst)


def compact_inplace(pool_bits: np.ndarray, tables: Tables, sel, budget, layers=None):
    """Algorithm 4 / Section 7.2, applied per (layer, KV head) keep mask: survivors outside the last X
    logical blocks move into the holes inside them, then the first Y - X blocks of the request go back
    to the serving system.

      requests r with B_r < L_r: region [Start, End) from `tail_region`; for every layer and head the
      copy pairs of that unit's keep mask (`copy_pairs_unit`), translated through the slot map
      (step 4), all copied at once (step 6; sources and destinations are disjoint);
      then page_table[r] = its last X pages ++ -1.., seq_len[r] = B_r, and, r ascending, the dropped
      pages are pushed on the free list in ascending logical order.
    sel[a][h][r]: ascending kept token indices of pool layer layers[a] (the keep mask as a list).
    Returns (new pool_bits, new Tables, order) where order[a][h][r][i] is the original token index
    of what now sits at logical slot i (None for requests that do not compact).
    """
    P, Hkv = pool_bits.shape[3], pool_bits.shape[4]
    n_pages = pool_bits.shape[2]
    layers = list(range(pool_bits.shape[0])) if layers is None else list(layers)
    new_pool = pool_bits.copy()
    pt = tables.page_table.copy()
    sl = tables.seq_len.copy()
    fl = tables.free_list.copy()
    fc = int(tables.free_count)
    R = len(sl)
    order = [[[None] * R for _ in range(Hkv)] for _ in layers]
    for r in range(R):
        L, B = int(sl[r]), int(budget[r])
        if B >= L:
            continue
        Y, X, start, end = tail_region(L, B, P)
        old = [int(x) for x in tables.page_table[r, :Y]]
        slot_of = slot_map(old, Y * P, P)                          # every allocated slot, used or not
        for a, layer in enumerate(layers):
            before = pool_bits[layer].reshape(2, n_pages * P, Hkv, -1)
            after = new_pool[layer].reshape(2, n_pages * P, Hkv, -1)
            for h in range(Hkv):
                kept = np.asarray(sel[a][h][r], dtype=np.int64)
                assert kept.shape[0] == B
                src, dst = copy_pairs_unit(kept, L, B, P)
                after[:, slot_of[dst], h, :] = before[:, slot_of[src], h, :]
                now = np.arange(start, end)
                now[dst - start] = src
                order[a][h][r] = now
        pt[r, :] = -1
        pt[r, :X] = old[Y - X:]
        sl[r] = B
        for p in old[:Y - X]:
            fl[fc] = p
            fc += 1
    return new_pool, Tables(pt, sl, fl, fc), order


# --------------------------------------------------------------------------------------------
# Section 6.1, Algorithm 2 — confidence monitor and budget update


def token_confidence(logits: np.ndarray, k: int) -> np.ndarray:
    """T_i = -(1/k) sum_{j=1..k} log P_i(j), P_i(j) the j-th largest probability (Section 6.1).

    With P = softmax(z): log P_i(j) = z_(j) - logsumexp(z), so T_i = logsumexp(z) - mean of
    the k largest logits.  float64 throughout.
    """
    z = np.asarray(logits, dtype=np.float64)
    m = z.max(axis=1, keepdims=True)
    lse = m[:, 0] + np.log(np.exp(z - m).sum(axis=1))
    topk = np.sort(z, axis=1)[:, -k:]
    return lse - topk.mean(axis=1)


def trace_confidence(TL: np.ndarray, w: int, s: int, b_percent: float) -> np.ndarray:
    """Sliding-window minimum pooling then bottom-b% selection (Section 6.1).

    R'_m = min TL[m*s : m*s + w], m = 0..floor((Lh - w)/s) (0-based form of the paper's
    1-based window); Q_b = the max(1, ceil(b/100 * M))-th smallest of the M pooled values
    (nearest rank); R = the pooled values <= Q_b in time order.
    """
    TL = np.asarray(TL)
    Lh = TL.shape[0]
    if Lh < w:
        return TL[:0]
    M = (Lh - w) // s + 1
    Rp = np.array([TL[m * s:m * s + w].min() for m in range(M)], dtype=TL.dtype)
    rank = max(1, int(math.ceil(b_percent * M / 100.0)))
    q = np.sort(Rp)[rank - 1]
    return Rp[Rp <= q]


def fit_slope(R: np.ndarray) -> float:
    """Slope of the first-order least-squares fit of R against its position 0..n-1."""
    y = np.asarray(R, dtype=np.float64)
    n = y.shape[0]
    if n < 2:
        return 0.0
    x = np.arange(n, dtype=np.float64)
    xm = x.sum() / n
    ym = y.sum() / n
    return float(((x - xm) * (y - ym)).sum() / ((x - xm) ** 2).sum())


@dataclass
class BudgetParams:
    k: int = 20
    w: int = 64
    s: int = 8
    b_percent: float = 10.0
    scale_up: float = 1.75
    B_upper: int = 30000
    clamp_lo_ppm: int = 0
    clamp_hi_ppm: int = 0


def budget_update(B: int, alpha: float, p: BudgetParams, L: int | None = None) -> int:
    """Algorithm 2 step 4: B' = min(floor(B*scale_up), B_upper) if alpha < 0 else B; then the
    optional integer clamp to [ceil(L*lo/1e6), floor(L*hi/1e6)] (an addition of this build)."""
    Bn = int(B)
    if alpha < 0:
        Bn = min(int(math.floor(float(B) * p.scale_up)), int(p.B_upper))
    if p.clamp_hi_ppm > 0:
        lo = -(-(int(L) * int(p.clamp_lo_ppm)) // 1000000)
        hi = (int(L) * int(p.clamp_hi_ppm)) // 1000000
        Bn = min(max(Bn, lo), hi)
    return Bn


def budget(logits, tok_indptr, hist, hist_len, budget_in, p: BudgetParams, seq_len=None):
    """actkv_budget: append token confidences (stored as float32) to each request's history,
    then trend-detect over the whole history and update the budget (Algorithm 2).

    hist float32 [R, cap], hist_len int [R].  Returns (hist, hist_len, budget_out, slopes,
    T) with T the float64 confidences of the new tokens.
    """
    hist = np.array(hist, dtype=np.float32, copy=True)
    hist_len = np.array(hist_len, dtype=np.int64, copy=True)
    R = len(hist_len)
    n_rows = int(tok_indptr[-1])
    T = token_confidence(logits[:n_rows], p.k) if n_rows > 0 else np.zeros(0)
    out = np.zeros(R, dtype=np.int32)
    slopes = np.zeros(R, dtype=np.float64)
    for r in range(R):
        new = T[tok_indptr[r]:tok_indptr[r + 1]].astype(np.float32)
        room = hist.shape[1] - hist_len[r]
        new = new[:room]
        hist[r, hist_len[r]:hist_len[r] + len(new)] = new
        hist_len[r] += len(new)
        Rr = trace_confidence(hist[r, :hist_len[r]], p.w, p.s, p.b_percent)
        slopes[r] = fit_slope(Rr)
        out[r] = budget_update(int(budget_in[r]), slopes[r], p, None if seq_len is None else int(seq_len[r]))
    return hist, hist_len.astype(np.int32), out, slopes, T
