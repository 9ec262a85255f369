"""Pins for the oracle's streaming (one action query per call, LSE supplied) score update
(Section 7.1, Algorithm 3 as triggered per decode step)."""
import math

import numpy as np
import torch

from oracle import actkv_oracle as O


def _unit(rng, W, G, L, D):
    return rng.standard_normal((W, G, D)), rng.standard_normal((L, D))


def _decode_lse(q, k, scale):
    """LSE each decode step's attention would hand over: query w sees the first L-W+w+1 keys."""
    W, G, _ = q.shape
    L = k.shape[0]
    lse = np.zeros((W, G))
    for w in range(W):
        for g in range(G):
            s = scale * (k[: L - W + w + 1] @ q[w, g])
            lse[w, g] = math.log(sum(math.exp(x) for x in s.tolist()))
    return lse


def test_single_step_is_a_softmax_row_maxed_over_the_group():
    rng = np.random.default_rng(0)
    q, k = _unit(rng, 1, 3, 40, 16)
    scale = 0.25
    lse = _decode_lse(q, k, scale)
    out = O.score_stream_step(np.zeros(0), 0, q[0], k, lse[0], scale)
    probs = torch.softmax(torch.from_numpy(scale * (q[0] @ k.T)), dim=-1).numpy()      # textbook softmax per head
    assert np.allclose(out, probs.max(axis=0), rtol=1e-12, atol=0)


def test_streaming_equals_the_batch_definition_with_the_causal_window():
    """Feeding the action queries one decode step at a time, the cache growing by one key per step,
    reproduces the pooled score of the whole window (mean over action tokens of the max over the
    group, keys not yet cached counting as zero)."""
    rng = np.random.default_rng(1)
    for (W, G, L, D) in [(1, 1, 5, 8), (7, 4, 60, 16), (12, 2, 12, 8)]:
        q, k = _unit(rng, W, G, L, D)
        scale = 1.0 / math.sqrt(D)
        batch, lse = O.score_unit(q, k, scale, causal=True)
        assert np.allclose(lse, _decode_lse(q, k, scale), rtol=1e-12)
        stream = O.score_stream(q, k, scale, lse)
        assert np.allclose(stream, batch.astype(np.float64), rtol=1e-6, atol=1e-12)    # batch is rounded to float32
        # the newest key was seen by the last query only
        last = np.exp(scale * (k[-1] @ q[-1].T) - lse[-1]).max() / W
        assert math.isclose(stream[-1], last, rel_tol=1e-12)


def test_running_mean_is_the_plain_mean_and_splits_anywhere():
    rng = np.random.default_rng(2)
    W, G, L, D = 9, 2, 50, 8
    q, k = _unit(rng, W, G, L, D)
    scale = 0.3
    lse = _decode_lse(q, k, scale)
    whole = O.score_stream(q, k, scale, lse)
    # plain mean of the per-step max-pooled probabilities, zeros where the key did not exist yet
    per_step = np.zeros((W, L))
    for w in range(W):
        n = L - W + w + 1
        per_step[w, :n] = np.exp(scale * (q[w] @ k[:n].T) - lse[w][:, None]).max(axis=0)
    assert np.allclose(whole, per_step.mean(axis=0), rtol=1e-12, atol=1e-15)
    # two calls (5 queries, then 4 more with the state carried) give the same state
    first = O.score_stream(q[:5], k[: L - 4], scale, lse[:5])
    both = O.score_stream(q[5:], k, scale, lse[5:], out_prev=first, n_prev=5)
    assert np.allclose(both, whole, rtol=1e-12, atol=1e-15)


def test_state_restarts_from_zero_at_region_entry():
    rng = np.random.default_rng(3)
    q, k = _unit(rng, 3, 2, 20, 8)
    lse = _decode_lse(q, k, 0.5)
    junk = rng.random(17)
    a = O.score_stream_step(junk, 0, q[0], k[:18], lse[0], 0.5)          # n_prev = 0: what was there is dropped
    b = O.score_stream_step(np.zeros(0), 0, q[0], k[:18], lse[0], 0.5)
    assert np.array_equal(a, b)


def test_mass_of_one_step_lies_between_one_and_group_size():
    rng = np.random.default_rng(4)
    q, k = _unit(rng, 1, 4, 300, 16)
    lse = _decode_lse(q, k, 0.25)
    out = O.score_stream_step(np.zeros(0), 0, q[0], k, lse[0], 0.25)
    assert 1.0 - 1e-12 <= out.sum() <= 4.0 + 1e-12
    same = np.repeat(q[:, :1], 4, axis=1)                                # identical heads: exactly one softmax row
    lse_s = _decode_lse(same, k, 0.25)
    assert math.isclose(O.score_stream_step(np.zeros(0), 0, same[0], k, lse_s[0], 0.25).sum(), 1.0, rel_tol=1e-12)
