"""Pins for the oracle's one-shot, block-level prefill (Section 4.2): the prompt is cut into blocks of b tokens, the last
block is the observation window that scores the whole prompt, a block's score is the mean of its tokens' averaged
scores, and Algorithm 1 runs on blocks.  The paper gives neither b nor an example; what can be fixed: the output is
plain causal attention; S and C are the window's column sums and counts; block scores are means; with b = 1 the
blocks are tokens; the score-free rules reproduce the closed forms at block granularity; a prompt that fits is kept
whole; a dictionary restatement on tiny inputs; decoding carries on with the pointer in the right place.
"""
import math

import numpy as np
import pytest

from oracle import RULE_ACCUMULATED, RULE_EVICT_LEFT, RULE_KEEP_LEFT, Oracle


def _prompt(seed, T, Hq, Hkv, d):
    r = np.random.default_rng(seed)
    k = r.standard_normal((1, T, Hkv, d)); k[..., 0] *= 3.0
    return r.standard_normal((1, T, Hq, d)), k, r.standard_normal((1, T, Hkv, d))


def _causal_probs(q, K):
    """[T, T] causal softmax(q K^T / sqrt(d)) for one head."""
    T, d = q.shape
    s = q @ K.T / math.sqrt(d)
    s[np.triu_indices(T, 1)] = -np.inf
    s -= s.max(axis=1, keepdims=True)
    p = np.exp(s)
    return p / p.sum(axis=1, keepdims=True)


def test_output_is_causal_attention_and_scores_come_from_the_window(oracle_lib):
    c, Hq, Hkv, d, T, b = 12, 4, 2, 8, 36, 4
    g = Hq // Hkv
    q, k, v = _prompt(41, T, Hq, Hkv, d)
    o = Oracle(c, Hq, Hkv, d, 1)
    out = o.prefill_oneshot_attend(q, k, v, b)
    for kh in range(Hkv):
        S = np.zeros(T)
        for hh in range(g):
            P = _causal_probs(q[0, :, kh * g + hh], k[0, :, kh])
            np.testing.assert_allclose(out[0, :, kh * g + hh], P @ v[0, :, kh], rtol=1e-11, atol=1e-13)
            S += P[T - b:].sum(axis=0) / g                       # only the window's rows score
        pos, So, Co, sb = o.unit(0, kh)
        np.testing.assert_allclose(So, S, rtol=1e-11)
        want_C = np.where(np.arange(T) < T - b, b, T - np.arange(T))   # window rows that see the token
        assert np.array_equal(Co, want_C) and list(pos) == list(range(T))
    # mass: every window row hands out exactly 1 per KV head
    assert abs(sum(o.unit(0, 0)[1]) - b) < 1e-10


def _brute_force_blocks(sbar, b, cb, rule=None):
    """Blocks as dictionaries; Algorithm 1 on block means."""
    nb = len(sbar) // b
    blocks = [{"first": kb * b, "score": float(np.mean(sbar[kb * b:(kb + 1) * b]))} for kb in range(nb)]
    cache, idx = [], 1
    for blk in blocks:
        cache.append(blk)
        if len(cache) > cb:
            l, r = cache[idx - 1], cache[idx]
            if rule == RULE_KEEP_LEFT:
                loser = r
            elif rule == RULE_EVICT_LEFT:
                loser = l
            else:
                loser = r if l["score"] > r["score"] else l
            cache = [x for x in cache if x is not loser]
            idx = idx % cb + 1
    return [x["first"] + t for x in cache for t in range(b)], idx


@pytest.mark.parametrize("accumulated", [False, True])
@pytest.mark.parametrize("c,b,T", [(12, 4, 36), (16, 2, 70), (8, 8, 40), (6, 1, 31), (12, 3, 12), (12, 3, 9)])
def test_block_tournament_matches_brute_force(oracle_lib, c, b, T, accumulated):
    """`accumulated`: block means of S instead of S / C (Section 4.1 "Importance Score", the criterion also tried)."""
    Hq, Hkv, d = 2, 1, 4
    q, k, v = _prompt(42, T, Hq, Hkv, d)
    o = Oracle(c, Hq, Hkv, d, 1, rule=RULE_ACCUMULATED) if accumulated else Oracle(c, Hq, Hkv, d, 1)
    o.prefill_oneshot_attend(q, k, v, b)
    sbar = o.unit(0, 0)[1].copy() if accumulated else o.unit(0, 0)[3].copy()
    S_before = o.unit(0, 0)[1].copy()
    o.evict_blocks()
    want, idx_b = _brute_force_blocks(sbar, b, c // b)
    pos, S, C, _ = o.unit(0, 0)
    assert list(pos) == want
    assert len(pos) == min(T, c) and np.all(np.diff(pos) > 0)
    np.testing.assert_array_equal(S, S_before[want])                       # scores travel with their tokens
    # whole blocks survive: positions come in runs of b consecutive tokens starting on a block boundary
    assert all(pos[i] % b == 0 and list(pos[i:i + b]) == list(range(pos[i], pos[i] + b)) for i in range(0, len(pos), b))
    assert o.n_seen(0) == T and o.n_evicted(0) == max(0, T - c)
    assert o.idx(0) == (idx_b - 1) * b + 1 == (o.n_evicted(0) % c) + 1


@pytest.mark.parametrize("rule", [RULE_EVICT_LEFT, RULE_KEEP_LEFT])
def test_score_free_rules_give_the_token_level_closed_forms_at_block_granularity(oracle_lib, rule):
    """Each block stands for one token of Algorithm 1: under a score-free rule the retained blocks of a prompt of nb
    blocks are the tokens plain TreeKV with budget c / b retains of an nb-token stream."""
    c, b, T = 32, 4, 33 * 4
    Hq = Hkv = 1; d = 2
    q, k, v = _prompt(43, T, Hq, Hkv, d)
    o = Oracle(c, Hq, Hkv, d, 1, rule=rule)
    o.prefill_oneshot(q, k, v, b)
    tok = Oracle(c // b, 1, 1, d, 1, rule=rule)
    for t in range(T // b):
        tok.decode_step(q[:, t], k[:, t], v[:, t])
    blocks = sorted(set(p // b for p in o.positions(0, 0)))
    assert blocks == list(tok.positions(0, 0))
    assert o.idx(0) == (tok.idx(0) - 1) * b + 1


def test_block_of_one_is_token_level_eviction_with_the_last_querys_weights(oracle_lib):
    """b = 1: the window is the last token, every C is 1, the importance score is the last query's attention weight,
    and the tournament is Algorithm 1's branch repeated on tokens with those frozen scores - what the chunked
    eviction does when it is handed the same scores."""
    c, d, T = 8, 4, 29
    q, k, v = _prompt(44, T, 1, 1, d)
    o = Oracle(c, 1, 1, d, 1)
    o.prefill_oneshot_attend(q, k, v, 1)
    pos, S, C, sb = o.unit(0, 0)
    P = _causal_probs(q[0, :, 0], k[0, :, 0])
    np.testing.assert_allclose(sb, P[-1], rtol=1e-11)
    assert np.all(C == 1)
    o.evict_blocks()
    # the same frozen scores through a plain token-level loop
    cache, idx = [], 1
    for t in range(T):
        cache.append(t)
        if len(cache) > c:
            l, r = cache[idx - 1], cache[idx]
            cache.remove(r if P[-1][l] > P[-1][r] else l)
            idx = idx % c + 1
    assert list(o.positions(0, 0)) == cache and o.idx(0) == idx


def test_prompt_that_fits_is_kept_whole_and_decoding_carries_on(oracle_lib):
    c, Hq, Hkv, d, b = 16, 2, 2, 4, 4
    q, k, v = _prompt(45, 12, Hq, Hkv, d)
    o = Oracle(c, Hq, Hkv, d, 1)
    o.prefill_oneshot(q, k, v, b)
    assert list(o.positions(0, 0)) == list(range(12)) and o.idx(0) == 1 and o.n_evicted(0) == 0
    r = np.random.default_rng(46)
    C0 = o.unit(0, 0)[2].copy()
    for t in range(12):
        o.decode_step(r.standard_normal((1, Hq, d)), r.standard_normal((1, Hkv, d)), r.standard_normal((1, Hkv, d)))
        pos, S, C, sb = o.unit(0, 0)
        assert len(pos) == min(13 + t, c) and np.all(np.diff(pos) > 0) and np.all(sb > 0) and np.all(sb <= 1 + 1e-12)
    # counters of the prompt's surviving tokens went on from the window's counts, one per decode step they were cached
    pos, S, C, sb = o.unit(0, 0)
    for p_, c_ in zip(pos, C):
        if p_ < 12:
            assert c_ == C0[p_] + 12
    assert o.n_evicted(0) == 24 - 16 and o.idx(0) == (o.n_evicted(0) % c) + 1


def test_oneshot_then_decode_continues_algorithm_1_at_the_right_pointer(oracle_lib):
    """After a compressing one-shot prefill the token-level pointer stands on the first token of the block the block
    pointer stood on; under the evict-left rule the following decode steps must evict exactly those slots."""
    c, b, T, d = 12, 3, 45, 2
    q, k, v = _prompt(47, T, 1, 1, d)
    o = Oracle(c, 1, 1, d, 1, rule=RULE_EVICT_LEFT)
    o.prefill_oneshot(q, k, v, b)
    r = np.random.default_rng(48)
    for t in range(2 * c):
        before = list(o.positions(0, 0))
        idx = o.idx(0)
        o.decode_step(r.standard_normal((1, 1, d)), r.standard_normal((1, 1, d)), r.standard_normal((1, 1, d)))
        after = list(o.positions(0, 0))
        assert after == before[:idx - 1] + before[idx:] + [T + t]      # slot idx (1-based) left, the new token joined
        assert o.idx(0) == idx % c + 1


def test_bad_arguments_are_refused(oracle_lib):
    q, k, v = _prompt(49, 10, 1, 1, 2)
    o = Oracle(8, 1, 1, 2, 1)
    with pytest.raises(ValueError):
        o.prefill_oneshot_attend(q, k, v, 4)              # 10 is not a multiple of 4
    with pytest.raises(ValueError):
        o.prefill_oneshot_attend(q[:, :9], k[:, :9], v[:, :9], 3)   # 8 is not a multiple of 3
    o.prefill_oneshot(q[:, :8], k[:, :8], v[:, :8], 4)
    with pytest.raises(ValueError):
        o.prefill_oneshot_attend(q[:, :8], k[:, :8], v[:, :8], 4)   # the cache is no longer empty
