"""Pins for the oracle's sink / recent-window protection (Section 5.2: a cache of 1024 split into 4 initial,
508 recent and 512 method-chosen tokens).  The paper gives the split, not the mechanics; the reading under test is stated in
the oracle's header.  What can be fixed without the CUDA library: nothing changes without protection; protected
tokens are never evicted; the middle region is plain TreeKV on the delayed sub-stream (closed forms of the
score-free rules carry over); a dictionary-based restatement on tiny inputs; the paper's 4 / 508 / 512 split.
"""
import math

import numpy as np
import pytest

from oracle import RULE_EVICT_LEFT, RULE_KEEP_LEFT, Oracle


def _stream(seed, T, Hq, Hkv, d, B=1):
    r = np.random.default_rng(seed)
    k = r.standard_normal((T, B, Hkv, d))
    k[..., 0] *= 4.0
    return r.standard_normal((T, B, Hq, d)), k, r.standard_normal((T, B, Hkv, d))


def test_no_protection_is_algorithm_1_unchanged(oracle_lib):
    c, Hq, Hkv, d, T = 6, 4, 2, 4, 40
    q, k, v = _stream(1, T, Hq, Hkv, d)
    a = Oracle(c, Hq, Hkv, d, 1)
    b = Oracle(c, Hq, Hkv, d, 1, n_sink=0, n_recent=0)
    for t in range(T):
        oa = a.decode_step(q[t], k[t], v[t]); ob = b.decode_step(q[t], k[t], v[t])
        assert np.array_equal(oa, ob)
        for kh in range(Hkv):
            assert np.array_equal(a.unit(0, kh)[1], b.unit(0, kh)[1]) and list(a.positions(0, kh)) == list(b.positions(0, kh))


@pytest.mark.parametrize("c,ns,nr", [(8, 1, 2), (12, 2, 5), (16, 4, 4), (9, 0, 3), (9, 3, 0)])
def test_protected_tokens_are_never_evicted_and_invariants_hold(oracle_lib, c, ns, nr):
    Hq, Hkv, d, T = 2, 2, 4, 6 * c + 5
    cm = c - ns - nr
    q, k, v = _stream(2, T, Hq, Hkv, d)
    o = Oracle(c, Hq, Hkv, d, 1, n_sink=ns, n_recent=nr)
    for t in range(T):
        o.decode_step(q[t], k[t], v[t])
        n = t + 1
        for kh in range(Hkv):
            pos, S, C, sb = o.unit(0, kh)
            assert len(pos) == min(n, c) and np.all(np.diff(pos) > 0)
            assert np.array_equal(C, n - pos)                                   # counters advance from arrival
            if n > c:
                assert list(pos[:ns]) == list(range(ns))                       # sinks stay
                assert list(pos[c - nr:]) == list(range(n - nr, n))            # the newest nr stay
                assert np.all(pos[ns:c - nr] >= ns) and np.all(pos[ns:c - nr] < n - nr)
        assert o.n_evicted(0) == max(0, n - c)
        assert o.idx(0) == (o.n_evicted(0) % cm) + 1                            # idx cycles over the middle region only


@pytest.mark.parametrize("rule", [RULE_EVICT_LEFT, RULE_KEEP_LEFT])
@pytest.mark.parametrize("c,ns,nr", [(12, 2, 2), (14, 1, 5), (20, 4, 8)])
def test_middle_region_is_plain_treekv_on_the_delayed_substream(oracle_lib, rule, c, ns, nr):
    """Under a score-free rule the retained set is a function of the schedule alone.  The tokens between the sinks
    and the recent window must then be exactly what plain TreeKV with budget c - ns - nr retains of the stream
    ns, ns+1, ..., delayed by nr steps - so the closed forms pinned for the unprotected cache carry over."""
    Hq = Hkv = 1
    d = 2
    cm = c - ns - nr
    T = 7 * c + 3
    q, k, v = _stream(3, T, Hq, Hkv, d)
    o = Oracle(c, Hq, Hkv, d, 1, rule=rule, n_sink=ns, n_recent=nr)
    plain = Oracle(cm, Hq, Hkv, d, 1, rule=rule)
    fed = 0
    for t in range(T):
        o.decode_step(q[t], k[t], v[t])
        n = t + 1
        want_fed = max(0, n - ns - nr)       # tokens that have left the recent window (and are not sinks)
        while fed < want_fed:
            plain.decode_step(q[fed], k[fed], v[fed])
            fed += 1
        if n > c:
            mid = o.positions(0, 0)[ns:c - nr]
            assert list(mid) == [ns + p for p in plain.positions(0, 0)], (t, list(mid))
            assert o.idx(0) == plain.idx(0)


def _brute_force(q, k, v, c, ns, nr):
    """Dictionary restatement for one head: tokens are dicts; the scope is found by counting, not by index
    arithmetic shared with the oracle."""
    d = q.shape[-1]
    cache, idx, outs, history = [], 1, [], []
    for t in range(q.shape[0]):
        cache.append({"pos": t, "k": k[t], "v": v[t], "S": 0.0, "C": 0})
        s = np.array([q[t] @ e["k"] for e in cache]) / math.sqrt(d)
        p = np.exp(s - s.max()); p /= p.sum()
        outs.append(sum(pi * e["v"] for pi, e in zip(p, cache)))
        for pi, e in zip(p, cache):
            e["S"] += pi; e["C"] += 1
        if len(cache) > c:
            eligible = cache[ns:len(cache) - nr]            # everything but the sinks and the nr newest
            assert len(eligible) == c - ns - nr + 1
            left, right = eligible[idx - 1], eligible[idx]
            loser = right if left["S"] / left["C"] > right["S"] / right["C"] else left
            cache = [e for e in cache if e is not loser]
            idx = idx % (c - ns - nr) + 1
        history.append([e["pos"] for e in cache])
    return np.array(outs), history


@pytest.mark.parametrize("c,ns,nr", [(6, 1, 2), (8, 2, 2), (7, 0, 4)])
def test_matches_brute_force_on_tiny_inputs(oracle_lib, c, ns, nr):
    d, T = 4, 40
    q, k, v = _stream(4, T, 1, 1, d)
    o = Oracle(c, 1, 1, d, 1, n_sink=ns, n_recent=nr)
    outs, hist = _brute_force(q[:, 0, 0], k[:, 0, 0], v[:, 0, 0], c, ns, nr)
    for t in range(T):
        out = o.decode_step(q[t], k[t], v[t])
        np.testing.assert_allclose(out[0, 0], outs[t], rtol=1e-12, atol=1e-14)
        assert list(o.positions(0, 0)) == hist[t], t


def test_chunked_prefill_with_protection_equals_token_by_token_under_score_free_rules(oracle_lib):
    c, ns, nr, d = 14, 2, 4, 2
    for rule in (RULE_EVICT_LEFT, RULE_KEEP_LEFT):
        for m in (1, 3, 8, 11, 30):
            T = 5 * c
            q, k, v = _stream(5, T, 1, 1, d)
            a = Oracle(c, 1, 1, d, 1, rule=rule, n_sink=ns, n_recent=nr)
            b = Oracle(c, 1, 1, d, 1, rule=rule, n_sink=ns, n_recent=nr)
            t = 0
            while t < T:
                mm = min(m, T - t)
                for s in range(t, t + mm):
                    a.decode_step(q[s], k[s], v[s])
                b.prefill_chunk(q[t:t + mm].transpose(1, 0, 2, 3), k[t:t + mm].transpose(1, 0, 2, 3),
                                v[t:t + mm].transpose(1, 0, 2, 3))
                t += mm
                assert list(a.positions(0, 0)) == list(b.positions(0, 0)), (rule, m, t)
                assert a.idx(0) == b.idx(0)


def test_the_papers_split_4_508_512(oracle_lib):
    """Section 5.2: a cache of 1024 = 4 initial + 508 recent + 512 selected tokens."""
    c, ns, nr, d, T = 1024, 4, 508, 2, 1024 + 700
    r = np.random.default_rng(6)
    o = Oracle(c, 1, 1, d, 1, n_sink=ns, n_recent=nr)
    q = r.standard_normal((T, 1, 1, d)); k = r.standard_normal((T, 1, 1, d)); v = r.standard_normal((T, 1, 1, d))
    o.prefill_chunk(q[:1024].transpose(1, 0, 2, 3), k[:1024].transpose(1, 0, 2, 3), v[:1024].transpose(1, 0, 2, 3))
    o.prefill_chunk(q[1024:].transpose(1, 0, 2, 3), k[1024:].transpose(1, 0, 2, 3), v[1024:].transpose(1, 0, 2, 3))
    pos = o.positions(0, 0)
    assert len(pos) == 1024 and list(pos[:4]) == [0, 1, 2, 3] and list(pos[-508:]) == list(range(T - 508, T))
    mid = pos[4:516]
    assert len(mid) == 512 and mid.min() >= 4 and mid.max() < T - 508 and np.all(np.diff(mid) > 0)
    assert o.idx(0) == (700 % 512) + 1


def test_bad_protection_is_refused(oracle_lib):
    with pytest.raises(ValueError):
        Oracle(8, 1, 1, 2, 1, n_sink=3, n_recent=4)      # one slot left: no room for a scope
