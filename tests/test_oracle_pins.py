"""Pins for the fp64 oracle: what the paper and the mathematics fix, checked without the CUDA library.

Each test names the passage it rests on.  A plausible mistake in the oracle (a
dropped term, a wrong index, a transposed operand, a wrong schedule) fails at
least one of them.
"""
import math
import os

import numpy as np
import pytest

from oracle import IDX_LITERAL, RULE_ACCUMULATED, RULE_EVICT_LEFT, RULE_KEEP_LEFT, RULE_SCORES, Oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _stream(seed, T, Hq, Hkv, d, B=1, peaked=False):
    r = _rng(seed)
    q = r.standard_normal((T, B, Hq, d))
    k = r.standard_normal((T, B, Hkv, d))
    v = r.standard_normal((T, B, Hkv, d))
    if peaked:
        k[..., 0] *= 4.0
    return q, k, v


def _softmax_attention(q, K, V):
    """Textbook softmax(q K^T / sqrt(d)) V (Section 3.1) with numpy; q [d], K,V [n,d]."""
    s = K @ q / math.sqrt(q.shape[0])
    s = s - s.max()
    p = np.exp(s)
    p /= p.sum()
    return p @ V, p


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = [x.strip() for x in line.split("=")]
            out[key] = [int(x) for x in val.split()]
    return out


# ---------------------------------------------------------------------------------------------
# Section 4.1 "Overall Idea": fixed cache size; order of Figure 3 preserved
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("c,Hq,Hkv", [(4, 1, 1), (8, 4, 2), (16, 2, 2)])
def test_budget_and_order_invariants(oracle_lib, c, Hq, Hkv):
    T, d, B = 5 * c + 3, 8, 2
    q, k, v = _stream(1, T, Hq, Hkv, d, B)
    o = Oracle(c, Hq, Hkv, d, B)
    for t in range(T):
        o.decode_step(q[t], k[t], v[t])
        for b in range(B):
            assert o.n_seen(b) == t + 1
            for kh in range(Hkv):
                pos, S, C, sb = o.unit(b, kh)
                assert len(pos) == min(t + 1, c)                       # never above budget
                assert np.all(np.diff(pos) > 0)                        # strictly increasing
                assert np.array_equal(C, (t + 1) - pos)                # C_j = N_seen - pos_j
                assert np.all(sb > 0) and np.all(sb <= 1 + 1e-12)      # averaged weight in (0,1]
            assert o.idx(b) == (o.n_evicted(b) % c) + 1                # idx cycles 1..c
            assert o.n_evicted(b) == max(0, t + 1 - c)


# ---------------------------------------------------------------------------------------------
# Algorithm 1: no eviction while length <= c, so the output is full causal attention (Section 3.1)
# ---------------------------------------------------------------------------------------------
def test_short_stream_equals_full_attention(oracle_lib):
    c, Hq, Hkv, d, T = 12, 4, 2, 16, 12
    g = Hq // Hkv
    q, k, v = _stream(2, T, Hq, Hkv, d)
    o = Oracle(c, Hq, Hkv, d, 1)
    for t in range(T):
        out = o.decode_step(q[t], k[t], v[t])
        for h in range(Hq):
            ref, _ = _softmax_attention(q[t, 0, h], k[: t + 1, 0, h // g], v[: t + 1, 0, h // g])
            np.testing.assert_allclose(out[0, h], ref, rtol=1e-12, atol=1e-12)
        assert o.n_evicted(0) == 0
    assert list(o.positions(0, 0)) == list(range(T))


# ---------------------------------------------------------------------------------------------
# Algorithm 1 on tiny inputs: output = brute-force attention restricted to retained(t-1) + {t}
# ---------------------------------------------------------------------------------------------
def test_output_is_attention_over_retained_set(oracle_lib):
    c, Hq, Hkv, d, T = 6, 2, 1, 4, 40
    q, k, v = _stream(3, T, Hq, Hkv, d, peaked=True)
    o = Oracle(c, Hq, Hkv, d, 1)
    retained = []
    for t in range(T):
        out = o.decode_step(q[t], k[t], v[t])
        vis = retained + [t]
        for h in range(Hq):
            ref, _ = _softmax_attention(q[t, 0, h], k[vis, 0, 0], v[vis, 0, 0])
            np.testing.assert_allclose(out[0, h], ref, rtol=1e-11, atol=1e-12)
        retained = list(o.positions(0, 0))
        assert len(retained) <= c


def _brute_force_treekv(q, k, v, c, accumulated=False):
    """Independent restatement for one head: dictionaries keyed by token, scores from their definition.

    Averaged attention weight of token j at step t (Section 4.1 "Importance Score"): the mean, over the
    steps since j arrived, of the attention weight j received.  `accumulated`: the sum instead of the mean
    (the accumulated attention weight the same paragraph names as a criterion that was also tried).
    """
    T, d = q.shape
    received = {}          # token -> list of weights received, one per step present
    cache = []             # retained tokens, ascending
    idx = 1
    history = []
    for t in range(T):
        cache.append(t)
        received[t] = []
        _, p = _softmax_attention(q[t], k[cache], v[cache])
        for w, j in zip(p, cache):
            received[j].append(w)
        if len(cache) > c:
            a, b = cache[idx - 1], cache[idx]
            sa = sum(received[a]) / (1 if accumulated else len(received[a]))
            sb = sum(received[b]) / (1 if accumulated else len(received[b]))
            cache.remove(b if sa > sb else a)
            idx = idx % c + 1
        history.append(list(cache))
    return history


def test_matches_brute_force_on_tiny_inputs(oracle_lib):
    for seed, c in [(11, 4), (12, 5), (13, 8)]:
        T, d = 37, 4
        q, k, v = _stream(seed, T, 1, 1, d, peaked=True)
        hist = _brute_force_treekv(q[:, 0, 0], k[:, 0, 0], v[:, 0, 0], c)
        o = Oracle(c, 1, 1, d, 1)
        for t in range(T):
            o.decode_step(q[t], k[t], v[t])
            assert list(o.positions(0, 0)) == hist[t], (seed, c, t)


def test_accumulated_criterion_matches_brute_force_and_differs_from_the_average(oracle_lib):
    """Section 4.1 "Importance Score": accumulated attention weights as the criterion, S in place of S / C."""
    differs = False
    for seed, c in [(11, 4), (12, 5), (13, 8)]:
        T, d = 37, 4
        q, k, v = _stream(seed, T, 1, 1, d, peaked=True)
        hist = _brute_force_treekv(q[:, 0, 0], k[:, 0, 0], v[:, 0, 0], c, accumulated=True)
        hist_avg = _brute_force_treekv(q[:, 0, 0], k[:, 0, 0], v[:, 0, 0], c)
        o = Oracle(c, 1, 1, d, 1, rule=RULE_ACCUMULATED)
        for t in range(T):
            o.decode_step(q[t], k[t], v[t])
            assert list(o.positions(0, 0)) == hist[t], (seed, c, t)
        differs |= hist[-1] != hist_avg[-1]
    assert differs   # the inputs tell the two criteria apart


def test_accumulated_criterion_under_uniform_attention_is_the_keep_left_ladder(oracle_lib):
    """With q = 0 every cached token receives 1 / len in every step, so of two tokens the older one has the strictly
    larger accumulated weight and the left member of every scope survives: the retained set is the closed form of the
    keep-left ablation (c = 8, 64 tokens: 1, 41, 49, 53, 57, 59, 61, 63).  The averaged criterion sees exact ties for
    tokens that arrived after the fill instead and ends elsewhere."""
    c, T, d = 8, 64, 2
    _, k, v = _stream(10, T, 1, 1, d)
    q = np.zeros((T, 1, 1, d))
    o = Oracle(c, 1, 1, d, 1, rule=RULE_ACCUMULATED)
    a = Oracle(c, 1, 1, d, 1, rule=RULE_SCORES)
    for t in range(T):
        o.decode_step(q[t], k[t], v[t])
        a.decode_step(q[t], k[t], v[t])
    assert list(o.positions(0, 0) + 1) == [1, 41, 49, 53, 57, 59, 61, 63]
    assert list(a.positions(0, 0)) != list(o.positions(0, 0))


# ---------------------------------------------------------------------------------------------
# Worked example: Section 4.1 "Eviction Scope" with the caption of Figure 3 (c = 4, 17 tokens)
# ---------------------------------------------------------------------------------------------
def test_worked_example_fig3(oracle_lib):
    gold = _read_golden("fig3_worked_example.txt")
    c, T = gold["c"][0], gold["T"][0]
    d = 4
    # token 2 (1-based) gets a key every query likes; token 1 gets one every query dislikes
    q = np.zeros((T, 1, 1, d)); q[..., 0] = 3.0
    k = _rng(5).standard_normal((T, 1, 1, d)) * 0.1
    v = _rng(6).standard_normal((T, 1, 1, d))
    k[0, 0, 0, 0] = -3.0
    k[1, 0, 0, 0] = 3.0
    o = Oracle(c, 1, 1, d, 1)
    idx_seen = {}
    for step in range(1, T + 1):
        idx_before = o.idx(0)
        before = [p + 1 for p in o.positions(0, 0)] + [step]
        o.decode_step(q[step - 1], k[step - 1], v[step - 1])
        after = [p + 1 for p in o.positions(0, 0)]
        if step < gold["first_eviction_step"][0]:
            assert after == list(range(1, step + 1)) and o.n_evicted(0) == 0
        else:
            idx_seen[step] = idx_before
            evicted = (set(before) - set(after)).pop()
            assert evicted in (before[idx_before - 1], before[idx_before])       # scope {idx, idx+1}
        if step == 5:
            assert after == gold["cache_after_step_5"]
        if step == 17:
            assert before[0] == gold["slot1_token_at_step_17"][0]
            assert evicted == before[gold["evicted_slot_at_step_17"][0] - 1]
            assert after[0] == gold["slot1_token_at_step_17"][0]
    assert idx_seen[5] == gold["idx_at_step_5"][0]
    assert [idx_seen[s] for s in (5, 6, 7, 8)] == gold["idx_sequence_steps_5_to_8"]
    assert idx_seen[17] == gold["idx_at_step_17"][0]
    for step in range(5, T + 1):
        assert idx_seen[step] == ((step - c - 1) % c) + 1


def test_printed_idx_formula_skips_slots(oracle_lib):
    """The update as printed in Algorithm 1 cannot be what Section 4.1's prose describes: for even c it
    never visits even slots.  The oracle keeps it only as a documented switch."""
    c, d, T = 4, 4, 20
    q, k, v = _stream(7, T, 1, 1, d)
    o = Oracle(c, 1, 1, d, 1, idx_mode=IDX_LITERAL)
    seen = set()
    for t in range(T):
        if t >= c:
            seen.add(o.idx(0))
        o.decode_step(q[t], k[t], v[t])
    assert seen == {1, 3}


# ---------------------------------------------------------------------------------------------
# Tree shape (Sections 1, 3.3, 4.1: sparse on the left, dense on the right) via score-free rules
# ---------------------------------------------------------------------------------------------
def _evict_left_offsets(c):
    """Closed form for the rule 'always evict slot idx' once T is a multiple of c and the cache has cycled:
    offsets r_j = (T-1) - pos_j satisfy r_j = 2(c-j) for j > c/2 and r_j = r_{2j} + c for j <= c/2 (1-based
    slot j).  One cycle of c evictions keeps every second element of [cache | next c tokens]; that is this
    recurrence."""
    r = [0] * (c + 1)
    for j in range(c, 0, -1):
        r[j] = 2 * (c - j) if j > c // 2 else r[2 * j] + c
    return r[1:]


@pytest.mark.parametrize("c", [4, 8, 16, 64])
def test_evict_left_closed_form(oracle_lib, c):
    d = 2
    cycles = int(math.log2(c)) + 3
    T = c * (cycles + 1)
    q, k, v = _stream(8, T, 1, 1, d)
    o = Oracle(c, 1, 1, d, 1, rule=RULE_EVICT_LEFT)
    for t in range(T):
        o.decode_step(q[t], k[t], v[t])
        if t >= 3 * c:
            gaps = np.diff(o.positions(0, 0))
            assert np.all(np.diff(gaps) <= 0), (t, gaps)     # gaps never grow towards the recent end
    offs = (T - 1) - o.positions(0, 0)
    assert list(offs) == _evict_left_offsets(c)
    assert offs[0] == c * int(math.log2(c))                  # the span of the tree is c log2 c


def test_evict_left_known_vectors(oracle_lib):
    """Spelled-out instances of the closed form (offsets of the retained tokens from the newest one)."""
    expect = {
        4: [8, 4, 2, 0],
        8: [24, 16, 12, 8, 6, 4, 2, 0],
        16: [64, 48, 40, 32, 28, 24, 20, 16, 14, 12, 10, 8, 6, 4, 2, 0],
    }
    for c, offs in expect.items():
        assert _evict_left_offsets(c) == offs
        T = c * 8
        q, k, v = _stream(9, T, 1, 1, 2)
        o = Oracle(c, 1, 1, 2, 1, rule=RULE_EVICT_LEFT)
        for t in range(T):
            o.decode_step(q[t], k[t], v[t])
        assert list((T - 1) - o.positions(0, 0)) == offs


def test_keep_left_ablation(oracle_lib):
    """Section 5.4 ablation (always keep the left token): token 1 stays forever; c=8, T=64 retains
    tokens 1,41,49,53,57,59,61,63 (1-based) - a binary ladder towards the recent end."""
    c, T = 8, 64
    q, k, v = _stream(10, T, 1, 1, 2)
    o = Oracle(c, 1, 1, 2, 1, rule=RULE_KEEP_LEFT)
    for t in range(T):
        o.decode_step(q[t], k[t], v[t])
        assert o.positions(0, 0)[0] == 0
    assert list(o.positions(0, 0) + 1) == [1, 41, 49, 53, 57, 59, 61, 63]


def test_cycle_is_a_tournament_over_disjoint_pairs(oracle_lib):
    """Within c consecutive evictions the scopes are the disjoint pairs (2i-1, 2i) of
    [cache at cycle start | next c tokens]: the tree of Figure 3."""
    c, d = 8, 4
    T = c * 5
    q, k, v = _stream(14, T, 2, 1, d, peaked=True)
    o = Oracle(c, 2, 1, d, 1)
    t = 0
    for _ in range(c):
        o.decode_step(q[t], k[t], v[t]); t += 1
    for cycle in range(4):
        start = list(o.positions(0, 0))
        universe = start + list(range(t, t + c))
        for i in range(c):
            before = list(o.positions(0, 0)) + [t]
            o.decode_step(q[t], k[t], v[t]); t += 1
            evicted = (set(before) - set(o.positions(0, 0))).pop()
            assert evicted in (universe[2 * i], universe[2 * i + 1])
        after = list(o.positions(0, 0))
        for i in range(c):
            assert after[i] in (universe[2 * i], universe[2 * i + 1])


# ---------------------------------------------------------------------------------------------
# Score bookkeeping (Algorithm 1, the C and S updates)
# ---------------------------------------------------------------------------------------------
def test_mass_conservation_decode_and_chunks(oracle_lib):
    """Softmax rows sum to one, so each call adds exactly (number of query rows) to the sum of S over a
    KV head, counting evicted mass; with the group mean this holds for any group size."""
    c, Hq, Hkv, d = 8, 4, 2, 8
    r = _rng(15)
    o = Oracle(c, Hq, Hkv, d, 1)
    # decode steps
    for t in range(6):
        before = [o.unit(0, kh)[1].sum() for kh in range(Hkv)]
        o.decode_attend(r.standard_normal((1, Hq, d)), r.standard_normal((1, Hkv, d)), r.standard_normal((1, Hkv, d)))
        for kh in range(Hkv):
            assert abs(o.unit(0, kh)[1].sum() - before[kh] - 1.0) < 1e-12
        o.evict()
    for m in (1, 3, 5, 11):
        before = [o.unit(0, kh)[1].sum() for kh in range(Hkv)]
        o.prefill_attend(r.standard_normal((1, m, Hq, d)), r.standard_normal((1, m, Hkv, d)), r.standard_normal((1, m, Hkv, d)))
        for kh in range(Hkv):
            pos, S, C, _ = o.unit(0, kh)
            assert abs(S.sum() - before[kh] - m) < 1e-11
            assert np.array_equal(C, o.n_seen(0) - pos)
        o.evict()
        assert o.length(0, 0) == min(c, o.n_seen(0))


def test_new_token_score_is_its_self_attention(oracle_lib):
    """Algorithm 1: the new slot enters with S=0, C=0 and both are advanced in the same step, so its
    first averaged score is its own attention weight."""
    c, d = 4, 4
    r = _rng(16)
    o = Oracle(c, 1, 1, d, 1)
    ks, vs = [], []
    for t in range(3):
        q = r.standard_normal((1, 1, d)); k = r.standard_normal((1, 1, d)); v = r.standard_normal((1, 1, d))
        ks.append(k[0, 0]); vs.append(v[0, 0])
        o.decode_attend(q, k, v)
        _, p = _softmax_attention(q[0, 0], np.array(ks), np.array(vs))
        pos, S, C, sb = o.unit(0, 0)
        assert C[-1] == 1 and abs(sb[-1] - p[-1]) < 1e-14


def test_strict_comparison_tie_evicts_left(oracle_lib):
    """Algorithm 1 compares with a strict '>': on an exact tie slot idx (the left one) goes.  With q = 0
    every weight is exactly 1/(c+1) once the cache is full; for c = 3 that is 0.25, sums of it are exact in
    binary floating point, so tokens that arrived after the fill tie exactly."""
    c, d = 3, 2
    o = Oracle(c, 1, 1, d, 1)
    z = np.zeros((1, 1, d))
    ties = 0
    for t in range(40):
        o.decode_attend(z, z, z)
        pos, S, C, sb = o.unit(0, 0)
        if len(pos) > c:
            i = o.idx(0)
            tie = sb[i - 1] == sb[i]
            o.evict()
            evicted = (set(pos) - set(o.positions(0, 0))).pop()
            if tie:
                ties += 1
                assert evicted == pos[i - 1]
                assert o.last_near_ties == 1 and o.last_min_gap == 0.0
            else:
                assert evicted == (pos[i] if sb[i - 1] > sb[i] else pos[i - 1])
        else:
            o.evict()
    assert ties >= 20


def test_hand_computed_scores(oracle_lib):
    """Three steps with q = 0 worked by hand: weights are 1, then 1/2 each, then 1/3 each."""
    d = 2
    o = Oracle(2, 1, 1, d, 1)
    z = np.zeros((1, 1, d))
    o.decode_step(z, z, z)
    o.decode_step(z, z, z)
    o.decode_attend(z, z, z)
    pos, S, C, sb = o.unit(0, 0)
    np.testing.assert_allclose(sb, [(1.5 + 1 / 3) / 3, (0.5 + 1 / 3) / 2, 1 / 3], rtol=1e-15)
    assert list(C) == [3, 2, 1]
    o.evict()                                  # idx = 1: scope (token 0, token 1), 11/18 > 5/12: token 1 goes
    assert list(o.positions(0, 0)) == [0, 2]
    assert o.idx(0) == 2
    # a causal chunk with q = 0: row i spreads 1/(i+1) over tokens 0..i
    o = Oracle(8, 1, 1, d, 1)
    zc = np.zeros((1, 4, 1, d))
    o.prefill_chunk(zc, zc, zc)
    pos, S, C, sb = o.unit(0, 0)
    np.testing.assert_allclose(S, [1 + 1 / 2 + 1 / 3 + 1 / 4, 1 / 2 + 1 / 3 + 1 / 4, 1 / 3 + 1 / 4, 1 / 4], rtol=1e-15)
    assert list(C) == [4, 3, 2, 1]


def test_gqa_group_mean_reduces_to_mha(oracle_lib):
    """With identical queries in a group the group mean equals the single-head weight, so a (Hq=4,Hkv=1)
    run with four copies of one query must retain what the (1,1) run retains."""
    c, d, T = 6, 8, 30
    q, k, v = _stream(18, T, 1, 1, d, peaked=True)
    o1 = Oracle(c, 1, 1, d, 1)
    o4 = Oracle(c, 4, 1, d, 1)
    for t in range(T):
        a = o1.decode_step(q[t], k[t], v[t])
        b = o4.decode_step(np.repeat(q[t], 4, axis=1), k[t], v[t])
        np.testing.assert_allclose(b[0, 2], a[0, 0], rtol=1e-13)
        assert list(o1.positions(0, 0)) == list(o4.positions(0, 0))
        np.testing.assert_allclose(o1.unit(0, 0)[1], o4.unit(0, 0)[1], rtol=1e-12)


# ---------------------------------------------------------------------------------------------
# Chunked prefill reading
# ---------------------------------------------------------------------------------------------
def test_chunk_of_one_equals_decode_step(oracle_lib):
    c, Hq, Hkv, d, T = 5, 4, 2, 8, 23
    q, k, v = _stream(19, T, Hq, Hkv, d, peaked=True)
    a = Oracle(c, Hq, Hkv, d, 1)
    b = Oracle(c, Hq, Hkv, d, 1)
    for t in range(T):
        oa = a.decode_step(q[t], k[t], v[t])
        ob = b.prefill_chunk(q[t][:, None], k[t][:, None], v[t][:, None])
        assert np.array_equal(oa, ob[:, 0])
        for kh in range(Hkv):
            ua, ub = a.unit(0, kh), b.unit(0, kh)
            assert all(np.array_equal(x, y) for x, y in zip(ua, ub))


def test_chunk_that_fits_equals_causal_attention(oracle_lib):
    c, Hq, Hkv, d = 16, 2, 2, 8
    r = _rng(20)
    o = Oracle(c, Hq, Hkv, d, 1)
    K = np.zeros((0, Hkv, d)); V = np.zeros((0, Hkv, d))
    for m in (5, 7, 4):
        q = r.standard_normal((1, m, Hq, d)); k = r.standard_normal((1, m, Hkv, d)); v = r.standard_normal((1, m, Hkv, d))
        out = o.prefill_chunk(q, k, v)
        K = np.concatenate([K, k[0]]); V = np.concatenate([V, v[0]])
        n0 = K.shape[0] - m
        for i in range(m):
            for h in range(Hq):
                ref, _ = _softmax_attention(q[0, i, h], K[: n0 + i + 1, h], V[: n0 + i + 1, h])
                np.testing.assert_allclose(out[0, i, h], ref, rtol=1e-12, atol=1e-13)
        assert o.n_evicted(0) == 0
    assert list(o.positions(0, 1)) == list(range(16))


@pytest.mark.parametrize("rule", [RULE_KEEP_LEFT, RULE_EVICT_LEFT])
@pytest.mark.parametrize("c,m", [(8, 2), (8, 3), (8, 4), (8, 5), (8, 8), (8, 20), (16, 4)])
def test_score_free_chunking_equals_token_by_token(oracle_lib, rule, c, m):
    """With a rule that ignores scores, cutting the stream into chunks (including chunks that do not divide
    c and chunks larger than c) must not change which tokens are retained: the schedule alone decides."""
    d, T = 2, 6 * max(c, m) + 1
    q, k, v = _stream(21, T, 1, 1, d)
    a = Oracle(c, 1, 1, d, 1, rule=rule)
    b = Oracle(c, 1, 1, d, 1, rule=rule)
    t = 0
    while t < T:
        mm = min(m, T - t)
        for s in range(t, t + mm):
            a.decode_step(q[s], k[s], v[s])
        b.prefill_chunk(q[t : t + mm].transpose(1, 0, 2, 3), k[t : t + mm].transpose(1, 0, 2, 3),
                        v[t : t + mm].transpose(1, 0, 2, 3))
        t += mm
        assert list(a.positions(0, 0)) == list(b.positions(0, 0)), (c, m, t)
        assert a.idx(0) == b.idx(0)


def test_chunk_scores_are_column_sums(oracle_lib):
    """S after a chunk = S before + column sums of the causal probability matrix (group mean)."""
    c, Hq, Hkv, d, m = 32, 4, 2, 8, 6
    g = Hq // Hkv
    r = _rng(22)
    o = Oracle(c, Hq, Hkv, d, 1)
    k0 = r.standard_normal((1, 5, Hkv, d)); v0 = r.standard_normal((1, 5, Hkv, d))
    o.prefill_chunk(r.standard_normal((1, 5, Hq, d)), k0, v0)
    S0 = [o.unit(0, kh)[1].copy() for kh in range(Hkv)]
    q = r.standard_normal((1, m, Hq, d)); k = r.standard_normal((1, m, Hkv, d)); v = r.standard_normal((1, m, Hkv, d))
    o.prefill_chunk(q, k, v)
    K = np.concatenate([k0[0], k[0]]); V = np.concatenate([v0[0], v[0]])
    for kh in range(Hkv):
        col = np.zeros(5 + m)
        for i in range(m):
            for hh in range(g):
                _, p = _softmax_attention(q[0, i, kh * g + hh], K[: 5 + i + 1, kh], V[: 5 + i + 1, kh])
                col[: 5 + i + 1] += p / g
        expect = np.concatenate([S0[kh], np.zeros(m)]) + col
        np.testing.assert_allclose(o.unit(0, kh)[1], expect, rtol=1e-12)


def test_ragged_batch_and_inactive_sequences(oracle_lib):
    """Sequences of a batch are independent: a ragged batched run equals separate single-sequence runs."""
    c, Hq, Hkv, d, B = 8, 2, 1, 4, 3
    r = _rng(23)
    ob = Oracle(c, Hq, Hkv, d, B)
    os_ = [Oracle(c, Hq, Hkv, d, 1) for _ in range(B)]
    for lens in ([5, 3, 0], [5, 5, 5], [0, 2, 5], [4, 0, 1]):
        m = 5
        q = r.standard_normal((B, m, Hq, d)); k = r.standard_normal((B, m, Hkv, d)); v = r.standard_normal((B, m, Hkv, d))
        out = ob.prefill_chunk(q, k, v, lens)
        for b in range(B):
            if lens[b]:
                o1 = os_[b].prefill_chunk(q[b : b + 1, : lens[b]], k[b : b + 1, : lens[b]], v[b : b + 1, : lens[b]])
                np.testing.assert_array_equal(out[b, : lens[b]], o1[0])
    for step in range(6):
        act = [1, step % 2, 1]
        q = r.standard_normal((B, Hq, d)); k = r.standard_normal((B, Hkv, d)); v = r.standard_normal((B, Hkv, d))
        out = ob.decode_step(q, k, v, act)
        for b in range(B):
            if act[b]:
                o1 = os_[b].decode_step(q[b : b + 1], k[b : b + 1], v[b : b + 1])
                np.testing.assert_array_equal(out[b], o1[0])
    for b in range(B):
        assert list(ob.positions(b, 0)) == list(os_[b].positions(0, 0))
        assert ob.idx(b) == os_[b].idx(0)


def _adversarial_hint(before, after, c):
    """The retained set that keeps the token a decision dropped and drops the one it kept, everything else alike:
    `before` are the c+1 positions ahead of the eviction, `after` the c positions it left."""
    dropped = [p for p in before if p not in set(after)]
    assert len(dropped) == 1
    j = list(before).index(dropped[0])
    return dropped[0], j


def test_near_tie_hint_is_only_used_at_near_ties(oracle_lib):
    """The near-tie hint (a test device, not part of Algorithm 1) may only change a decision whose relative score gap
    is below the tolerance.  A twin oracle plays Algorithm 1 unaided; the oracle under test gets, at every eviction,
    the hint that asks for the OPPOSITE of the twin's decision in every unit (it contains the loser of the scope
    and not the winner).  With the working tolerance of 1e-4 and well-separated scores nothing may flip."""
    c, d, T, B, Hq, Hkv = 6, 4, 42, 2, 4, 2
    q, k, v = _stream(24, T, Hq, Hkv, d, B, peaked=True)
    a = Oracle(c, Hq, Hkv, d, B)
    b = Oracle(c, Hq, Hkv, d, B)
    decisions = 0
    for t in range(T):
        a.decode_attend(q[t], k[t], v[t])
        b.decode_attend(q[t], k[t], v[t])
        before = {(s, kh): list(a.positions(s, kh)) for s in range(B) for kh in range(Hkv)}
        idx = a.idx(0)
        a.evict()
        if t < c:
            b.evict()
            continue
        hint = np.full((B, Hkv, c), -1, np.int32)
        cnt = np.full((B, Hkv), c, np.int32)
        for (s, kh), bef in before.items():
            aft = list(a.positions(s, kh))
            lost, j = _adversarial_hint(bef, aft, c)
            assert j in (idx - 1, idx)                               # the dropped slot is a member of the scope
            kept = bef[idx - 1] if j == idx else bef[idx]
            h = sorted((set(bef) - {kept}))                          # keeps the loser, drops the winner
            assert len(h) == c and lost in h and kept not in h
            hint[s, kh] = h
        b.evict(hint, cnt, near_tie_tol=1e-4)
        assert b.last_min_gap >= 1e-4, "the stream was meant to have well-separated scores"
        assert b.last_near_ties == 0 and b.last_hint_flips == 0
        decisions += B * Hkv
        for s in range(B):
            for kh in range(Hkv):
                assert list(a.positions(s, kh)) == list(b.positions(s, kh)), (t, s, kh)
    assert decisions == (T - c) * B * Hkv and b.total_hint_flips == 0


def test_near_tie_hint_decides_real_near_ties(oracle_lib):
    """The other direction: with q = 0 every weight is 1/len, so tokens that arrived after the cache filled have
    equal averaged scores up to rounding (relative gap ~1e-16).  There the adversarial hint must win, every time
    the two members of the scope both arrived after the fill."""
    c, d, T = 4, 4, 30
    r = _rng(25)
    k = r.standard_normal((T, 1, 1, d)); v = r.standard_normal((T, 1, 1, d)); q = np.zeros((T, 1, 1, d))
    b = Oracle(c, 1, 1, d, 1)
    flips = 0
    for t in range(T):
        b.decode_attend(q[t], k[t], v[t])
        if t < c:
            b.evict()
            continue
        bef = list(b.positions(0, 0))
        idx = b.idx(0)
        l, rr = bef[idx - 1], bef[idx]
        # what Algorithm 1 does unaided on this state
        pos, S, C, sb = b.unit(0, 0)
        unaided_evicts_right = sb[idx - 1] > sb[idx]
        kept = l if unaided_evicts_right else rr
        h = sorted(set(bef) - {kept})
        gap = abs(sb[idx - 1] - sb[idx]) / max(abs(sb[idx - 1]), abs(sb[idx]))
        b.evict(np.array([[h]], np.int32), np.array([[c]], np.int32), near_tie_tol=1e-4)
        if gap < 1e-4:
            assert b.last_near_ties == 1 and b.last_hint_flips == 1
            assert list(b.positions(0, 0)) == h
            flips += 1
        else:
            assert b.last_hint_flips == 0 and kept in list(b.positions(0, 0))
    assert flips >= 5


def test_near_tie_hint_with_absurd_tolerance(oracle_lib):
    c, d = 4, 4
    q, k, v = _stream(24, c + 1, 1, 1, d, peaked=True)
    # with an absurdly large tolerance every decision is a "near-tie" and the hint decides
    b2 = Oracle(c, 1, 1, d, 1)
    for t in range(c + 1):
        b2.decode_attend(q[t], k[t], v[t])
        if t == c:
            want = np.array([[[1, 2, 3, 4]]], np.int32)        # keep token 1, evict token 0
            b2.evict(want, np.array([[4]], np.int32), near_tie_tol=10.0)
            assert list(b2.positions(0, 0)) == [1, 2, 3, 4]
            want = None
        else:
            b2.evict()
