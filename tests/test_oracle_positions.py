"""Pins for the oracle's in-cache positions (Section 4.1 "Position Encoding": positional encodings are re-assigned
after eviction, as in StreamingLLM).  q and k arrive without positional encoding; attention encodes the token in
cache slot j at position j and the query at its own slot.
"""
import math
import os

import numpy as np
import pytest

import workloads as W
from oracle import Oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _tables(slots, d, base=1e4):
    """cos / sin by slot, single precision (an input of the method, as a model's rotary cache is)."""
    inv = base ** (-np.arange(d // 2, dtype=np.float64) * 2.0 / d)
    ang = np.arange(slots, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def _assign(cache_positions_and_new):
    """The paper's rule: whatever stream positions the cached tokens and the new one have, they are encoded at
    0, 1, 2, ... in cache order."""
    return list(range(len(cache_positions_and_new)))


def test_papers_position_example():
    g = {}
    for line in open(os.path.join(GOLDEN, "position_example.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            key, val = [x.strip() for x in line.split("=")]
            g[key] = [int(x) for x in val.split()]
    assert _assign(g["cache"] + g["new_token"]) == g["assigned"]


def _rope_f64(x, p, cos, sin):
    half = x.shape[-1] // 2
    c, s = cos[p].astype(np.float64), sin[p].astype(np.float64)
    return np.concatenate([x[:half] * c - x[half:] * s, x[half:] * c + x[:half] * s])


def _brute_force(q, k, v, c, cos, sin):
    """Dictionary restatement with in-cache positions, fp64 rotation, no rounding."""
    d = q.shape[-1]
    cache, idx, outs, history = [], 1, [], []
    for t in range(q.shape[0]):
        cache.append({"pos": t, "k": k[t], "v": v[t], "S": 0.0, "C": 0})
        assigned = _assign([e["pos"] for e in cache])
        qq = _rope_f64(q[t], assigned[-1], cos, sin)
        s = np.array([qq @ _rope_f64(e["k"], a, cos, sin) for e, a in zip(cache, assigned)]) / math.sqrt(d)
        p = np.exp(s - s.max()); p /= p.sum()
        outs.append(sum(pi * e["v"] for pi, e in zip(p, cache)))
        for pi, e in zip(p, cache):
            e["S"] += pi; e["C"] += 1
        if len(cache) > c:
            l, r = cache[idx - 1], cache[idx]
            loser = r if l["S"] / l["C"] > r["S"] / r["C"] else l
            cache = [e for e in cache if e is not loser]
            idx = idx % c + 1
        history.append([e["pos"] for e in cache])
    return np.array(outs), history


def test_matches_brute_force_with_reassigned_positions(oracle_lib):
    c, d, T = 6, 8, 40
    r = np.random.default_rng(31)
    q = r.standard_normal((T, d)); k = r.standard_normal((T, d)); v = r.standard_normal((T, d))
    k[:, 0] *= 3.0
    cos, sin = _tables(c + 1, d)
    o = Oracle(c, 1, 1, d, 1)
    o.set_rope(cos, sin, round_bf16=False)
    outs, hist = _brute_force(q, k, v, c, cos, sin)
    for t in range(T):
        out = o.decode_step(q[t][None, None], k[t][None, None], v[t][None, None])
        # the oracle rotates in single precision (its stated contract), the restatement in double
        np.testing.assert_allclose(out[0, 0], outs[t], rtol=2e-5, atol=2e-6)
        assert list(o.positions(0, 0)) == hist[t], t
    assert hist[-1] != list(range(T - c, T))     # evictions did happen in the middle of the cache
    # the stored keys are the keys as given, not rotated ones
    K, _ = o.kv(0, 0)
    np.testing.assert_array_equal(K, k[hist[-1]])


def test_without_eviction_equals_stream_positions(oracle_lib):
    """While nothing has been evicted slot j holds token j, so in-cache positions are the stream positions: the
    result must equal the position-agnostic oracle fed with inputs that were rotated beforehand at their stream
    positions (what the workload generator does), up to the single-precision rotation."""
    c, Hq, Hkv, d, T = 16, 4, 2, 8, 16
    r = np.random.default_rng(32)
    q = r.standard_normal((T, 1, Hq, d)).astype(np.float32)
    k = r.standard_normal((T, 1, Hkv, d)).astype(np.float32)
    v = r.standard_normal((T, 1, Hkv, d)).astype(np.float32)
    cos, sin = _tables(T, d)
    a = Oracle(c, Hq, Hkv, d, 1)
    a.set_rope(cos, sin, round_bf16=False)
    b = Oracle(c, Hq, Hkv, d, 1)
    pos = np.arange(T)
    qr = W.rope(q[:, 0], pos, 1e4)[:, None]; kr = W.rope(k[:, 0], pos, 1e4)[:, None]
    # decode steps, then the same as one chunk
    for t in range(T):
        oa = a.decode_step(q[t], k[t], v[t]); ob = b.decode_step(qr[t], kr[t], v[t])
        np.testing.assert_allclose(oa, ob, rtol=1e-4, atol=1e-5)
    a2 = Oracle(c, Hq, Hkv, d, 1); a2.set_rope(cos, sin, round_bf16=False)
    b2 = Oracle(c, Hq, Hkv, d, 1)
    oa = a2.prefill_chunk(q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3))
    ob = b2.prefill_chunk(qr.transpose(1, 0, 2, 3), kr.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3))
    np.testing.assert_allclose(oa, ob, rtol=1e-4, atol=1e-5)
    for kh in range(Hkv):
        np.testing.assert_allclose(a2.unit(0, kh)[1], b2.unit(0, kh)[1], rtol=1e-4)


def test_rotation_arithmetic_on_exactly_representable_values(oracle_lib):
    """Inputs and table entries with few significant bits make every product and sum exact, so the rotated dot
    product can be written down by hand: one query, one key, d = 2, slot 0 for both (cache of one token)."""
    d = 2
    cos = np.array([[0.5]], np.float32); sin = np.array([[0.25]], np.float32)     # not a rotation: the arithmetic is what is pinned
    o = Oracle(4, 1, 1, d, 1)
    o.set_rope(cos, sin, round_bf16=True)
    q = np.array([1.5, -2.0]); k = np.array([0.75, 3.0]); v = np.array([1.0, 2.0])
    out = o.decode_step(q[None, None], k[None, None], v[None, None])
    np.testing.assert_array_equal(out[0, 0], v)       # a single token gets weight 1
    # second token at slot 1 with a different table row: weights follow the hand-computed logits
    cos = np.array([[0.5], [1.0]], np.float32); sin = np.array([[0.25], [-0.5]], np.float32)
    o = Oracle(4, 1, 1, d, 1)
    o.set_rope(cos, sin, round_bf16=True)
    o.decode_step(q[None, None], k[None, None], v[None, None])
    q2 = np.array([2.0, 1.0]); k2 = np.array([-1.0, 0.5]); v2 = np.array([-3.0, 0.5])
    out = o.decode_step(q2[None, None], k2[None, None], v2[None, None])
    rot = lambda x, c, s: np.array([x[0] * c - x[1] * s, x[1] * c + x[0] * s])
    qq = rot(q2, 1.0, -0.5)                       # the query sits in slot 1
    logits = np.array([qq @ rot(k, 0.5, 0.25), qq @ rot(k2, 1.0, -0.5)]) / math.sqrt(d)
    p = np.exp(logits - logits.max()); p /= p.sum()
    np.testing.assert_allclose(out[0, 0], p[0] * v + p[1] * v2, rtol=1e-14)
    np.testing.assert_allclose(o.unit(0, 0)[1], [1.0 + p[0], p[1]], rtol=1e-14)


def test_rotated_operands_are_rounded_to_bf16_when_asked(oracle_lib):
    """With a bf16 cache the rotated q and k are rounded to bf16 before the dot product (the paper's set-up is bf16
    throughout): the logit of a single key against itself must be the squared norm of the ROUNDED rotated vector."""
    d = 4
    cos, sin = _tables(3, d)
    x = W.round_bf16(np.array([1.0078125, -0.33203125, 0.7265625, 2.140625], np.float32)).astype(np.float64)
    z = np.zeros(d)
    v0 = np.array([1.0, 0, 0, 0]); v1 = np.array([0, 1.0, 0, 0])
    # slot 0 holds a zero key (logit 0), slot 1 holds x, and the query is x too
    res = []
    for rb in (True, False):
        orc = Oracle(4, 1, 1, d, 1); orc.set_rope(cos, sin, round_bf16=rb)
        orc.decode_step(z[None, None], z[None, None], v0[None, None])
        out = orc.decode_step(x[None, None], x[None, None], v1[None, None])
        res.append(out[0, 0])
    def expect(rb):
        c, s = cos[1].astype(np.float64), sin[1].astype(np.float64)
        r = np.concatenate([x[:2] * c - x[2:] * s, x[2:] * c + x[:2] * s]).astype(np.float32)
        if rb:
            r = W.round_bf16(r)
        lg = np.array([0.0, float(r.astype(np.float64) @ r.astype(np.float64)) / 2.0])
        p = np.exp(lg - lg.max()); p /= p.sum()
        return p[0] * v0 + p[1] * v1
    np.testing.assert_allclose(res[0], expect(True), rtol=1e-12)
    np.testing.assert_allclose(res[1], expect(False), rtol=1e-5)
    assert abs(res[0][1] - res[1][1]) > 1e-5          # the rounding is visible
