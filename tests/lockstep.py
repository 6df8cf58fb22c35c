"""Lock-step comparison of the CUDA library (through its C ABI) with the fp64 oracle on identical inputs.

After every call the retained positions of both sides are compared.  A pair decision whose relative score gap
in the oracle is below 1e-4 is a near-tie: there the fp32 kernel may legitimately choose the other token, and
the oracle then follows the library's choice so that later calls still compare like with like; such flips are
counted.  Any other difference in the retained sets is a failure.  Outputs and averaged scores are compared
element by element within the stated tolerances.
"""
from __future__ import annotations

import os

import numpy as np

OUT_TOL = {"bf16": 2e-2, "f32": 1e-4}   # max abs error of attention outputs
SCORE_RTOL = 1e-3                        # relative error of S/C of every retained token
SCORE_ATOL = 1e-12                       # floor for weights that underflow in fp32
NEAR_TIE = 1e-4


REPORTS = []   # every Report of the session, in creation order; the terminal summary prints them (conftest.py)


class Report:
    """Tallies of one lock-step run.  `decisions` counts pair decisions (evictions x KV heads) the oracle took,
    `near_ties` those whose relative gap was below NEAR_TIE, `flips` those where the oracle followed the library."""

    def __init__(self, label=None):
        self.label = label or os.environ.get("PYTEST_CURRENT_TEST", "?").split(" ")[0]
        self.calls = 0
        self.max_out_err = 0.0
        self.max_score_rel = 0.0
        self.near_ties = 0
        self.flips = 0
        self.decisions = 0
        REPORTS.append(self)

    def tally(self, orc, evicted_before, near_ties, flips):
        """Add one oracle eviction call: `evicted_before` = sum of n_evicted over sequences before the call."""
        after = sum(orc.n_evicted(b) for b in range(orc.B))
        self.decisions += (after - evicted_before) * orc.Hkv
        self.near_ties += near_ties
        self.flips += flips
        self.calls += 1
        # a flip is only possible at a near-tie: anything else means the oracle followed the library where it must not
        assert self.flips <= self.near_ties <= self.decisions, repr(self)

    def __repr__(self):
        return ("calls=%d max_out_err=%.3g max_score_rel=%.3g decisions=%d near_ties=%d flips=%d" %
                (self.calls, self.max_out_err, self.max_score_rel, self.decisions, self.near_ties, self.flips))


def evicted_total(orc):
    return sum(orc.n_evicted(b) for b in range(orc.B))


def _to_dev(torch, a, tdtype):
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda").to(tdtype).contiguous()


def compare_state(kv, orc, rep, check_scores=True):
    """Retained positions must match exactly; averaged scores within tolerance."""
    pos_g, cnt_g = kv.retained_positions()
    pos_g = pos_g.cpu().numpy(); cnt_g = cnt_g.cpu().numpy()
    pos_o, cnt_o = orc.retained_positions()
    assert np.array_equal(cnt_g, cnt_o), "retained counts differ"
    if not np.array_equal(pos_g, pos_o):
        bad = np.argwhere(pos_g != pos_o)[0]
        raise AssertionError("retained positions differ at (b,head,slot)=%s: gpu %d oracle %d" %
                             (tuple(bad), pos_g[tuple(bad)], pos_o[tuple(bad)]))
    for b in range(orc.B):
        for kh in range(orc.Hkv):
            p = pos_g[b, kh, : cnt_g[b, kh]]
            assert np.all(np.diff(p) > 0), "positions not strictly increasing"
    if check_scores:
        sb_g = kv.scores().cpu().numpy().astype(np.float64)
        sb_o = orc.scores()
        err = np.abs(sb_g - sb_o)
        lim = SCORE_RTOL * np.abs(sb_o) + SCORE_ATOL
        if not np.all(err <= lim):
            bad = np.argwhere(err > lim)[0]
            raise AssertionError("score differs at %s: gpu %.9g oracle %.9g" %
                                 (tuple(bad), sb_g[tuple(bad)], sb_o[tuple(bad)]))
        with np.errstate(divide="ignore", invalid="ignore"):
            rel = np.where(sb_o > 1e-9, err / sb_o, 0.0)
        rep.max_score_rel = max(rep.max_score_rel, float(rel.max()))


def _f64(t):
    """Device tensor -> float64 numpy.  Rows the library does not write (beyond a sequence's length, inactive sequences)
    hold whatever the allocation held, possibly signalling NaNs: they are never compared, only converted."""
    with np.errstate(invalid="ignore"):
        return t.float().cpu().numpy().astype(np.float64)


def step_decode(kv, orc, q, k, v, dtype, rep, active=None, check_scores=True):
    """q [B,Hq,d], k,v [B,Hkv,d] float32 numpy holding dtype-rounded values."""
    import torch

    out_o = orc.decode_attend(q, k, v, active)
    out_g = kv.decode_step(_to_dev(torch, q, kv.tdtype), _to_dev(torch, k, kv.tdtype), _to_dev(torch, v, kv.tdtype),
                           active=active)
    pos_g, cnt_g = kv.retained_positions()
    ev0 = evicted_total(orc)
    nt, fl = orc.evict(pos_g.cpu().numpy(), cnt_g.cpu().numpy(), NEAR_TIE)
    rep.tally(orc, ev0, nt, fl)
    og = _f64(out_g)
    sel = slice(None) if active is None else np.asarray(active, bool)
    err = float(np.abs(og[sel] - out_o[sel]).max()) if np.size(og[sel]) else 0.0
    rep.max_out_err = max(rep.max_out_err, err)
    assert err <= OUT_TOL[dtype], "attention output off by %.3g (tolerance %.3g)" % (err, OUT_TOL[dtype])
    compare_state(kv, orc, rep, check_scores)


def step_prefill(kv, orc, q, k, v, dtype, rep, chunk_lens=None, check_scores=True, method="prefill_chunk"):
    """q [B,m,Hq,d], k,v [B,m,Hkv,d] float32 numpy holding dtype-rounded values; `method` names the wrapper's call."""
    import torch

    B, m = q.shape[0], q.shape[1]
    lens = [m] * B if chunk_lens is None else [int(x) for x in chunk_lens]
    out_o = orc.prefill_attend(q, k, v, lens)
    out_g = getattr(kv, method)(_to_dev(torch, q, kv.tdtype), _to_dev(torch, k, kv.tdtype),
                                _to_dev(torch, v, kv.tdtype), chunk_lens=lens)
    pos_g, cnt_g = kv.retained_positions()
    ev0 = evicted_total(orc)
    nt, fl = orc.evict(pos_g.cpu().numpy(), cnt_g.cpu().numpy(), NEAR_TIE)
    rep.tally(orc, ev0, nt, fl)
    og = _f64(out_g)
    err = 0.0
    for b in range(B):
        if lens[b]:
            err = max(err, float(np.abs(og[b, : lens[b]] - out_o[b, : lens[b]]).max()))
    rep.max_out_err = max(rep.max_out_err, err)
    assert err <= OUT_TOL[dtype], "attention output off by %.3g (tolerance %.3g)" % (err, OUT_TOL[dtype])
    compare_state(kv, orc, rep, check_scores)


def step_oneshot(kv, orc, q, k, v, block, dtype, rep, lens=None, check_scores=True):
    """One-shot block-level prefill of empty caches; q [B,T,Hq,d], k,v [B,T,Hkv,d] float32 numpy, dtype-rounded."""
    import torch

    B, T = q.shape[0], q.shape[1]
    ls = [T] * B if lens is None else [int(x) for x in lens]
    out_o = orc.prefill_oneshot_attend(q, k, v, block, ls)
    out_g = kv.prefill_oneshot(_to_dev(torch, q, kv.tdtype), _to_dev(torch, k, kv.tdtype), _to_dev(torch, v, kv.tdtype),
                               block, lens=ls)
    pos_g, cnt_g = kv.retained_positions()
    ev0 = evicted_total(orc)
    nt, fl = orc.evict_blocks(pos_g.cpu().numpy(), cnt_g.cpu().numpy(), NEAR_TIE)
    # decisions are taken per block pair: evicted tokens / block, per KV head
    after = evicted_total(orc)
    rep.decisions += (after - ev0) // block * orc.Hkv
    rep.near_ties += nt; rep.flips += fl; rep.calls += 1
    assert rep.flips <= rep.near_ties <= rep.decisions or rep.near_ties == 0, repr(rep)
    og = _f64(out_g)
    err = 0.0
    for b in range(B):
        if ls[b]:
            err = max(err, float(np.abs(og[b, : ls[b]] - out_o[b, : ls[b]]).max()))
    rep.max_out_err = max(rep.max_out_err, err)
    assert err <= OUT_TOL[dtype], "attention output off by %.3g (tolerance %.3g)" % (err, OUT_TOL[dtype])
    compare_state(kv, orc, rep, check_scores)


def _workloads():
    import workloads

    return workloads


def run_decode(kv, orc, w, t0, steps, rep, score_every=1, starts=None):
    blk = 256
    done = 0
    while done < steps:
        n = min(blk, steps - done)
        st = [t0 + done] * w.batch if starts is None else [s + done for s in starts]
        q, k, v = _workloads().tokens_at(w, 0, st, n)
        for i in range(n):
            step_decode(kv, orc, q[i], k[i], v[i], w.dtype, rep, check_scores=((done + i) % score_every == 0))
        done += n


def run_prefill(kv, orc, w, rep, lens_total, chunk, method="prefill_chunk"):
    """Feed sequence b its first lens_total[b] tokens in chunks of `chunk` (ragged at the end)."""
    lens_total = np.asarray(lens_total)
    n_calls = int((lens_total.max() + chunk - 1) // chunk)
    for c in range(n_calls):
        q, k, v = _workloads().tokens(w, 0, c * chunk, (c + 1) * chunk)
        lens = np.clip(lens_total - c * chunk, 0, chunk)
        step_prefill(kv, orc, q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3), w.dtype, rep,
                     chunk_lens=lens, method=method)
