"""Parity at the configurations' full per-layer sizes, in the launch configuration the benchmark times.

One layer of each configuration is run at its full batch / head count / budget / chunk size.  The oracle cannot
follow every unit at these sizes, so:
  * decode (configuration 2's shape): single-head oracles follow sampled (sequence, head) units in lock-step;
  * chunked prefill (configurations 4 and 5, and the maximum chunk): an oracle with one KV head and the group's g
    query heads follows every sampled (sequence, KV head) unit in lock-step through prefill_attend + evict(hint) -
    retained positions exactly, averaged scores within 1e-3, every output row of the unit within 2e-2, after every
    call - at the launch shape the library picks by itself (the two-tile tensor-core kernel on 512 and more CTAs);
    beside it, sampled output rows are recomputed one by one in fp64 as plain softmax attention over [tokens
    retained before the chunk | chunk tokens up to the row's own] from the raw input stream, and the cache
    invariants that hold at any size are checked after every call (length = min(seen, budget), strictly increasing
    positions, every averaged score in [0, 1]).
Inputs are seeded Gaussians drawn with torch on the device with the recipe's structure (keys with the configuration's
outlier channels or per-sequence scale; q and k carry rotary embedding at their stream positions);
the lock-step tests on slices use the recipe's own counter-based generator.
"""
import math

import numpy as np
import pytest

import workloads as W
from lockstep import NEAR_TIE, OUT_TOL, SCORE_ATOL, SCORE_RTOL, Report, evicted_total

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2501_04987_b200 import _build

    _build.build()
    from paper_2501_04987_b200 import binding

    return binding


def _draw(torch, gen, shape, scale_last=None, seq_scale=None, pos=None, base=None):
    """Seeded Gaussians on the device with the recipe's structure: outlier key channels or per-sequence key scale, and -
    when `pos` (stream positions, broadcastable to shape[:-2]) is given - rotate-half rotary embedding at those
    positions, then rounding to bf16."""
    x = torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32)
    if scale_last is not None:
        x[..., scale_last] *= 8.0
    if seq_scale is not None:
        x *= seq_scale.view(-1, *([1] * (x.dim() - 1)))
    if pos is not None:
        d = shape[-1]
        inv_freq = base ** (-torch.arange(d // 2, device="cuda", dtype=torch.float64) * 2.0 / d)
        ang = pos.to(torch.float64).unsqueeze(-1).unsqueeze(-1) * inv_freq            # [..., 1, d/2]
        cos, sin = torch.cos(ang).float(), torch.sin(ang).float()
        x1, x2 = x[..., : d // 2], x[..., d // 2:]
        x = torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)
    return x.to(torch.bfloat16)


def _softmax_rows(q, K, V):
    s = K @ q / math.sqrt(q.shape[0])
    s -= s.max()
    p = np.exp(s)
    p /= p.sum()
    return p @ V


def _check_invariants(kv, seen):
    pos, cnt = kv.retained_positions()
    pos = pos.cpu().numpy(); cnt = cnt.cpu().numpy()
    sb = kv.scores().cpu().numpy()
    B = pos.shape[0]
    for b in range(B):
        want = min(seen[b], kv.budget)
        assert np.all(cnt[b] == want)
        if want > 1:
            assert np.all(np.diff(pos[b, :, :want], axis=1) > 0)
        if want:
            assert np.all(sb[b, :, :want] >= 0) and np.all(sb[b, :, :want] <= 1.0 + 1e-5)
            assert np.all(pos[b, :, :want] < seen[b]) and np.all(pos[b, :, 0] >= 0)
    return pos, cnt


def test_cfg2_full_layer_decode_sampled_units(gpu):
    """Configuration 2, one full layer: 8 sequences x 32 heads, budget 1024, past one full idx cycle of decode."""
    import torch
    from oracle import Oracle

    w = W.CONFIGS["cfg2"]
    kv = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, 0)
    gen = torch.Generator(device="cuda"); gen.manual_seed(w.seed)
    out_ch = W.outlier_channels(w.head_dim, w.n_outliers)
    sampled = [(0, 0), (3, 17), (7, 31)]
    orcs = [Oracle(w.budget, 1, 1, w.head_dim, 1) for _ in sampled]
    steps = w.budget + 1024 + 60
    reps = [Report() for _ in sampled]
    max_err = 0.0
    for t in range(steps):
        pos = torch.full((w.batch,), t, device="cuda")
        q = _draw(torch, gen, (w.batch, w.n_heads, w.head_dim), pos=pos, base=w.rope_base)
        k = _draw(torch, gen, (w.batch, w.n_kv_heads, w.head_dim), scale_last=out_ch, pos=pos, base=w.rope_base)
        v = _draw(torch, gen, (w.batch, w.n_kv_heads, w.head_dim))
        out = kv.decode_step(q, k, v)
        pos, cnt = kv.retained_positions()
        for (b, h), orc, rep in zip(sampled, orcs, reps):
            qo = q[b, h].float().cpu().numpy()[None, None]
            ko = k[b, h].float().cpu().numpy()[None, None]
            vo = v[b, h].float().cpu().numpy()[None, None]
            ref = orc.decode_attend(qo, ko, vo)
            hp = pos[b, h].cpu().numpy()[None, None]; hc = cnt[b, h].cpu().numpy()[None, None]
            ev0 = evicted_total(orc)
            nt, fl = orc.evict(hp, hc, NEAR_TIE)
            rep.tally(orc, ev0, nt, fl)
            err = float(np.abs(out[b, h].float().cpu().numpy() - ref[0, 0]).max())
            max_err = max(max_err, err); rep.max_out_err = max(rep.max_out_err, err)
            assert err <= 2e-2, (t, b, h, err)
            assert np.array_equal(orc.retained_positions()[0][0, 0], hp[0, 0]), (t, b, h)
        if t % 97 == 0 or t == steps - 1:
            sb = kv.scores().cpu().numpy()
            for (b, h), orc in zip(sampled, orcs):
                so = orc.scores()[0, 0]
                assert np.all(np.abs(sb[b, h] - so) <= 1e-3 * np.abs(so) + 1e-12), (t, b, h)
    _check_invariants(kv, [steps] * w.batch)
    st = kv.stats()
    assert st["device_error"] == 0 and st["evictions"] == w.batch * (steps - w.budget)
    print("cfg2 full layer: max out err %.3g" % max_err, reps)


def _lockstep_sampled(orc, rep, sampled, q, k, v, out, lens, pos_g, cnt_g, sb_g, decode):
    """One call of the single-KV-head oracle (sequence s of the oracle = sampled unit s) beside the library's call.
    q,k,v,out: the call's device tensors; pos_g, cnt_g, sb_g: the library's read-outs after the call (numpy)."""
    g = orc.Hq
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    if decode:
        qs = np.stack([f64(q[b, kh * g:(kh + 1) * g]) for (b, kh) in sampled])            # [S, g, d]
        ks = np.stack([f64(k[b, kh:kh + 1]) for (b, kh) in sampled])
        vs = np.stack([f64(v[b, kh:kh + 1]) for (b, kh) in sampled])
        out_o = orc.decode_attend(qs, ks, vs)
        out_g = np.stack([f64(out[b, kh * g:(kh + 1) * g]) for (b, kh) in sampled])
        err = float(np.abs(out_g - out_o).max())
    else:
        qs = np.stack([f64(q[b, :, kh * g:(kh + 1) * g]) for (b, kh) in sampled])         # [S, m, g, d]
        ks = np.stack([f64(k[b, :, kh:kh + 1]) for (b, kh) in sampled])
        vs = np.stack([f64(v[b, :, kh:kh + 1]) for (b, kh) in sampled])
        ls = [lens[b] for (b, kh) in sampled]
        out_o = orc.prefill_attend(qs, ks, vs, ls)
        err = 0.0
        for s, (b, kh) in enumerate(sampled):
            if ls[s]:
                err = max(err, float(np.abs(f64(out[b, :ls[s], kh * g:(kh + 1) * g]) - out_o[s, :ls[s]]).max()))
    rep.max_out_err = max(rep.max_out_err, err)
    assert err <= OUT_TOL["bf16"], "sampled units' outputs off by %.3g" % err
    hp = np.stack([pos_g[b, kh] for (b, kh) in sampled])[:, None, :].astype(np.int32)
    hc = np.array([[cnt_g[b, kh]] for (b, kh) in sampled], np.int32)
    ev0 = evicted_total(orc)
    nt, fl = orc.evict(hp, hc, NEAR_TIE)
    rep.tally(orc, ev0, nt, fl)
    pos_o, cnt_o = orc.retained_positions()
    assert np.array_equal(cnt_o, hc), "retained counts differ from the oracle's"
    if not np.array_equal(pos_o, hp):
        bad = np.argwhere(pos_o != hp)[0]
        raise AssertionError("retained positions differ at sampled unit %s slot %d: library %d oracle %d" %
                             (sampled[bad[0]], bad[2], hp[tuple(bad)], pos_o[tuple(bad)]))
    so = orc.scores()[:, 0, :]
    sg = np.stack([sb_g[b, kh] for (b, kh) in sampled]).astype(np.float64)
    e = np.abs(sg - so)
    lim = SCORE_RTOL * np.abs(so) + SCORE_ATOL
    if not np.all(e <= lim):
        bad = np.argwhere(e > lim)[0]
        raise AssertionError("score differs at sampled unit %s slot %d: library %.9g oracle %.9g" %
                             (sampled[bad[0]], bad[1], sg[tuple(bad)], so[tuple(bad)]))
    with np.errstate(divide="ignore", invalid="ignore"):
        rel = np.where(so > 1e-9, e / so, 0.0)
    rep.max_score_rel = max(rep.max_score_rel, float(rel.max()))


def _prefill_fullsize(gpu, w, lens_total, decode_steps, n_sample_rows=6, first_chunk=None, positions=False):
    import torch
    from oracle import Oracle

    B, Hq, Hkv, d, m, c = w.batch, w.n_heads, w.n_kv_heads, w.head_dim, w.chunk, w.budget
    g = Hq // Hkv
    kv = gpu.TreeKV(c, Hq, Hkv, d, w.dtype, B, m)
    gen = torch.Generator(device="cuda"); gen.manual_seed(w.seed)
    rs = np.random.default_rng(w.seed)
    seq_scale = torch.from_numpy(W.seq_key_scales(w)).cuda() if w.key_scale else None
    sampled = sorted(set([(0, 0), (B - 1, Hkv - 1), (B // 2, Hkv // 2)]))
    orc = Oracle(c, g, 1, d, len(sampled))   # sequence s of the oracle follows sampled unit s (one KV head, g query heads)
    if positions:  # in-cache positions: the same tables on both sides; the brute-force rows below assume none, so they are skipped
        cos, sin = W.rope_tables(c + m, d, w.rope_base)
        kv.set_positions(torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda())
        orc.set_rope(cos, sin, round_bf16=True)
    rep = Report()
    hist_k = {u: np.zeros((0, d)) for u in sampled}   # full key / value streams of the sampled units (fp64)
    hist_v = {u: np.zeros((0, d)) for u in sampled}
    seen = [0] * B
    lens_total = list(lens_total)
    # call boundaries: chunks of m, optionally after a shorter first chunk
    bounds = [0] + ([first_chunk] if first_chunk else [])
    while bounds[-1] < max(lens_total):
        bounds.append(bounds[-1] + m)
    max_err = 0.0
    for call in range(len(bounds) - 1):
        lens = [max(0, min(bounds[call + 1], L) - bounds[call]) for L in lens_total]
        # the recipe rotates q and k at their stream positions (with in-cache positions they stay unrotated)
        pos = None if positions else (torch.tensor(seen, device="cuda").view(B, 1) + torch.arange(m, device="cuda").view(1, m))
        q = _draw(torch, gen, (B, m, Hq, d), pos=pos, base=w.rope_base)
        k = _draw(torch, gen, (B, m, Hkv, d), seq_scale=seq_scale, pos=pos, base=w.rope_base)
        v = _draw(torch, gen, (B, m, Hkv, d))
        pos_before, cnt_before = kv.retained_positions()
        pos_before = pos_before.cpu().numpy(); cnt_before = cnt_before.cpu().numpy()
        out = kv.prefill_chunk(q, k, v, chunk_lens=lens)
        for (b, kh) in sampled:
            mb = lens[b]
            if mb == 0 or positions:
                continue
            kc = k[b, :mb, kh].float().cpu().numpy().astype(np.float64)
            vc = v[b, :mb, kh].float().cpu().numpy().astype(np.float64)
            Kall = np.concatenate([hist_k[(b, kh)], kc]); Vall = np.concatenate([hist_v[(b, kh)], vc])
            hist_k[(b, kh)], hist_v[(b, kh)] = Kall, Vall
            keep = pos_before[b, kh, : cnt_before[b, kh]]
            rows = sorted(set([0, mb - 1] + [int(x) for x in rs.integers(0, mb, n_sample_rows)]))
            for t in rows:
                vis = np.concatenate([keep, np.arange(seen[b], seen[b] + t + 1)])
                for hh in (0, g - 1):
                    h = kh * g + hh
                    ref = _softmax_rows(q[b, t, h].float().cpu().numpy().astype(np.float64), Kall[vis], Vall[vis])
                    err = float(np.abs(out[b, t, h].float().cpu().numpy() - ref).max())
                    max_err = max(max_err, err)
                    assert err <= 2e-2, (call, b, t, h, err)
        seen = [s + l for s, l in zip(seen, lens)]
        pos_g, cnt_g = _check_invariants(kv, seen)
        _lockstep_sampled(orc, rep, sampled, q, k, v, out, lens, pos_g, cnt_g, kv.scores().cpu().numpy(), decode=False)
    assert [kv.tokens_seen(b) for b in range(B)] == seen
    # batched decode steps at ragged stream positions: sampled rows against brute force over the retained set
    for step in range(decode_steps):
        pos = None if positions else torch.tensor(seen, device="cuda").view(B)
        q = _draw(torch, gen, (B, Hq, d), pos=pos, base=w.rope_base)
        k = _draw(torch, gen, (B, Hkv, d), seq_scale=seq_scale, pos=pos, base=w.rope_base)
        v = _draw(torch, gen, (B, Hkv, d))
        pos_before, cnt_before = kv.retained_positions()
        pos_before = pos_before.cpu().numpy(); cnt_before = cnt_before.cpu().numpy()
        out = kv.decode_step(q, k, v)
        for (b, kh) in ([] if positions else sampled):
            hist_k[(b, kh)] = np.concatenate([hist_k[(b, kh)], k[b, kh].float().cpu().numpy().astype(np.float64)[None]])
            hist_v[(b, kh)] = np.concatenate([hist_v[(b, kh)], v[b, kh].float().cpu().numpy().astype(np.float64)[None]])
            vis = np.concatenate([pos_before[b, kh, : cnt_before[b, kh]], [seen[b]]])
            for hh in (0, g - 1):
                h = kh * g + hh
                ref = _softmax_rows(q[b, h].float().cpu().numpy().astype(np.float64), hist_k[(b, kh)][vis], hist_v[(b, kh)][vis])
                err = float(np.abs(out[b, h].float().cpu().numpy() - ref).max())
                max_err = max(max_err, err)
                assert err <= 2e-2, (step, b, h, err)
        seen = [s + 1 for s in seen]
        pos_g, cnt_g = kv.retained_positions()
        _lockstep_sampled(orc, rep, sampled, q, k, v, out, None, pos_g.cpu().numpy(), cnt_g.cpu().numpy(),
                          kv.scores().cpu().numpy(), decode=True)
    _check_invariants(kv, seen)
    assert kv.stats()["device_error"] == 0
    print(rep)
    return max_err


def test_cfg4_full_layer_prefill_then_decode(gpu):
    """Configuration 4, one full layer: 32 sequences, 32 query / 8 KV heads, budget 2048, 4096-token prefill in
    chunks of 1024 (8192 CTAs of the tensor-core kernel per chunk), then decode steps."""
    w = W.CONFIGS["cfg4"]
    err = _prefill_fullsize(gpu, w, [4096] * w.batch, decode_steps=40)
    print("cfg4 full layer: max sampled out err %.3g" % err)


def test_cfg5_full_layer_ragged_prefill(gpu):
    """Configuration 5's per-layer shape (4 sequences, GQA 4:1, budget 4096, chunks of 1024) with ragged lengths that
    end in different, partial chunks; lengths are cut to about 2.5 budgets to keep the run short."""
    w = W.CONFIGS["cfg5"]
    lens = [2 * 4096 + 1024 + 517, 2 * 4096 + 100, 10 * 1024, 2 * 4096 + 1]
    err = _prefill_fullsize(gpu, w, lens, decode_steps=24)
    print("cfg5 full layer: max sampled out err %.3g" % err)


def test_cfg5_full_layer_prefill_with_in_cache_positions(gpu):
    """The same shape with in-cache positions (Section 4.1 "Position Encoding"): the key / query encoding kernel in front
    of the two-tile tensor-core kernel at its full grid, then the mma.sync decode kernel encoding its tiles, with
    one-head oracles in lock-step (every output row of the sampled units, retained positions, scores)."""
    w = W.CONFIGS["cfg5"]
    lens = [4096 + 1024 + 300, 4096 + 1024, 5 * 1024, 4096 + 17]
    _prefill_fullsize(gpu, w, lens, decode_steps=8, positions=True)


@pytest.mark.parametrize("c,Hq,Hkv", [(16384, 8, 2), (65536, 1, 1)])
def test_large_budget_decode_through_eight_block_clusters(gpu, c, Hq, Hkv):
    """Budgets of 16384 (one sequence, two KV heads, g = 4) and of 65536, the largest the library accepts (one head):
    the decode kernel runs as clusters of eight blocks with 2049 / 8193 rows each, close to the largest shared-memory
    footprint.  The cache is filled token by token, then steps across the first evictions are checked on every head
    against fp64 softmax attention over the retained set, with the cache invariants."""
    import torch

    d, B = 128, 1
    g = Hq // Hkv
    kv = gpu.TreeKV(c, Hq, Hkv, d, "bf16", B, 0)
    gen = torch.Generator(device="cuda"); gen.manual_seed(20250111)
    steps = c + 24
    q = _draw(torch, gen, (steps, B, Hq, d))
    k = _draw(torch, gen, (steps, B, Hkv, d))
    v = _draw(torch, gen, (steps, B, Hkv, d))
    kh64 = k[:, 0].float().cpu().numpy().astype(np.float64)   # [steps, Hkv, d]
    vh64 = v[:, 0].float().cpu().numpy().astype(np.float64)
    out = torch.empty((B, Hq, d), dtype=torch.bfloat16, device="cuda")
    max_err = 0.0
    for t in range(steps):
        check = t >= c - 8 or t in (0, 1, 17, 4097)
        if check:
            pos_before, cnt_before = kv.retained_positions()
            pos_before = pos_before.cpu().numpy(); cnt_before = cnt_before.cpu().numpy()
        kv.decode_step(q[t], k[t], v[t], out)
        if check:
            o = out.float().cpu().numpy()
            for kh in range(Hkv):
                vis = np.concatenate([pos_before[0, kh, : cnt_before[0, kh]], [t]])
                for hh in range(g):
                    h = kh * g + hh
                    ref = _softmax_rows(q[t, 0, h].float().cpu().numpy().astype(np.float64), kh64[vis, kh], vh64[vis, kh])
                    err = float(np.abs(o[0, h] - ref).max())
                    max_err = max(max_err, err)
                    assert err <= 2e-2, (t, h, err)
    _check_invariants(kv, [steps])
    st = kv.stats()
    assert st["device_error"] == 0 and st["evictions"] == steps - c
    print("c=%d decode: max out err %.3g" % (c, max_err))


@pytest.mark.parametrize("path", [1, 2, 3])
def test_maximum_chunk_with_many_wraps(gpu, path):
    """The longest chunk the library accepts (8192 tokens) into a budget of 1024: one call evicts through eight wraps of
    the idx cycle, with a rebase of the not yet paired rows after each.  Run with the CUDA-core kernel and with both
    tensor-core kernels; sampled output rows against fp64 attention over [retained before the call | chunk so far]."""
    import torch

    w = W.parity_slice(W.CONFIGS["cfg5"], layers=1, batch=1, n_heads=2, n_kv_heads=1, budget=1024, chunk=8192, key_scale=False)
    kv_holder = {}

    class _Forced:
        """binding.TreeKV with the prefill path fixed at creation."""
        def __getattr__(self, name):
            return getattr(gpu, name)

        def TreeKV(self, *a, **k):
            kv = gpu.TreeKV(*a, **k)
            kv.set_option(gpu.OPT_PREFILL_PATH, path)
            kv_holder["kv"] = kv
            return kv

    err = _prefill_fullsize(_Forced(), w, [700 + 2 * 8192], decode_steps=6, n_sample_rows=5, first_chunk=700)
    st = kv_holder["kv"].stats()
    assert st["evictions"] == 700 + 2 * 8192 + 6 - 1024 and st["device_error"] == 0
    print("m=8192 into c=1024, path %d: max sampled out err %.3g" % (path, err))
