"""GPU parity on random walks through the C ABI: every seed draws a cache geometry (dtype, head_dim, group size, batch,
budget, chunk capacity), optional protected tokens, in-cache positions and the accumulated criterion, kernel options,
and a sequence of calls that mixes decode steps under changing active sets with ragged chunks (zero lengths
included) and, where the geometry allows it, a one-shot block prefill as the first call.  The CUDA library runs in
lock-step with the fp64 oracle and is held to the usual bars after every call: retained positions exactly up to
counted near-ties, outputs within 2e-2 (bf16) / 1e-4 (fp32), averaged scores within 1e-3.  The fixed cases of the
other files aim at known corners; this one looks for the corners nobody thought of.
"""
import numpy as np
import pytest

import workloads as W
from lockstep import Report, step_decode, step_oneshot, step_prefill

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


def _draw_geometry(rng):
    dtype = "bf16" if rng.random() < 0.7 else "f32"
    d = 128 if rng.random() < 0.65 else 64
    hkv = int(rng.integers(1, 4))
    g = int(rng.choice([1, 2, 4, 8]))
    batch = int(rng.integers(1, 4))
    budget = int([rng.integers(2, 12), rng.integers(12, 160), rng.integers(160, 400)][int(rng.integers(0, 3))])
    max_chunk = int([0, rng.integers(1, 40), rng.integers(40, 300), 128, 256][int(rng.integers(0, 5))])
    return dtype, d, hkv, g, batch, budget, max_chunk


def _chunk_lens(rng, batch, max_chunk):
    """Ragged lengths: zero, anything, the full capacity, or a multiple of 128 (the case in which the tensor-core
    kernels read the chunk from the caller's tensors)."""
    lens = []
    for _ in range(batch):
        r = rng.random()
        if r < 0.15:
            lens.append(0)
        elif r < 0.35:
            lens.append(max_chunk)
        elif r < 0.5 and max_chunk >= 128:
            lens.append(128 * int(rng.integers(1, max_chunk // 128 + 1)))
        else:
            lens.append(int(rng.integers(1, max_chunk + 1)))
    return lens


@pytest.mark.parametrize("seed", range(64))
def test_random_walk(gpu, seed):
    import torch
    from oracle import RULE_ACCUMULATED, RULE_SCORES, Oracle

    rng = np.random.default_rng(977 + seed)
    dtype, d, hkv, g, batch, budget, max_chunk = _draw_geometry(rng)
    positions = rng.random() < 0.35
    accumulated = rng.random() < 0.25   # Section 4.1 "Importance Score": S instead of S / C as the criterion
    ns = nr = 0
    if budget >= 4 and rng.random() < 0.4:
        ns = int(rng.integers(0, min(6, budget - 2) + 1))
        nr = int(rng.integers(0, budget - 2 - ns + 1))
    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=batch, n_heads=g * hkv, n_kv_heads=hkv, head_dim=d, dtype=dtype,
                       budget=budget, chunk=max_chunk, rotate=not positions, seed=31000 + seed)
    kv = gpu.TreeKV(budget, g * hkv, hkv, d, dtype, batch, max_chunk)
    orc = Oracle(budget, g * hkv, hkv, d, batch, n_sink=ns, n_recent=nr, rule=RULE_ACCUMULATED if accumulated else RULE_SCORES)
    if accumulated:
        kv.set_rule(gpu.RULE_ACCUMULATED)
    if ns or nr:
        kv.set_protection(ns, nr)
    if positions:
        cos, sin = W.rope_tables(budget + max(1, max_chunk), d, w.rope_base)
        kv.set_positions(torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda())
        orc.set_rope(cos, sin, round_bf16=(dtype == "bf16"))
    # kernel options: every value is valid on every geometry (a path a context cannot take falls back to the one it can)
    opts = {}
    if rng.random() < 0.5:
        opts[gpu.OPT_DECODE_PATH] = int(rng.integers(0, 2))
    if rng.random() < 0.5:
        opts[gpu.OPT_DECODE_SPLIT] = int(rng.choice([0, 1, 2, 4, 8]))
    if max_chunk and dtype == "bf16" and d == 128:
        opts[gpu.OPT_PREFILL_PATH] = int(rng.integers(0, 4))
        opts[gpu.OPT_PREFILL_KEY_SPLIT] = int(rng.integers(0, 4))
        opts[gpu.OPT_PREFILL_APPEND] = int(rng.integers(0, 2))
    if max_chunk and rng.random() < 0.5:
        opts[gpu.OPT_EVICTION_STREAM] = 1
    for o in (gpu.OPT_DECODE_PATH, gpu.OPT_DECODE_SPLIT, gpu.OPT_PREFILL_PATH, gpu.OPT_PREFILL_KEY_SPLIT,
              gpu.OPT_PREFILL_APPEND, gpu.OPT_EVICTION_STREAM):   # the path first: setting it resets the split
        if o in opts:
            kv.set_option(o, opts[o])
    label = "seed %d: %s d=%d Hkv=%d g=%d B=%d c=%d max_chunk=%d ns=%d nr=%d positions=%d accumulated=%d opts=%s" % (
        seed, dtype, d, hkv, g, batch, budget, max_chunk, ns, nr, positions, accumulated, opts)
    print(label)
    rep = Report()
    seen = [0] * batch

    def chunk_call(lens, oneshot_block=0):
        m = max(max(lens), 1)
        q, k, v = W.tokens_at(w, 0, seen, m)
        q, k, v = (x.transpose(1, 0, 2, 3) for x in (q, k, v))
        if oneshot_block:
            step_oneshot(kv, orc, q, k, v, oneshot_block, dtype, rep, lens=lens)
        else:
            step_prefill(kv, orc, q, k, v, dtype, rep, chunk_lens=lens)
        for b in range(batch):
            seen[b] += lens[b]

    # a one-shot block prefill can only be the first call of a sequence
    blocks = [bl for bl in (1, 2, 4, 8, 16, 32) if budget % bl == 0 and bl <= max_chunk]
    if blocks and not (ns or nr) and rng.random() < 0.3:
        bl = int(rng.choice(blocks))
        lens = [bl * int(rng.integers(0, max_chunk // bl + 1)) for _ in range(batch)]
        if max(lens) > 0:
            chunk_call(lens, oneshot_block=bl)
    tokens_left = 1400 + 3 * budget   # bounds the oracle's work per seed
    for _ in range(int(rng.integers(8, 17))):
        if max_chunk and rng.random() < 0.55:
            lens = _chunk_lens(rng, batch, max_chunk)
            if sum(lens) > tokens_left:
                continue
            tokens_left -= sum(lens)
            chunk_call(lens)
        else:
            for _ in range(int(rng.integers(1, 25 + budget // 3))):   # long enough to fill large budgets and evict
                active = None if rng.random() < 0.6 else [bool(rng.random() < 0.6) for _ in range(batch)]
                q, k, v = W.tokens_at(w, 0, seen, 1)
                step_decode(kv, orc, q[0], k[0], v[0], dtype, rep, active=active)
                for b in range(batch):
                    seen[b] += 1 if active is None or active[b] else 0
    st = kv.stats()
    assert st["device_error"] == 0, label
    for b in range(batch):
        assert kv.tokens_seen(b) == seen[b], label
    assert rep.flips <= rep.near_ties, label
