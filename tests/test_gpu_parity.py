"""GPU parity: the CUDA library, called through its C ABI, against the fp64 oracle on the same seeded inputs.

Bars: retained positions bit-exact except at counted near-ties (oracle pair gap < 1e-4 relative); attention
outputs within 2e-2 (bf16) / 1e-4 (fp32) max abs; averaged scores within 1e-3 relative.
"""
import numpy as np
import pytest

import workloads as W
from lockstep import Report, compare_state, step_decode, step_prefill
from lockstep import run_decode as _run_decode, run_prefill as _run_prefill

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


def _pair(binding, w, max_chunk=None):
    from oracle import Oracle

    mc = w.chunk if max_chunk is None else max_chunk
    kv = binding.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, mc)
    orc = Oracle(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.batch)
    return kv, orc


# ---------------------------------------------------------------------------------------------------------
def test_cfg1_full_decode_fp32(gpu):
    """Configuration 1 at full size: fp32, 4 heads, d=64, c=256, 2048 decode steps, compared after every step."""
    w = W.CONFIGS["cfg1"]
    kv, orc = _pair(gpu, w)
    rep = Report()
    _run_decode(kv, orc, w, 0, w.decode_steps, rep)
    print("cfg1", rep)
    assert kv.tokens_seen(0) == 2048
    st = kv.stats()
    assert st["evictions"] == 2048 - 256 and st["device_error"] == 0
    assert rep.flips <= rep.near_ties


@pytest.mark.parametrize("split", [1, 2, 4, 8])
def test_decode_split_factors_agree_with_oracle(gpu, split):
    w = W.parity_slice(W.CONFIGS["cfg1"], budget=37, decode_steps=150)
    kv, orc = _pair(gpu, w)
    kv.set_option(gpu.OPT_DECODE_SPLIT, split)
    rep = Report()
    _run_decode(kv, orc, w, 0, w.decode_steps, rep)


def test_cfg2_slice_decode_bf16_mha(gpu):
    """Configuration 2's shape (d=128, bf16, MHA, c=1024) on 2 sequences x 4 heads, 3c+ tokens (3 idx cycles)."""
    w = W.parity_slice(W.CONFIGS["cfg2"], layers=1, batch=2, n_heads=4, n_kv_heads=4, decode_steps=3 * 1024 + 40)
    kv, orc = _pair(gpu, w)
    rep = Report()
    _run_decode(kv, orc, w, 0, w.decode_steps, rep, score_every=8)
    compare_state(kv, orc, rep)
    print("cfg2 slice", rep)


def test_cfg4_slice_prefill_then_gqa_decode(gpu):
    """Configuration 4's shape (GQA 4:1, d=128, bf16, c=2048, key scales): 4096-token prefill in 1024-token
    chunks, then one full idx cycle of decode steps."""
    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=8, n_kv_heads=2)
    kv, orc = _pair(gpu, w)
    rep = Report()
    _run_prefill(kv, orc, w, rep, [4096, 4096], 1024)
    _run_decode(kv, orc, w, 4096, 2048 + 64, rep, score_every=16)
    compare_state(kv, orc, rep)
    print("cfg4 slice", rep)


def test_cfg3_slice_chunked_prefill_mha(gpu):
    """Configuration 3's shape (MHA, c=2048, chunks of 512): 4 filling chunks + 8 steady chunks, then decode."""
    w = W.parity_slice(W.CONFIGS["cfg3"], layers=1, n_heads=2, n_kv_heads=2)
    kv, orc = _pair(gpu, w)
    rep = Report()
    _run_prefill(kv, orc, w, rep, [12 * 512], 512)
    _run_decode(kv, orc, w, 12 * 512, 48, rep)
    print("cfg3 slice", rep)


def test_cfg5_slice_ragged_gqa_prefill(gpu):
    """Configuration 5's shape (GQA 4:1, c=4096, chunks of 1024, ragged lengths, key scales): two sequences that
    end in different, partial chunks; then batched decode with every sequence at its own stream position."""
    w = W.parity_slice(W.CONFIGS["cfg5"], layers=1, batch=2, n_heads=4, n_kv_heads=1)
    lens = [2 * 4096 + 1024 + 517, 2 * 4096 + 100]
    kv, orc = _pair(gpu, w)
    rep = Report()
    _run_prefill(kv, orc, w, rep, lens, 1024)
    assert [kv.tokens_seen(b) for b in range(2)] == lens
    _run_decode(kv, orc, w, 0, 24, rep, starts=lens)
    print("cfg5 slice", rep)


@pytest.mark.parametrize("key_split", [1, 2])
@pytest.mark.parametrize("g,lens,chunk,budget", [
    (4, [2 * 1024 + 517, 2 * 1024 + 40], 512, 1024),   # GQA, ragged tails: a partial last tile and an empty second sub-tile
    (1, [5 * 384 + 200, 3 * 384], 384, 512),           # MHA, 1.5 pairs of tiles per chunk, chunks that wrap the idx cycle
    (8, [1300, 64], 256, 256),                         # eight heads per group: 16 tokens per sub-tile
    (2, [3 * 64 + 9, 50], 64, 96),                     # a first chunk of one key tile: the second block of a key-split pair has none
])
def test_two_tile_tensor_core_prefill_kernel(gpu, g, lens, chunk, budget, key_split):
    """The prefill kernel that gives a thread block two tiles of 128 query rows is only chosen for large grids;
    here it is forced on small ragged cases and followed in lock-step like the one-tile kernel - one block per tile
    pair, and pairs of blocks that split the key tiles and exchange row statistics and partial outputs."""
    w = W.parity_slice(W.CONFIGS["cfg5"], layers=1, batch=2, n_heads=g * 2, n_kv_heads=2, budget=budget, chunk=chunk)
    kv, orc = _pair(gpu, w)
    kv.set_option(gpu.OPT_PREFILL_PATH, 3)
    kv.set_option(gpu.OPT_PREFILL_KEY_SPLIT, key_split)
    rep = Report()
    _run_prefill(kv, orc, w, rep, lens, chunk)
    assert [kv.tokens_seen(b) for b in range(2)] == lens
    _run_decode(kv, orc, w, 0, 8, rep, starts=lens)
    assert kv.stats()["device_error"] == 0
    print("two-tile prefill g=%d" % g, rep)


@pytest.mark.parametrize("g,batch,hkv,budget,chunk,lens", [
    (1, 3, 1, 512, 384, [4 * 384 + 100, 2 * 384, 3 * 384 + 300]),   # 6 tile pairs: 4 in whole clusters, 2 split; ragged ends
    (4, 1, 1, 256, 320, [5 * 320 + 64]),                             # 5 tile pairs: 4 whole, 1 split; chunks wrap the cycle
    (2, 1, 3, 300, 256, [6 * 256 + 31]),                             # 6 pairs over 3 units
])
def test_two_tile_kernel_with_the_last_wave_split(gpu, g, batch, hkv, budget, chunk, lens):
    """The two-tile prefill kernel gives the tile pairs of a last, at most half-full wave to clusters of two thread blocks
    that halve the key tiles; the pairs of the full waves run in clusters too, one whole pair per block, exchanging
    nothing.  Option value 3 applies that rule for a machine of four SMs, so that small grids mix both kinds of cluster in
    one launch (here also with sequences that end early, i.e. blocks with nothing to do beside a busy partner)."""
    w = W.parity_slice(W.CONFIGS["cfg5"], layers=1, batch=batch, n_heads=g * hkv, n_kv_heads=hkv, budget=budget, chunk=chunk)
    kv, orc = _pair(gpu, w)
    kv.set_option(gpu.OPT_PREFILL_PATH, 3)
    kv.set_option(gpu.OPT_PREFILL_KEY_SPLIT, 3)
    rep = Report()
    _run_prefill(kv, orc, w, rep, lens, chunk)
    assert [kv.tokens_seen(b) for b in range(batch)] == lens
    _run_decode(kv, orc, w, 0, 6, rep, starts=lens)
    assert kv.stats()["device_error"] == 0


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("append", [0, 1])
@pytest.mark.parametrize("g,budget,chunk,lens", [
    (1, 300, 256, [5 * 256, 3 * 256]),        # budget not a multiple of the tile: both cached segments end in partial tiles
    (4, 512, 128, [9 * 128, 9 * 128 + 64]),   # GQA; the second sequence ends in a ragged chunk (append kernel for that call)
    (2, 200, 384, [4 * 384, 384]),            # chunks longer than the budget: several wraps per call
])
def test_fused_append_and_chunk_tiles_from_the_input_tensors(gpu, path, append, g, budget, chunk, lens):
    """When every chunk length of a call is a multiple of 128 the tensor-core kernels read the chunk's own key / value
    tiles from the caller's tensors and append the chunk themselves (two launches per call instead of three); forced
    to the separate append kernel the same calls must give the same result.  Both are followed by the oracle."""
    import torch

    w = W.parity_slice(W.CONFIGS["cfg5"], layers=1, batch=2, n_heads=g * 2, n_kv_heads=2, budget=budget, chunk=chunk)
    kv, orc = _pair(gpu, w)
    kv.set_option(gpu.OPT_PREFILL_PATH, path)
    kv.set_option(gpu.OPT_PREFILL_APPEND, append)
    rep = Report()
    _run_prefill(kv, orc, w, rep, lens, chunk)
    assert [kv.tokens_seen(b) for b in range(2)] == lens
    _run_decode(kv, orc, w, 0, 6, rep, starts=lens)
    # one more full chunk for both sequences, without read-outs in between: the launch count shows which way it went
    q, k, v = W.tokens_at(w, 0, [x + 6 for x in lens], chunk)
    l0 = kv.stats()["kernel_launches"]
    step_prefill(kv, orc, q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3), w.dtype, rep)
    torch.cuda.synchronize()
    read_outs = 3  # retained positions (twice) and scores of the comparison
    assert kv.stats()["kernel_launches"] - l0 - read_outs == (2 if append == 0 else 3)
    assert kv.stats()["device_error"] == 0


# ---------------------------------------------------------------------------------------------------------
# edge cases
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d,hq,hkv", [("bf16", 64, 4, 2), ("f32", 128, 2, 2), ("bf16", 128, 8, 1), ("f32", 64, 8, 4)])
def test_shapes_and_group_sizes(gpu, dtype, d, hq, hkv):
    w = W.parity_slice(W.CONFIGS["cfg1"], dtype=dtype, head_dim=d, n_heads=hq, n_kv_heads=hkv, batch=3, budget=24,
                       chunk=16, n_outliers=2)
    kv, orc = _pair(gpu, w)
    rep = Report()
    _run_prefill(kv, orc, w, rep, [40, 33, 16], 16)
    _run_decode(kv, orc, w, 0, 60, rep, starts=[40, 33, 16])


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_maximum_batch_with_changing_active_sets(gpu, dtype):
    """1024 sequences (the largest batch), a different random subset of them stepping each time: sequences drift apart,
    so every step mixes units that are still filling with units at different points of their eviction cycle."""
    w = W.parity_slice(W.CONFIGS["cfg1"], dtype=dtype, head_dim=64, n_heads=2, n_kv_heads=2, batch=1024, budget=12, chunk=0,
                       n_outliers=2)
    kv, orc = _pair(gpu, w)
    rep = Report()
    rs = np.random.default_rng(7)
    seen = np.zeros(w.batch, np.int64)
    for step in range(36):
        active = rs.random(w.batch) < (0.9 if step < 6 else 0.6)
        active[step % w.batch] = True
        q, k, v = W.tokens_at(w, 0, seen, 1)
        step_decode(kv, orc, q[0], k[0], v[0], w.dtype, rep, active=active.astype(np.uint8), check_scores=(step % 6 == 5))
        seen += active
    assert [kv.tokens_seen(b) for b in (0, 511, 1023)] == [int(seen[b]) for b in (0, 511, 1023)]
    assert kv.stats()["evictions"] == int(np.maximum(seen - w.budget, 0).sum())
    print("batch 1024", dtype, rep)


@pytest.mark.parametrize("c", [2, 3, 5])
def test_tiny_budgets(gpu, c):
    w = W.parity_slice(W.CONFIGS["cfg1"], budget=c, chunk=7, batch=2)
    kv, orc = _pair(gpu, w)
    rep = Report()
    _run_decode(kv, orc, w, 0, 4 * c + 3, rep)
    q, k, v = W.tokens(w, 0, 4 * c + 3, 4 * c + 3 + 7)          # a chunk larger than the budget, mid-cycle
    step_prefill(kv, orc, q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3), w.dtype, rep)
    _run_decode(kv, orc, w, 4 * c + 10, 2 * c + 1, rep)


@pytest.mark.parametrize("c,m", [(8, 3), (8, 5), (8, 8), (8, 20), (16, 4), (16, 24), (12, 7)])
def test_chunks_that_wrap_the_eviction_cycle(gpu, c, m):
    """Chunks that do not divide the budget, straddle the wrap of idx, or exceed the budget (several wraps)."""
    w = W.parity_slice(W.CONFIGS["cfg1"], budget=c, chunk=m, batch=2, n_heads=2, n_kv_heads=2)
    kv, orc = _pair(gpu, w)
    rep = Report()
    total = 6 * max(c, m) + 5
    _run_prefill(kv, orc, w, rep, [total, total - m - 2], m)
    _run_decode(kv, orc, w, 0, 3, rep, starts=[total, total - m - 2])
    # a chunk right after decode steps: arbitrary cycle position
    t0 = [total + 3, total - m + 1]
    q, k, v = W.tokens_at(w, 0, t0, m)
    step_prefill(kv, orc, q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3), w.dtype, rep)


@pytest.mark.parametrize("rule", [1, 2])
def test_score_free_rules_match_closed_structure(gpu, rule):
    """With the score-free rules the retained set depends on the schedule alone: chunked and token-by-token
    feeding retain the same tokens, and they equal the oracle's."""
    from oracle import Oracle

    w = W.parity_slice(W.CONFIGS["cfg1"], budget=16, chunk=6, batch=1, n_heads=1, n_kv_heads=1)
    a = gpu.TreeKV(16, 1, 1, 64, "f32", 1, 6)
    b = gpu.TreeKV(16, 1, 1, 64, "f32", 1, 6)
    a.set_rule(rule); b.set_rule(rule)
    orc = Oracle(16, 1, 1, 64, 1, rule=rule)
    import torch

    T = 16 * 7 + 6
    q, k, v = W.tokens(w, 0, 0, T)
    tq, tk, tv = (torch.from_numpy(x).cuda() for x in (q, k, v))
    for t in range(0, T, 6):
        n = min(6, T - t)
        for s in range(t, t + n):
            a.decode_step(tq[s], tk[s], tv[s])
            orc.decode_step(q[s], k[s], v[s])
        b.prefill_chunk(tq[t:t + n].transpose(0, 1).contiguous(), tk[t:t + n].transpose(0, 1).contiguous(),
                        tv[t:t + n].transpose(0, 1).contiguous())
        pa = a.retained_positions()[0].cpu().numpy()
        pb = b.retained_positions()[0].cpu().numpy()
        assert np.array_equal(pa, pb)
        assert np.array_equal(pa, orc.retained_positions()[0])


@pytest.mark.parametrize("dtype,d,g,path", [("bf16", 128, 4, 0), ("bf16", 128, 1, 3), ("f32", 64, 2, 0), ("bf16", 64, 8, 0)])
def test_accumulated_criterion(gpu, dtype, d, g, path):
    """Section 4.1 "Importance Score": the accumulated attention weight S as the criterion instead of S / C.  Chunked
    prefill (tensor-core and CUDA-core kernels), decode (both kernels) and a one-shot block prefill in lock-step with
    the oracle under the same rule; on these inputs the rule retains other tokens than the average does."""
    from lockstep import step_oneshot
    from oracle import RULE_ACCUMULATED, Oracle

    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=2 * g, n_kv_heads=2, head_dim=d, dtype=dtype, budget=96,
                       chunk=128)
    kv = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, d, dtype, 2, 128)
    kv.set_rule(gpu.RULE_ACCUMULATED)
    if path:
        kv.set_option(gpu.OPT_PREFILL_PATH, path)
    orc = Oracle(w.budget, w.n_heads, w.n_kv_heads, d, 2, rule=RULE_ACCUMULATED)
    avg = Oracle(w.budget, w.n_heads, w.n_kv_heads, d, 2)
    rep = Report()
    q, k, v = W.tokens(w, 0, 0, 128)
    qt, kt, vt = (x.transpose(1, 0, 2, 3) for x in (q, k, v))
    step_oneshot(kv, orc, qt, kt, vt, 8, dtype, rep, lens=[128, 64])
    avg.prefill_oneshot(qt, kt, vt, 8, [128, 64])
    seen = [128, 64]
    for lens in ([128, 128], [77, 128], [128, 0]):
        qc, kc, vc = W.tokens_at(w, 0, seen, 128)
        step_prefill(kv, orc, qc.transpose(1, 0, 2, 3), kc.transpose(1, 0, 2, 3), vc.transpose(1, 0, 2, 3), dtype, rep,
                     chunk_lens=lens)
        avg.prefill_chunk(qc.transpose(1, 0, 2, 3), kc.transpose(1, 0, 2, 3), vc.transpose(1, 0, 2, 3), lens)
        seen = [a + b for a, b in zip(seen, lens)]
    for _ in range(w.budget + 30):
        qd, kd, vd = W.tokens_at(w, 0, seen, 1)
        step_decode(kv, orc, qd[0], kd[0], vd[0], dtype, rep)
        avg.decode_step(qd[0], kd[0], vd[0])
        seen = [a + 1 for a in seen]
    assert kv.stats()["device_error"] == 0 and rep.decisions > 0
    assert not np.array_equal(orc.retained_positions()[0], avg.retained_positions()[0])


def test_inactive_sequences_are_untouched(gpu):
    import torch

    w = W.parity_slice(W.CONFIGS["cfg1"], budget=10, batch=3)
    kv, orc = _pair(gpu, w)
    rep = Report()
    seen = [0, 0, 0]
    for step in range(45):
        act = [1, step % 3 != 0, step % 2]
        q, k, v = W.tokens_at(w, 0, seen, 1)
        step_decode(kv, orc, q[0], k[0], v[0], w.dtype, rep, active=act)
        seen = [s + (1 if a else 0) for s, a in zip(seen, act)]
    assert [kv.tokens_seen(b) for b in range(3)] == seen
    # an inactive row of `out` is not written
    out = torch.full((3, 4, 64), 7.0, device="cuda")
    q, k, v = W.tokens_at(w, 0, seen, 1)
    kv.decode_step(torch.from_numpy(q[0]).cuda(), torch.from_numpy(k[0]).cuda(), torch.from_numpy(v[0]).cuda(), out=out,
                   active=[0, 1, 0])
    assert torch.all(out[0] == 7.0) and torch.all(out[2] == 7.0) and not torch.all(out[1] == 7.0)


def test_stream_shorter_than_budget_is_full_attention(gpu):
    """Nothing is evicted while the stream fits the budget; the output is plain causal softmax attention
    (checked against torch in fp64 as well as the oracle)."""
    import torch

    w = W.parity_slice(W.CONFIGS["cfg1"], budget=64, decode_steps=64)
    kv, orc = _pair(gpu, w)
    rep = Report()
    q, k, v = W.tokens(w, 0, 0, 64)
    outs = []
    for t in range(64):
        step_decode(kv, orc, q[t], k[t], v[t], w.dtype, rep)
    tq, tk, tv = (torch.from_numpy(x).double() for x in (q, k, v))
    kv2 = gpu.TreeKV(64, 4, 4, 64, "f32", 1, 0)
    for t in range(64):
        o = kv2.decode_step(tq[t].float().cuda(), tk[t].float().cuda(), tv[t].float().cuda()).cpu().double()
        s = torch.einsum("hd,thd->ht", tq[t, 0], tk[: t + 1, 0]) / 8.0
        ref = torch.einsum("ht,thd->hd", torch.softmax(s, -1), tv[: t + 1, 0])
        assert (o[0] - ref).abs().max() < 1e-5
    assert kv2.stats()["evictions"] == 0
    assert kv2.retained_positions()[0].cpu().numpy()[0, 0].tolist() == list(range(64))


def test_bitwise_reproducible(gpu):
    """Scores are accumulated in a fixed order (no floating-point atomics): two runs give identical bits."""
    import torch

    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=96, chunk=32)
    results = []
    for _ in range(2):
        kv = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
        outs = []
        for c in range(8):
            q, k, v = W.tokens(w, 0, c * 32, (c + 1) * 32)
            t = [torch.from_numpy(x.transpose(1, 0, 2, 3).copy()).cuda().bfloat16() for x in (q, k, v)]
            outs.append(kv.prefill_chunk(*t).clone())
        q, k, v = W.tokens(w, 0, 256, 256 + 150)
        for s in range(150):
            t = [torch.from_numpy(x[s]).cuda().bfloat16() for x in (q, k, v)]
            outs.append(kv.decode_step(*t).clone())
        results.append((torch.cat([o.flatten() for o in outs]), kv.scores().clone(), kv.retained_positions()[0].clone()))
    for x, y in zip(*results):
        assert torch.equal(x, y)


@pytest.mark.parametrize("shape", ["one_block_per_unit", "clusters"])
def test_chained_launches_match_synchronised_launches(gpu, shape):
    """The kernels of consecutive calls overlap at their edges (programmatic dependent launch; the decode kernel also
    prefetches into L2 with a token count that may be one step old).  A stream of prefill chunks and decode steps
    enqueued without any synchronisation must give the same bits as the same calls with a device synchronisation
    after each one - on a batch large enough for one block per unit and on a small one that runs as clusters."""
    import torch

    if shape == "one_block_per_unit":
        w = W.parity_slice(W.CONFIGS["cfg2"], layers=1, batch=20, n_heads=8, n_kv_heads=8, budget=160, chunk=64)
    else:
        w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=1, n_heads=8, n_kv_heads=2, budget=1024, chunk=256)
    n_chunks, steps = w.budget // w.chunk + 3, 200
    qs, ks, vs = W.tokens(w, 0, 0, n_chunks * w.chunk + steps)
    dev = [torch.from_numpy(x).cuda().bfloat16() for x in (qs, ks, vs)]          # [T, B, H, d]
    chunks = [[x[c * w.chunk:(c + 1) * w.chunk].transpose(0, 1).contiguous() for x in dev] for c in range(n_chunks)]
    t0 = n_chunks * w.chunk
    results = []
    for sync in (False, True):
        kv = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
        outs_p = [torch.empty_like(chunks[0][0]) for _ in range(n_chunks)]
        outs_d = torch.empty((steps, w.batch, w.n_heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        for c in range(n_chunks):
            kv.prefill_chunk(*chunks[c], out=outs_p[c])
            if sync:
                torch.cuda.synchronize()
        for s in range(steps):
            kv.decode_step(dev[0][t0 + s], dev[1][t0 + s], dev[2][t0 + s], out=outs_d[s])
            if sync:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        assert kv.stats()["device_error"] == 0
        results.append((torch.stack(outs_p).clone(), outs_d.clone(), kv.scores().clone(), kv.retained_positions()[0].clone()))
    for x, y in zip(*results):
        assert torch.equal(x, y)


def test_eviction_stream_gives_the_same_bits_and_follows_the_oracle(gpu):
    """With the eviction stream on, a chunk's score update + eviction runs on a stream of the context's own while the
    caller's stream goes on (here: with the next layer's chunk).  A stack of four contexts driven chunk after chunk and
    then step after step without any synchronisation must end in exactly the state, and give exactly the outputs, of
    the same stack with everything on one stream; and one context with the option on is followed by the oracle."""
    import torch

    w = W.parity_slice(W.CONFIGS["cfg3"], layers=4, batch=1, n_heads=4, n_kv_heads=4, budget=512, chunk=256)
    n_chunks, steps = 6, 40
    ins = []
    for layer in range(w.layers):
        qs, ks, vs = W.tokens(w, layer, 0, n_chunks * w.chunk + steps)
        ins.append([torch.from_numpy(x).cuda().bfloat16() for x in (qs, ks, vs)])   # [T, B, H, d]
    t0 = n_chunks * w.chunk
    results = []
    for side in (0, 1):
        ctxs = [gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk) for _ in range(w.layers)]
        for kv in ctxs:
            kv.set_option(gpu.OPT_EVICTION_STREAM, side)
        outs_p = torch.empty((n_chunks, w.layers, w.batch, w.chunk, w.n_heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
        outs_d = torch.empty((steps, w.layers, w.batch, w.n_heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
        chunks = [[[x[c * w.chunk:(c + 1) * w.chunk].transpose(0, 1).contiguous() for x in ins[layer]]
                   for layer in range(w.layers)] for c in range(n_chunks)]
        torch.cuda.synchronize()
        for c in range(n_chunks):
            for layer, kv in enumerate(ctxs):
                kv.prefill_chunk(*chunks[c][layer], out=outs_p[c, layer])
        for s in range(steps):
            for layer, kv in enumerate(ctxs):
                kv.decode_step(ins[layer][0][t0 + s], ins[layer][1][t0 + s], ins[layer][2][t0 + s], out=outs_d[s, layer])
        state = [(kv.scores().clone(), kv.retained_positions()[0].clone()) for kv in ctxs]
        torch.cuda.synchronize()
        assert all(kv.stats()["device_error"] == 0 for kv in ctxs)
        results.append((outs_p.clone(), outs_d.clone(), state))
        if side:
            ctxs[0].set_option(gpu.OPT_EVICTION_STREAM, 0)   # switching it off again synchronises and frees the stream
        del ctxs
    assert torch.equal(results[0][0], results[1][0]) and torch.equal(results[0][1], results[1][1])
    for (sa, pa), (sb, pb) in zip(results[0][2], results[1][2]):
        assert torch.equal(sa, sb) and torch.equal(pa, pb)

    # calls of every other kind right behind a chunk, without synchronising: each orders itself behind the eviction
    kv = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    ref = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    kv.set_option(gpu.OPT_EVICTION_STREAM, 1)
    for c in range(4):
        kv.prefill_chunk(*chunks[c][0]); ref.prefill_chunk(*chunks[c][0])
    img, seen = kv.export_state()                       # export behind a pending eviction
    img_r, seen_r = ref.export_state()
    assert seen == seen_r and torch.equal(img, img_r)
    kv.prefill_chunk(*chunks[4][0])
    kv.reset()                                          # reset behind a pending eviction, then the same stream again
    kv.import_state(img, seen)
    kv.prefill_chunk(*chunks[4][0]); ref.prefill_chunk(*chunks[4][0])
    assert torch.equal(kv.scores(), ref.scores()) and torch.equal(kv.retained_positions()[0], ref.retained_positions()[0])
    assert kv.stats()["device_error"] == 0
    del kv, ref

    w1 = W.parity_slice(W.CONFIGS["cfg5"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=256, chunk=128)
    kv, orc = _pair(gpu, w1)
    kv.set_option(gpu.OPT_EVICTION_STREAM, 1)
    rep = Report()
    _run_prefill(kv, orc, w1, rep, [7 * 128 + 50, 5 * 128], 128)
    _run_decode(kv, orc, w1, 0, 20, rep, starts=[7 * 128 + 50, 5 * 128])
    assert kv.stats()["device_error"] == 0


def test_eviction_beside_an_attention_grid_that_leaves_few_sms_free(gpu):
    """An attention grid just below the machine (32 units x 4 query tiles = 128 thread blocks on 148 SMs) leaves 20 SMs
    to the eviction kernel of the previous layer, which is then launched with 20 blocks for its 32 units: some blocks
    take two units in turn.  Same bits as on one stream, and in lock-step with the oracle, ragged and inactive
    sequences included."""
    import torch

    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=32, n_kv_heads=16, budget=192, chunk=256)
    if torch.cuda.get_device_properties(0).multi_processor_count <= 128:
        pytest.skip("the case needs more than 128 SMs")
    kv, orc = _pair(gpu, w)
    ref = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    kv.set_option(gpu.OPT_EVICTION_STREAM, 1)
    rep = Report()
    seen = [0, 0]
    for lens in ([256, 256], [256, 256], [256, 131], [256, 0], [256, 256]):
        q, k, v = W.tokens_at(w, 0, seen, 256)
        q, k, v = (x.transpose(1, 0, 2, 3) for x in (q, k, v))
        step_prefill(kv, orc, q, k, v, w.dtype, rep, chunk_lens=lens)
        ref.prefill_chunk(*(torch.from_numpy(np.ascontiguousarray(x)).cuda().bfloat16() for x in (q, k, v)), chunk_lens=lens)
        seen = [a + b for a, b in zip(seen, lens)]
        assert torch.equal(kv.scores(), ref.scores()) and torch.equal(kv.retained_positions()[0], ref.retained_positions()[0])
    assert kv.stats()["device_error"] == 0 and rep.decisions > 0


@pytest.mark.parametrize("pinned", [True, False])
def test_host_entry_points_match_device_entry_points(gpu, pinned):
    """Page-locked host tensors are read by the decode kernel directly; pageable ones go through staging copies."""
    import torch

    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=64, chunk=32)
    a = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    b = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    for c in range(4):
        q, k, v = W.tokens(w, 0, c * 32, (c + 1) * 32)
        h = [torch.from_numpy(x.transpose(1, 0, 2, 3).copy()).bfloat16().pin_memory() for x in (q, k, v)]
        oh = torch.empty_like(h[0]).pin_memory()
        b.prefill_chunk_host(h[0], h[1], h[2], oh)
        od = a.prefill_chunk(*[x.cuda() for x in h])
        torch.cuda.synchronize()
        assert torch.equal(od.cpu(), oh)
    q, k, v = W.tokens(w, 0, 128, 128 + 40)
    for s in range(40):
        h = [torch.from_numpy(x[s]).bfloat16() for x in (q, k, v)]
        oh = torch.empty_like(h[0])
        if pinned:
            h = [x.pin_memory() for x in h]
            oh = oh.pin_memory()
        b.decode_step_host(h[0], h[1], h[2], oh)
        od = a.decode_step(*[x.cuda() for x in h])
        torch.cuda.synchronize()
        assert torch.equal(od.cpu(), oh)
    assert torch.equal(a.retained_positions()[0], b.retained_positions()[0])


def test_host_decode_pipeline_without_intermediate_syncs(gpu):
    """Many host-tensor decode steps over three contexts (layers), enqueued back to back on a side stream with no
    synchronisation in between and mixed with device-tensor calls: every output and the final caches must equal
    those of the device entry point."""
    import torch

    w = W.parity_slice(W.CONFIGS["cfg2"], layers=3, batch=2, n_heads=4, n_kv_heads=4, budget=48, chunk=0)
    host = [gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, 0) for _ in range(w.layers)]
    dev = [gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, 0) for _ in range(w.layers)]
    steps = 150
    ins = []
    for layer in range(w.layers):
        q, k, v = W.tokens(w, layer, 0, steps)
        ins.append([torch.from_numpy(x).bfloat16().pin_memory() for x in (q, k, v)])
    outs_h = [torch.zeros((steps, w.batch, w.n_heads, w.head_dim), dtype=torch.bfloat16).pin_memory() for _ in range(w.layers)]
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for s in range(steps):
            for layer in range(w.layers):
                q, k, v = ins[layer]
                if s % 7 == 3 and layer == 1:   # a device-tensor call in the middle of the pipeline, same stream
                    o = host[layer].decode_step(q[s].cuda(non_blocking=True), k[s].cuda(non_blocking=True),
                                                v[s].cuda(non_blocking=True))
                    outs_h[layer][s].copy_(o, non_blocking=True)
                else:
                    host[layer].decode_step_host(q[s], k[s], v[s], outs_h[layer][s])
    side.synchronize()
    for layer in range(w.layers):
        q, k, v = ins[layer]
        for s in range(steps):
            od = dev[layer].decode_step(q[s].cuda(), k[s].cuda(), v[s].cuda())
            assert torch.equal(od.cpu(), outs_h[layer][s]), (layer, s)
        assert torch.equal(dev[layer].retained_positions()[0], host[layer].retained_positions()[0])
        assert torch.equal(dev[layer].scores(), host[layer].scores())
        assert host[layer].stats()["device_error"] == 0


def test_argument_and_state_errors(gpu):
    import torch

    kv = gpu.TreeKV(16, 4, 4, 64, "f32", 2, 0)
    x = torch.zeros((2, 4, 64), device="cuda")
    # decode-only context refuses prefill
    xc = torch.zeros((2, 4, 4, 64), device="cuda")
    assert gpu.treekv_prefill_chunk(kv._h, xc.data_ptr(), xc.data_ptr(), xc.data_ptr(), xc.data_ptr(), None, 4) == 2
    # misaligned pointer
    assert gpu.treekv_decode_step(kv._h, x.data_ptr() + 4, x.data_ptr(), x.data_ptr(), x.data_ptr()) == 1
    kv2 = gpu.TreeKV(16, 4, 4, 64, "f32", 2, 8)
    assert gpu.treekv_prefill_chunk(kv2._h, xc.data_ptr(), xc.data_ptr(), xc.data_ptr(), xc.data_ptr(), [9, 1], 16) == 1
    assert gpu.treekv_prefill_chunk(kv2._h, xc.data_ptr(), xc.data_ptr(), xc.data_ptr(), xc.data_ptr(), [5, 1], 4) == 1
    # nothing was enqueued by the refused calls
    assert kv2.tokens_seen(0) == 0 and kv2.stats()["kernel_launches"] == 1
    # reset brings back the empty cache
    kv.decode_step(x, x, x)
    assert kv.tokens_seen(0) == 1
    kv.reset()
    assert kv.tokens_seen(0) == 0
    assert kv.retained_positions()[1].cpu().numpy().tolist() == [[0] * 4] * 2


def test_device_side_give_up_surfaces_as_timeout_status(gpu):
    """A bounded wait that gives up must reach the caller as TREEKV_ERR_TIMEOUT and be cleared by a reset.  No real
    kernel ever gives up in a healthy run, so the library's self-test kernel makes one wait run out: a few dozen
    polls of a barrier that nothing signals, nothing asynchronous outstanding, the cache untouched."""
    import torch

    kv = gpu.TreeKV(16, 4, 4, 64, "f32", 2, 0)
    x = torch.randn((2, 4, 64), device="cuda")
    kv.decode_step(x, x, x)
    assert kv.stats()["device_error"] == 0
    assert gpu.treekv_selftest_wait_giveup(kv._h, 0) == 1 and gpu.treekv_selftest_wait_giveup(kv._h, 5000) == 1
    assert gpu.treekv_selftest_wait_giveup(kv._h, 48) == 0
    st = kv.stats(check=False)
    assert st["status"] == 6 and st["device_error"] == 64
    assert gpu.status_string(6) == "device-side wait timed out"
    with pytest.raises(gpu.TreeKVError):
        kv.stats()
    # the context and the GPU stay usable: the cache was not touched, and a reset clears the error word
    assert kv.tokens_seen(0) == 1 and kv.retained_positions()[1].cpu().numpy().tolist() == [[1] * 4] * 2
    kv.reset()
    st = kv.stats()
    assert st["device_error"] == 0 and st["status"] == 0
    kv.decode_step(x, x, x)
    torch.cuda.synchronize()
    assert kv.stats()["device_error"] == 0 and kv.tokens_seen(0) == 1
