"""GPU parity with in-cache positions (Section 4.1 "Position Encoding": positions are re-assigned after eviction): q and
k arrive without rotary embedding, the library encodes the key in cache slot j at position j and the query at its
own slot.  Both sides take the same single-precision cos / sin tables as input and compute the rotated operands with
the same two fp32 operations per output, rounded to the cache dtype, so the usual bars apply unchanged: retained
positions exactly up to counted near-ties, outputs within 2e-2 (bf16) / 1e-4 (fp32), scores within 1e-3.
"""
import numpy as np
import pytest

import workloads as W
from lockstep import Report, run_decode, run_prefill, step_oneshot

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


def _pair(binding, w, max_chunk, ns=0, nr=0):
    import torch
    from oracle import Oracle

    kv = binding.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, max_chunk)
    orc = Oracle(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.batch, n_sink=ns, n_recent=nr)
    if ns or nr:
        kv.set_protection(ns, nr)
    cos, sin = W.rope_tables(w.budget + max(1, max_chunk), w.head_dim, w.rope_base)
    kv.set_positions(torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda())
    orc.set_rope(cos, sin, round_bf16=(w.dtype == "bf16"))
    return kv, orc


_DECODE_CASES = [("bf16", 128, 8, 2, 0, 40), ("bf16", 64, 2, 2, 2, 40), ("f32", 64, 4, 4, 0, 40), ("f32", 128, 4, 1, 4, 40),
                 ("bf16", 128, 2, 2, 8, 40), ("bf16", 128, 8, 2, 1, 300), ("bf16", 64, 4, 1, 4, 200)]


@pytest.mark.parametrize("dtype,d,hq,hkv,split,budget,path",
                         [c + (0,) for c in _DECODE_CASES] + [c + (1,) for c in _DECODE_CASES if c[0] == "bf16"])
def test_decode_with_in_cache_positions(gpu, dtype, d, hq, hkv, split, budget, path):
    """Both decode kernels: the mma.sync kernel (bf16, automatic) encodes each key tile at its slots in shared memory,
    the CUDA-core kernel (path 1, and fp32) in registers; budgets of several tiles per warp put the segment boundary
    of the cycle layout and ragged tails inside tiles."""
    w = W.parity_slice(W.CONFIGS["cfg2"], layers=1, batch=2, n_heads=hq, n_kv_heads=hkv, head_dim=d, dtype=dtype, budget=budget,
                       chunk=0, rotate=False)
    kv, orc = _pair(gpu, w, 0)
    if path:
        kv.set_option(gpu.OPT_DECODE_PATH, path)
    if split:
        kv.set_option(gpu.OPT_DECODE_SPLIT, split)
    rep = Report()
    run_decode(kv, orc, w, 0, budget + (2 * budget if budget <= 40 else budget // 2) + 9, rep)
    assert kv.stats()["device_error"] == 0 and rep.decisions > 0


@pytest.mark.parametrize("dtype,d,g,path", [("bf16", 128, 4, 0), ("bf16", 128, 4, 1), ("bf16", 128, 4, 3), ("bf16", 128, 1, 2),
                                            ("f32", 64, 1, 0), ("bf16", 64, 2, 0)])
def test_chunked_prefill_then_decode_with_in_cache_positions(gpu, dtype, d, g, path):
    """bf16 / head_dim 128 takes the tensor-core kernels (paths 0, 2, 3), which run on keys and queries that a kernel of
    their own has encoded at their slots first; path 1, fp32 and head_dim 64 take the CUDA-core kernel, which encodes
    while it streams."""
    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=2 * g, n_kv_heads=2, head_dim=d, dtype=dtype, budget=96,
                       chunk=64, rotate=False)
    kv, orc = _pair(gpu, w, 64)
    if path:
        kv.set_option(gpu.OPT_PREFILL_PATH, path)
    rep = Report()
    run_prefill(kv, orc, w, rep, [5 * 64 + 20, 3 * 64], 64)
    run_decode(kv, orc, w, 0, 110, rep, starts=[5 * 64 + 20, 3 * 64])
    assert kv.stats()["device_error"] == 0


def test_larger_chunked_prefill_with_in_cache_positions_on_the_tensor_cores(gpu):
    """Several key tiles per thread block, chunks that wrap the eviction cycle, a ragged tail, protected tokens."""
    w = W.parity_slice(W.CONFIGS["cfg3"], layers=1, batch=2, n_heads=2, n_kv_heads=2, budget=384, chunk=256, rotate=False)
    kv, orc = _pair(gpu, w, 256, ns=4, nr=60)
    rep = Report()
    run_prefill(kv, orc, w, rep, [5 * 256 + 77, 4 * 256], 256)
    run_decode(kv, orc, w, 0, 20, rep, starts=[5 * 256 + 77, 4 * 256])
    assert kv.stats()["device_error"] == 0


def test_positions_with_protected_tokens_and_oneshot_prefill(gpu):
    # the paper's language-model set-up in small: sinks + recent window + re-assigned positions, token by token
    w = W.parity_slice(W.CONFIGS["cfg2"], layers=1, batch=1, n_heads=2, n_kv_heads=2, budget=64, chunk=0, rotate=False)
    kv, orc = _pair(gpu, w, 0, ns=4, nr=28)
    rep = Report()
    run_decode(kv, orc, w, 0, 64 + 3 * 32 + 5, rep)
    # one-shot block prefill with positions, then decode
    w2 = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=128, chunk=512, rotate=False)
    kv2, orc2 = _pair(gpu, w2, 512)
    q, k, v = W.tokens(w2, 0, 0, 512)
    step_oneshot(kv2, orc2, q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3), 32, w2.dtype, rep,
                 lens=[512, 256])
    run_decode(kv2, orc2, w2, 0, 40, rep, starts=[512, 256])
    assert kv.stats()["device_error"] == 0 and kv2.stats()["device_error"] == 0


def test_without_eviction_matches_caller_side_rotation(gpu):
    """While nothing has been evicted, slot = stream position: the library with in-cache positions must give what the
    position-agnostic library gives on inputs the generator rotated itself (the two differ only by the rounding of
    the rotation: fp32 here, so 1e-4 holds)."""
    import torch

    base = W.parity_slice(W.CONFIGS["cfg1"], batch=1, budget=64, chunk=0)
    raw = W.parity_slice(base, rotate=False)
    a = gpu.TreeKV(64, 4, 4, 64, "f32", 1, 0)
    cos, sin = W.rope_tables(65, 64, base.rope_base)
    a.set_positions(torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda())
    b = gpu.TreeKV(64, 4, 4, 64, "f32", 1, 0)
    qa, ka, va = W.tokens(raw, 0, 0, 64)
    qb, kb, vb = W.tokens(base, 0, 0, 64)
    for t in range(64):
        oa = a.decode_step(*(torch.from_numpy(x[t]).cuda() for x in (qa, ka, va)))
        ob = b.decode_step(*(torch.from_numpy(x[t]).cuda() for x in (qb, kb, vb)))
        assert (oa - ob).abs().max().item() <= 1e-4, t


def test_argument_and_state_errors(gpu):
    import torch

    kv = gpu.TreeKV(16, 2, 2, 64, "f32", 1, 8)
    cos = torch.zeros((24, 32), device="cuda"); sin = torch.zeros((24, 32), device="cuda")
    assert gpu.treekv_set_positions(kv._h, cos.data_ptr(), sin.data_ptr(), 23) == 1      # too few slots
    assert gpu.treekv_set_positions(kv._h, cos.data_ptr(), None, 24) == 1
    assert gpu.treekv_set_positions(kv._h, cos.data_ptr(), sin.data_ptr(), 24) == 0
    assert gpu.treekv_set_positions(kv._h, None, None, 0) == 0
    x = torch.zeros((1, 2, 64), device="cuda")
    kv.decode_step(x, x, x)
    assert gpu.treekv_set_positions(kv._h, cos.data_ptr(), sin.data_ptr(), 24) == 2      # the cache is in use
    # tensor-core prefill with positions keeps the encoded queries in a buffer sized for max_chunk: a larger stride of the
    # caller's tensors is refused before anything is enqueued
    kv2 = gpu.TreeKV(256, 2, 2, 128, "bf16", 1, 128)
    cos2 = torch.zeros((384, 64), device="cuda"); sin2 = torch.zeros((384, 64), device="cuda")
    kv2.set_positions(cos2, sin2)
    y = torch.zeros((1, 256, 2, 128), device="cuda", dtype=torch.bfloat16)
    with pytest.raises(gpu.TreeKVError) as ei:
        kv2.prefill_chunk(y, y, y, chunk_lens=[128])
    assert ei.value.status == 4 and kv2.tokens_seen(0) == 0
    kv2.prefill_chunk(y[:, :128].contiguous(), y[:, :128].contiguous(), y[:, :128].contiguous())
    assert kv2.tokens_seen(0) == 128 and kv2.stats()["device_error"] == 0
