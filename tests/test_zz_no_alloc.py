"""treekv_prefill_chunk_static_scratch against treekv_prefill_chunk, and against the oracle.

The static-scratch entry point exists for callers that are not allowed to allocate device memory at the point
where they run (a frozen memory pool, someone else's allocator, a loop that cannot take cudaMalloc's
synchronisation): its per-call scratch is a fixed area inside the library instead of caller-sized memory.
It must give what the regular entry point gives: bit for bit when that one is told to use the same (CUDA-core)
attention kernel, and within the parity tolerances when it runs the tensor-core kernel.  Several calls in a row
are checked, because the area is shared by all calls and keeps the previous call's contents.  This file is
collected last on purpose.
"""
import numpy as np
import pytest

import workloads as W
from lockstep import Report, step_prefill

pytestmark = pytest.mark.gpu


def _tk():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2501_04987_b200 import _build

    _build.build()
    from paper_2501_04987_b200 import binding as tk

    return torch, tk


def _chunk(torch, w, call, m):
    q, k, v = W.tokens(w, 0, call * m, (call + 1) * m)
    return tuple(torch.from_numpy(np.ascontiguousarray(x.transpose(1, 0, 2, 3))).cuda().bfloat16() for x in (q, k, v))


@pytest.mark.parametrize("budget,m,calls", [
    (96, 64, [[64, 64], [64, 50], [64, 64]]),    # filling, first evictions, a ragged chunk that wraps the eviction cycle
    (24, 64, [[64, 64], [64, 17], [30, 64]]),    # chunks longer than the budget: several wraps per call, rows re-based
])
def test_static_scratch_prefill_matches_regular_entry_point(budget, m, calls):
    torch, tk = _tk()
    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=budget, chunk=m)
    same = tk.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    same.set_option(tk.OPT_PREFILL_PATH, 1)   # the CUDA-core attention kernel, as the static-scratch call runs
    tc = tk.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)   # tensor-core kernel
    alt = tk.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    stream = torch.cuda.current_stream().cuda_stream
    tol = 2e-2  # bf16 output tolerance used by the parity tests
    for call, lens in enumerate(calls):
        tq, tkk, tv = _chunk(torch, w, call, m)
        outs = {}
        for name, ctx, fn in (("same", same, tk.treekv_prefill_chunk), ("tc", tc, tk.treekv_prefill_chunk),
                              ("alt", alt, tk.treekv_prefill_chunk_static_scratch)):
            outs[name] = torch.zeros_like(tq)
            st = fn(ctx._h, tq.data_ptr(), tkk.data_ptr(), tv.data_ptr(), outs[name].data_ptr(), lens, m, stream)
            assert st == 0, tk.status_string(st)
        torch.cuda.synchronize()
        # same arithmetic: identical bits in outputs, retained sets and scores
        assert torch.equal(outs["same"], outs["alt"])
        assert torch.equal(same.retained_positions()[0], alt.retained_positions()[0])
        assert torch.equal(same.retained_positions()[1], alt.retained_positions()[1])
        assert torch.equal(same.scores(), alt.scores())
        assert [alt.tokens_seen(b) for b in range(2)] == [same.tokens_seen(b) for b in range(2)]
        # tensor-core kernel: within the parity tolerances (retained sets are compared through the oracle below)
        assert (outs["tc"].float() - outs["alt"].float()).abs().max().item() <= tol
    assert alt.stats()["device_error"] == 0


def test_static_scratch_prefill_in_lockstep_with_the_oracle():
    """bf16, d = 128, GQA 4:1: the static-scratch call against the fp64 oracle call by call (retained positions exactly
    up to counted near-ties, scores within 1e-3, outputs within 2e-2), through fill, evictions and a wrap."""
    torch, tk = _tk()
    from oracle import Oracle

    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=80, chunk=48)
    kv = tk.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    orc = Oracle(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.batch)
    rep = Report()
    for call, lens in enumerate([[48, 48], [48, 31], [48, 48], [7, 48], [48, 48]]):
        q, k, v = W.tokens(w, 0, call * 48, (call + 1) * 48)
        step_prefill(kv, orc, q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3), w.dtype, rep,
                     chunk_lens=lens, method="prefill_chunk_static_scratch")
    assert kv.stats()["device_error"] == 0 and rep.decisions > 0
    print("static scratch", rep)


def test_static_scratch_rejects_oversized_calls():
    torch, tk = _tk()
    # 8 sequences x 8 KV heads, budget 4096, chunk 1024: about 90 MiB of scratch, far beyond the 16 MiB area
    kv = tk.TreeKV(4096, 32, 8, 128, "bf16", 8, 1024)
    x = torch.zeros((8, 1024, 32, 128), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((8, 1024, 8, 128), dtype=torch.bfloat16, device="cuda")
    st = tk.treekv_prefill_chunk_static_scratch(kv._h, x.data_ptr(), y.data_ptr(), y.data_ptr(), x.data_ptr(), None, 1024,
                                                torch.cuda.current_stream().cuda_stream)
    assert st == 4
    assert kv.tokens_seen(0) == 0 and kv.stats()["kernel_launches"] == 1   # nothing was enqueued
