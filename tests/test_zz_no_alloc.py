"""treekv_prefill_chunk_static_scratch against treekv_prefill_chunk.

The static-scratch entry point exists for callers that are not allowed to allocate device memory at the point
where they run (a frozen memory pool, someone else's allocator, a loop that cannot take cudaMalloc's
synchronisation): its per-call scratch is a fixed area inside the library instead of caller-sized memory.
It must give exactly what the regular entry point gives.  Two calls in a row are checked, because the area is
shared by all calls and keeps the previous call's contents.  This file is collected last on purpose.
"""
import numpy as np
import pytest

import workloads as W

pytestmark = pytest.mark.gpu


def test_static_scratch_prefill_matches_regular_entry_point():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2501_04987_b200 import _build

    _build.build()
    from paper_2501_04987_b200 import binding as tk

    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=96, chunk=64)
    ref = tk.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    alt = tk.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    stream = torch.cuda.current_stream().cuda_stream
    tol = 2e-2  # bf16 output tolerance used by the parity tests
    # three calls in a row: filling, first evictions, a ragged chunk that wraps the eviction cycle
    for call, lens in enumerate([[64, 64], [64, 50], [64, 64]]):
        q, k, v = W.tokens(w, 0, call * 64, (call + 1) * 64)
        tq, tkk, tv = (torch.from_numpy(np.ascontiguousarray(x.transpose(1, 0, 2, 3))).cuda().bfloat16() for x in (q, k, v))
        out_ref = torch.zeros_like(tq)
        out_alt = torch.zeros_like(tq)
        st = tk.treekv_prefill_chunk(ref._h, tq.data_ptr(), tkk.data_ptr(), tv.data_ptr(), out_ref.data_ptr(), lens, 64, stream)
        assert st == 0, tk.status_string(st)
        st = tk.treekv_prefill_chunk_static_scratch(alt._h, tq.data_ptr(), tkk.data_ptr(), tv.data_ptr(),
                                                    out_alt.data_ptr(), lens, 64, stream)
        assert st == 0, tk.status_string(st)
        torch.cuda.synchronize()
        assert (out_ref.float() - out_alt.float()).abs().max().item() <= tol
        assert torch.equal(ref.retained_positions()[0], alt.retained_positions()[0])
        assert torch.equal(ref.retained_positions()[1], alt.retained_positions()[1])
        s_ref, s_alt = ref.scores(), alt.scores()
        assert ((s_ref - s_alt).abs() <= 1e-3 * s_ref.abs() + 1e-12).all()
        assert [alt.tokens_seen(b) for b in range(2)] == [ref.tokens_seen(b) for b in range(2)]
    assert alt.stats()["device_error"] == 0


def test_static_scratch_rejects_oversized_calls():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2501_04987_b200 import binding as tk

    # 8 sequences x 8 KV heads, budget 4096, chunk 1024: about 90 MiB of scratch, far beyond the 16 MiB area
    kv = tk.TreeKV(4096, 32, 8, 128, "bf16", 8, 1024)
    x = torch.zeros((8, 1024, 32, 128), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((8, 1024, 8, 128), dtype=torch.bfloat16, device="cuda")
    st = tk.treekv_prefill_chunk_static_scratch(kv._h, x.data_ptr(), y.data_ptr(), y.data_ptr(), x.data_ptr(), None, 1024,
                                                torch.cuda.current_stream().cuda_stream)
    assert st == 4
    assert kv.tokens_seen(0) == 0 and kv.stats()["kernel_launches"] == 1   # nothing was enqueued
