"""GPU parity with protected tokens (Section 5.2: initial "sink" tokens and a recent window are never evicted; Algorithm 1
runs on the slots between them): the CUDA library through its C ABI against the fp64 oracle in lock-step, with the
same bars as the unprotected path.  Every kernel that knows the cache geometry is exercised: both decode kernels at
every cluster size (including the step that ends a cycle, where the recent window is moved next to the middle
region), the CUDA-core and both tensor-core prefill kernels, chunks that wrap the cycle, the static-scratch entry
point, the state image, and the paper's own split 4 + 508 + 512.
"""
import numpy as np
import pytest

import workloads as W
from lockstep import Report, run_decode, run_prefill

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


def _pair(binding, w, ns, nr, max_chunk=None):
    from oracle import Oracle

    mc = w.chunk if max_chunk is None else max_chunk
    kv = binding.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, mc)
    kv.set_protection(ns, nr)
    orc = Oracle(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.batch, n_sink=ns, n_recent=nr)
    return kv, orc


def _check_protected(kv, ns, nr, seen):
    pos, cnt = kv.retained_positions()
    pos = pos.cpu().numpy(); cnt = cnt.cpu().numpy()
    for b, n in enumerate(seen):
        if n > kv.budget:
            assert np.all(pos[b, :, :ns] == np.arange(ns)) and np.all(pos[b, :, kv.budget - nr:] == np.arange(n - nr, n))


@pytest.mark.parametrize("dtype,split", [("f32", 0), ("bf16", 1), ("bf16", 2), ("bf16", 4), ("bf16", 8), ("f32", 2)])
@pytest.mark.parametrize("c,ns,nr", [(48, 4, 12), (40, 2, 30), (33, 0, 7), (33, 5, 0)])
def test_decode_with_protection(gpu, dtype, split, c, ns, nr):
    """Token-by-token decode through several cycles of the middle region (c - ns - nr evictions each), including
    windows longer than the middle region, where the rows moved at the end of a cycle overlap their destination."""
    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=c, chunk=0, dtype=dtype,
                       head_dim=128 if dtype == "bf16" else 64)
    kv, orc = _pair(gpu, w, ns, nr)
    if split:
        kv.set_option(gpu.OPT_DECODE_SPLIT, split)
    rep = Report()
    steps = c + 3 * (c - ns - nr) + 5
    run_decode(kv, orc, w, 0, steps, rep)
    _check_protected(kv, ns, nr, [steps] * 2)
    st = kv.stats()
    assert st["device_error"] == 0 and st["evictions"] == 2 * (steps - c)


@pytest.mark.parametrize("path", [1, 2, 3])
@pytest.mark.parametrize("c,ns,nr,chunk,lens", [
    (256, 4, 124, 128, [5 * 128 + 77, 3 * 128]),      # chunk = middle region: every steady chunk ends a cycle
    (384, 4, 60, 256, [4 * 256 + 100, 2 * 256 + 1]),  # chunks that wrap the cycle in the middle
    (200, 8, 150, 128, [700, 650]),                   # window longer than the middle region (42 slots): many wraps per chunk
])
def test_chunked_prefill_with_protection(gpu, path, c, ns, nr, chunk, lens):
    w = W.parity_slice(W.CONFIGS["cfg5"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=c, chunk=chunk)
    kv, orc = _pair(gpu, w, ns, nr)
    kv.set_option(gpu.OPT_PREFILL_PATH, path)
    rep = Report()
    run_prefill(kv, orc, w, rep, lens, chunk)
    assert [kv.tokens_seen(b) for b in range(2)] == lens
    _check_protected(kv, ns, nr, lens)
    run_decode(kv, orc, w, 0, c - ns - nr + 9, rep, starts=lens)     # decode on through a full cycle
    assert kv.stats()["device_error"] == 0


def test_fp32_prefill_and_static_scratch_with_protection(gpu):
    w = W.parity_slice(W.CONFIGS["cfg1"], batch=2, budget=40, chunk=24)
    kv, orc = _pair(gpu, w, 3, 11)
    rep = Report()
    run_prefill(kv, orc, w, rep, [150, 131], 24)
    run_decode(kv, orc, w, 0, 40, rep, starts=[150, 131])
    # the static-scratch entry point stages the rows it moves at a wrap, which includes the whole recent window
    w2 = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=8, n_kv_heads=2, budget=80, chunk=48)
    kv2, orc2 = _pair(gpu, w2, 4, 40)
    run_prefill(kv2, orc2, w2, rep, [6 * 48, 5 * 48 + 7], 48, method="prefill_chunk_static_scratch")
    assert kv.stats()["device_error"] == 0 and kv2.stats()["device_error"] == 0


def test_the_papers_split_4_508_512(gpu):
    """Section 5.2's cache of 1024 = 4 initial + 508 recent + 512 selected tokens, Llama-2-7B head shape (bf16, d = 128):
    a 1024-token chunked prefill, then decode through more than one cycle of the 512 selected slots."""
    w = W.parity_slice(W.CONFIGS["cfg2"], layers=1, batch=1, n_heads=2, n_kv_heads=2, budget=1024, chunk=256)
    kv, orc = _pair(gpu, w, 4, 508)
    rep = Report()
    run_prefill(kv, orc, w, rep, [1024 + 256], 256)
    run_decode(kv, orc, w, 0, 560, rep, starts=[1280], score_every=16)
    _check_protected(kv, 4, 508, [1280 + 560])
    pos = kv.retained_positions()[0].cpu().numpy()[0]
    assert np.all(np.diff(pos[:, 4:516], axis=1) > 0) and pos[:, 4:516].max() < 1280 + 560 - 508
    assert kv.stats()["device_error"] == 0
    print("4/508/512", rep)


def test_state_image_and_argument_checks_with_protection(gpu):
    import torch

    w = W.parity_slice(W.CONFIGS["cfg1"], batch=1, budget=24, chunk=0)
    kv, orc = _pair(gpu, w, 2, 9)
    rep = Report()
    run_decode(kv, orc, w, 0, 61, rep)
    image, seen = kv.export_state()
    twin = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, 0)
    twin.set_protection(2, 9)
    twin.import_state(image, seen)
    q, k, v = W.tokens_at(w, 0, [61], 30)
    for s in range(30):
        a = kv.decode_step(*(torch.from_numpy(x[s]).cuda() for x in (q, k, v)))
        b = twin.decode_step(*(torch.from_numpy(x[s]).cuda() for x in (q, k, v)))
        assert torch.equal(a, b)
    assert torch.equal(kv.retained_positions()[0], twin.retained_positions()[0]) and torch.equal(kv.scores(), twin.scores())
    # protection can only be set on an empty context and must leave room for a scope
    assert gpu.treekv_set_protection(kv._h, 1, 1) == 2
    fresh = gpu.TreeKV(8, 1, 1, 64, "f32", 1, 0)
    assert gpu.treekv_set_protection(fresh._h, 4, 3) == 1 and gpu.treekv_set_protection(fresh._h, -1, 0) == 1
    assert gpu.treekv_set_protection(fresh._h, 3, 3) == 0
    kv.reset()
    assert gpu.treekv_set_protection(kv._h, 0, 0) == 0
