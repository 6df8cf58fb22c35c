"""GPU parity of the one-shot, block-level prefill (Section 4.2) against the fp64 oracle, in lock-step: outputs of the
whole prompt, retained positions (whole blocks) exactly up to counted near-ties, averaged scores (window sums over
window counts) within 1e-3 - then decode steps and chunks that carry on from the compressed cache, which exercises
the counters that started at the observation window.  All three attention kernels, block sizes from 1 to 64,
prompts that fit, prompts that wrap the block cycle several times, ragged batches.
"""
import numpy as np
import pytest

import workloads as W
from lockstep import Report, run_decode, step_oneshot, step_prefill

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


def _pair(binding, w, max_chunk):
    from oracle import Oracle

    kv = binding.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, max_chunk)
    orc = Oracle(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.batch)
    return kv, orc


def _prompt(w, T):
    q, k, v = W.tokens(w, 0, 0, T)
    return q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3)


@pytest.mark.parametrize("path", [1, 2, 3])
@pytest.mark.parametrize("c,block,lens,g", [
    (256, 32, [1024, 768], 4),      # four / three budgets: the block pointer wraps, rows are re-based
    (128, 64, [640, 128], 1),       # two cache blocks; one prompt that just fits
    (192, 16, [400, 1008], 2),      # ragged, lengths not multiples of the query tile
    (64, 1, [300, 64], 4),          # blocks of one token: token-level eviction with the last query's weights
])
def test_oneshot_prefill_then_decode_and_chunks(gpu, path, c, block, lens, g):
    T = max(lens)
    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=2 * g, n_kv_heads=2, budget=c, chunk=T)
    kv, orc = _pair(gpu, w, T)
    kv.set_option(gpu.OPT_PREFILL_PATH, path)
    rep = Report()
    q, k, v = _prompt(w, T)
    step_oneshot(kv, orc, q, k, v, block, w.dtype, rep, lens=lens)
    assert [kv.tokens_seen(b) for b in range(2)] == lens
    pos, cnt = kv.retained_positions()
    pos = pos.cpu().numpy()
    for b in range(2):
        n = min(lens[b], c)
        p = pos[b, :, :n]
        assert np.all(p[:, ::block] % block == 0) and np.all(np.diff(p.reshape(2, -1, block), axis=2) == 1)   # whole blocks
    # carry on: decode through more than a cycle, then a chunk
    run_decode(kv, orc, w, 0, c + 7, rep, starts=lens)
    seen = [x + c + 7 for x in lens]
    qc, kc, vc = W.tokens_at(w, 0, seen, 48)
    step_prefill(kv, orc, qc.transpose(1, 0, 2, 3), kc.transpose(1, 0, 2, 3), vc.transpose(1, 0, 2, 3), w.dtype, rep)
    st = kv.stats()
    assert st["device_error"] == 0 and st["evictions"] == sum(max(0, x + c + 7 + 48 - c) for x in lens)


def test_oneshot_prefill_fp32(gpu):
    w = W.parity_slice(W.CONFIGS["cfg1"], batch=3, budget=48, chunk=200)
    kv, orc = _pair(gpu, w, 200)
    rep = Report()
    q, k, v = _prompt(w, 200)
    step_oneshot(kv, orc, q, k, v, 8, w.dtype, rep, lens=[200, 0, 40])
    run_decode(kv, orc, w, 0, 60, rep, starts=[200, 0, 40])
    assert kv.stats()["device_error"] == 0


def test_oneshot_state_image_and_argument_checks(gpu):
    import torch

    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=1, n_heads=4, n_kv_heads=2, budget=64, chunk=256)
    kv, orc = _pair(gpu, w, 256)
    rep = Report()
    q, k, v = _prompt(w, 256)
    step_oneshot(kv, orc, q, k, v, 16, w.dtype, rep)
    image, seen = kv.export_state()
    twin = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, 256)
    twin.import_state(image, seen)
    assert torch.equal(kv.scores(), twin.scores())           # the scoring start travels with the image
    qd, kd, vd = W.tokens_at(w, 0, [256], 20)
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda().to(kv.tdtype)
    for s in range(20):
        assert torch.equal(kv.decode_step(dev(qd[s]), dev(kd[s]), dev(vd[s])), twin.decode_step(dev(qd[s]), dev(kd[s]), dev(vd[s])))
    assert torch.equal(kv.retained_positions()[0], twin.retained_positions()[0]) and torch.equal(kv.scores(), twin.scores())
    # argument and state errors: nothing is enqueued
    x = torch.zeros((1, 256, 4, 128), dtype=torch.bfloat16, device="cuda"); y = torch.zeros((1, 256, 2, 128), dtype=torch.bfloat16, device="cuda")
    args = (x.data_ptr(), y.data_ptr(), y.data_ptr(), x.data_ptr())
    assert gpu.treekv_prefill_oneshot(kv._h, *args, None, 256, 16) == 2        # the cache is not empty
    fresh = gpu.TreeKV(64, 4, 2, 128, "bf16", 1, 256)
    assert gpu.treekv_prefill_oneshot(fresh._h, *args, [250], 256, 16) == 1    # not a multiple of the block
    assert gpu.treekv_prefill_oneshot(fresh._h, *args, None, 256, 24) == 1     # the budget is not a multiple of the block
    fresh.set_protection(4, 8)
    assert gpu.treekv_prefill_oneshot(fresh._h, *args, None, 256, 16) == 4     # protected tokens: not defined
    assert fresh.tokens_seen(0) == 0 and fresh.stats()["kernel_launches"] == 1
