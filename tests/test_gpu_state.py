"""State image (export / import): the image equals the oracle's state in cache order, and a context that imports it
continues the stream bit for bit like the context that exported it."""
import numpy as np
import pytest

import workloads as W
from lockstep import Report, step_decode, step_prefill

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


def _image_parts(torch, kv, image):
    """Views of the image's parts (each starts on a 256-byte boundary)."""
    units, c, d, B = kv.batch * kv.n_kv_heads, kv.budget, kv.head_dim, kv.batch
    e = 2 if kv.tdtype == torch.bfloat16 else 4
    al = lambda x: (x + 255) // 256 * 256
    sizes = [units * c * d * e, units * c * d * e, units * c * 4, units * c * 4, B * 4]
    offs = np.concatenate([[0], np.cumsum([al(s) for s in sizes])])[:5]
    K = image[offs[0]:offs[0] + sizes[0]].view(kv.tdtype).view(kv.batch, kv.n_kv_heads, c, d)
    V = image[offs[1]:offs[1] + sizes[1]].view(kv.tdtype).view(kv.batch, kv.n_kv_heads, c, d)
    S = image[offs[2]:offs[2] + sizes[2]].view(torch.float32).view(kv.batch, kv.n_kv_heads, c)
    P = image[offs[3]:offs[3] + sizes[3]].view(torch.int32).view(kv.batch, kv.n_kv_heads, c)
    N = image[offs[4]:offs[4] + sizes[4]].view(torch.int32)
    return K, V, S, P, N


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_image_matches_oracle_and_import_continues_bitwise(gpu, dtype):
    import torch
    from oracle import Oracle

    w = W.parity_slice(W.CONFIGS["cfg4"], layers=1, batch=2, n_heads=4, n_kv_heads=2, head_dim=64 if dtype == "f32" else 128,
                       dtype=dtype, budget=96, chunk=32)
    a = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    orc = Oracle(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.batch)
    rep = Report()
    lens_total = np.array([5 * 32 + 7, 3 * 32])          # ragged: the sequences stand at different cycle positions
    for c in range(6):
        q, k, v = W.tokens(w, 0, c * 32, (c + 1) * 32)
        lens = np.clip(lens_total - c * 32, 0, 32)
        step_prefill(a, orc, q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3), w.dtype, rep, chunk_lens=lens)
    starts = [int(x) for x in lens_total]
    q, k, v = W.tokens_at(w, 0, starts, 10)
    for s in range(10):
        step_decode(a, orc, q[s], k[s], v[s], w.dtype, rep)
    seen = [x + 10 for x in starts]

    image, tokens = a.export_state()
    assert tokens == seen and image.numel() == gpu.treekv_state_bytes(a._h)
    K, V, S, P, N = _image_parts(torch, a, image)
    assert N.cpu().numpy().tolist() == seen
    for b in range(w.batch):
        for kh in range(w.n_kv_heads):
            pos = orc.positions(b, kh)
            n = len(pos)
            assert n == min(seen[b], w.budget)
            Ko, Vo = orc.kv(b, kh)
            assert np.array_equal(P[b, kh, :n].cpu().numpy(), pos) and np.all(P[b, kh, n:].cpu().numpy() == -1)
            assert np.array_equal(K[b, kh, :n].float().cpu().numpy().astype(np.float64), Ko)
            assert np.array_equal(V[b, kh, :n].float().cpu().numpy().astype(np.float64), Vo)
            sbar = S[b, kh, :n].cpu().numpy().astype(np.float64) / (seen[b] - pos)
            so = orc.scores()[b, kh, :n]
            assert np.all(np.abs(sbar - so) <= 1e-3 * np.abs(so) + 1e-12)
            assert np.all(S[b, kh, n:].cpu().numpy() == 0)

    # a fresh context and a used one (different contents, different cycle position) both take over the stream
    fresh = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    used = gpu.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, w.chunk)
    junk = [torch.randn((w.batch, h, w.head_dim), device="cuda").to(a.tdtype) for h in (w.n_heads, w.n_kv_heads, w.n_kv_heads)]
    for _ in range(w.budget + 13):
        used.decode_step(*junk)
    fresh.import_state(image, tokens)
    used.import_state(image, tokens)
    ctxs = [a, fresh, used]
    assert [[x.tokens_seen(b) for b in range(w.batch)] for x in ctxs] == [seen] * 3
    q, k, v = W.tokens_at(w, 0, seen, 150)
    to_dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda().to(a.tdtype)
    for s in range(150):
        outs = [x.decode_step(to_dev(q[s]), to_dev(k[s]), to_dev(v[s])) for x in ctxs]
        assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2]), s
    qc, kc, vc = W.tokens_at(w, 0, [x + 150 for x in seen], 32)      # and a prefill chunk after the hand-over
    chunk = [to_dev(x.transpose(1, 0, 2, 3)) for x in (qc, kc, vc)]
    outs = [x.prefill_chunk(*chunk) for x in ctxs]
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
    for x in ctxs[1:]:
        assert torch.equal(x.retained_positions()[0], a.retained_positions()[0])
        assert torch.equal(x.scores(), a.scores())
        assert x.stats()["evictions"] == a.stats()["evictions"] and x.stats()["device_error"] == 0


def test_state_image_argument_errors(gpu):
    import torch

    kv = gpu.TreeKV(16, 4, 4, 64, "f32", 2, 0)
    n = gpu.treekv_state_bytes(kv._h)
    assert n > 0 and gpu.treekv_state_bytes(None) == 0
    buf = torch.zeros(n + 64, dtype=torch.uint8, device="cuda")
    assert gpu.treekv_import_state(kv._h, buf.data_ptr() + 4, [0, 0]) == 1        # misaligned image
    assert gpu.treekv_import_state(kv._h, buf.data_ptr(), [0, -1]) == 1           # impossible token count
    assert gpu.lib.treekv_export_state(kv._h, None, None, None) == 1
    assert kv.tokens_seen(0) == 0 and kv.stats()["kernel_launches"] == 1          # nothing was enqueued
