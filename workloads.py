"""Seeded synthetic workloads shared by the tests, the smoke check and the benchmark.

This module only makes inputs: Gaussian q/k/v from a counter-based generator,
a few key channels scaled up so attention is peaked, an optional per-sequence
key scale, rotary position embedding at the token's stream position, and
rounding to the storage dtype.  It contains none of the cache policy's
arithmetic and imports neither the CUDA package nor the oracle.

The five configurations mirror the shapes of the models the paper evaluates
(Section 5.1: Llama-2-7B, and a Llama-3 family model) with synthetic tensors in
place of PG19 / OpenWebText2 / LongBench activations, which are not available
offline.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    batch: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str            # "f32" | "bf16"
    budget: int           # cache size c
    chunk: int            # prefill chunk length m (0: decode only)
    prefill_len: int      # tokens fed through prefill_chunk per sequence (max over the batch)
    decode_steps: int
    rope_base: float
    n_outliers: int       # key channels scaled x8 (lowest-frequency rotary pairs)
    key_scale: bool       # per-sequence key scale drawn in [0.5, 2]
    ragged: bool          # prefill lengths drawn in [prefill_len/2, prefill_len]
    seed: int
    rotate: bool = True   # False: q, k are left without rotary embedding (for caches that assign positions themselves)

    @property
    def group(self) -> int:
        return self.n_heads // self.n_kv_heads


CONFIGS = {
    # 1: single layer, fp32, token-by-token decode of a 2048-token stream
    "cfg1": Workload("cfg1", 1, 1, 4, 4, 64, "f32", 256, 0, 0, 2048, 1e4, 2, False, False, 20250105),
    # 2: Llama-2-7B-shaped decode, batch 8, budget 1024, 16384 tokens per sequence
    "cfg2": Workload("cfg2", 32, 8, 32, 32, 128, "bf16", 1024, 0, 0, 16384, 1e4, 4, False, False, 20250106),
    # 3: Llama-2-7B-shaped chunked prefill, 32768 tokens in 512-token chunks to budget 2048, then 256 decode steps
    "cfg3": Workload("cfg3", 32, 1, 32, 32, 128, "bf16", 2048, 512, 32768, 256, 1e4, 4, False, False, 20250107),
    # 4: Llama-3-8B-shaped GQA decode, batch 32, budget 2048, 4096-token prefill then 8192 decode steps
    "cfg4": Workload("cfg4", 32, 32, 32, 8, 128, "bf16", 2048, 1024, 4096, 8192, 5e5, 0, True, False, 20250108),
    # 5: Llama-3-8B-shaped GQA chunked prefill, batch 4, ragged 65536..131072 tokens, chunks of 1024 to budget 4096
    "cfg5": Workload("cfg5", 32, 4, 32, 8, 128, "bf16", 4096, 1024, 131072, 1024, 5e5, 0, True, True, 20250109),
}


def parity_slice(w: Workload, **kw) -> Workload:
    """A reduced copy of a configuration (same head_dim / dtype / budget / chunk unless overridden)."""
    return replace(w, **kw)


# --------------------------------------------------------------------------------------
# dtype rounding (round-to-nearest-even to bfloat16, kept in a float32 container)
# --------------------------------------------------------------------------------------
def round_bf16(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def round_to(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.asarray(x, dtype=np.float32)
    return round_bf16(x) if dtype == "bf16" else x


# --------------------------------------------------------------------------------------
# counter-based Gaussian blocks: (seed, tensor, layer, sequence, token block) -> values
# --------------------------------------------------------------------------------------
_TOKEN_BLOCK = 256
_TENSOR_ID = {"q": 0, "k": 1, "v": 2}


def _normal_block(seed: int, tensor: str, layer: int, seq: int, blk: int, n_heads: int, d: int, rows: int = _TOKEN_BLOCK) -> np.ndarray:
    """First `rows` tokens of a 256-token block (the generator fills the block token by token, so a prefix of the
    block is the same whether or not the rest is drawn)."""
    bitgen = np.random.Philox(key=seed, counter=[blk, seq, layer, _TENSOR_ID[tensor]])
    return np.random.Generator(bitgen).standard_normal((rows, n_heads, d), dtype=np.float32)


def _normal_tokens(seed, tensor, layer, seq, t0, t1, n_heads, d):
    out = np.empty((t1 - t0, n_heads, d), np.float32)
    t = t0
    while t < t1:
        blk = t // _TOKEN_BLOCK
        lo = t - blk * _TOKEN_BLOCK
        hi = min(_TOKEN_BLOCK, t1 - blk * _TOKEN_BLOCK)
        out[t - t0 : t - t0 + hi - lo] = _normal_block(seed, tensor, layer, seq, blk, n_heads, d, hi)[lo:hi]
        t += hi - lo
    return out


def outlier_channels(d: int, n_outliers: int):
    """Channels of the lowest-frequency rotary pairs: scaling both members of a pair commutes with the rotation."""
    npairs = n_outliers // 2
    half = d // 2
    ch = []
    for p in range(npairs):
        ch += [half - 1 - p, d - 1 - p]
    return sorted(ch)


def rope(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotate-half rotary embedding: x [T, H, d], pos [T]; angle = pos * base**(-2i/d) for pair (i, i+d/2)."""
    d = x.shape[-1]
    half = d // 2
    inv_freq = base ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]
    cos = np.cos(ang)[:, None, :]
    sin = np.sin(ang)[:, None, :]
    x1 = x[..., :half].astype(np.float64)
    x2 = x[..., half:].astype(np.float64)
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1).astype(np.float32)


def rope_tables(slots: int, d: int, base: float):
    """cos, sin [slots, d/2] in single precision: the rotary cache a model hands to a library that assigns
    positions by cache slot (angle = slot * base**(-2i/d))."""
    inv_freq = base ** (-np.arange(d // 2, dtype=np.float64) * 2.0 / d)
    ang = np.arange(slots, dtype=np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def seq_key_scales(w: Workload) -> np.ndarray:
    if not w.key_scale:
        return np.ones(w.batch, np.float32)
    g = np.random.Generator(np.random.Philox(key=w.seed, counter=[0, 0, 0, 7]))
    return g.uniform(0.5, 2.0, size=w.batch).astype(np.float32)


def seq_prefill_lens(w: Workload) -> np.ndarray:
    if not w.ragged:
        return np.full(w.batch, w.prefill_len, np.int64)
    g = np.random.Generator(np.random.Philox(key=w.seed, counter=[0, 0, 0, 8]))
    return g.integers(w.prefill_len // 2, w.prefill_len + 1, size=w.batch).astype(np.int64)


def tokens_at(w: Workload, layer: int, starts, T: int):
    """q [T,B,Hq,d], k,v [T,B,Hkv,d] (float32 holding dtype-rounded values): sequence b gets its stream
    positions starts[b] .. starts[b]+T-1.

    Sequence b's token t is the same regardless of how the stream is cut into
    calls, so the oracle and the CUDA library can be fed identical bits.
    """
    q = np.empty((T, w.batch, w.n_heads, w.head_dim), np.float32)
    k = np.empty((T, w.batch, w.n_kv_heads, w.head_dim), np.float32)
    v = np.empty((T, w.batch, w.n_kv_heads, w.head_dim), np.float32)
    scales = seq_key_scales(w)
    out_ch = outlier_channels(w.head_dim, w.n_outliers)
    for b in range(w.batch):
        t0 = int(starts[b])
        t1 = t0 + T
        pos = np.arange(t0, t1)
        qb = _normal_tokens(w.seed, "q", layer, b, t0, t1, w.n_heads, w.head_dim)
        kb = _normal_tokens(w.seed, "k", layer, b, t0, t1, w.n_kv_heads, w.head_dim)
        vb = _normal_tokens(w.seed, "v", layer, b, t0, t1, w.n_kv_heads, w.head_dim)
        if out_ch:
            kb[..., out_ch] *= 8.0
        kb *= scales[b]
        q[:, b] = rope(qb, pos, w.rope_base) if w.rotate else qb
        k[:, b] = rope(kb, pos, w.rope_base) if w.rotate else kb
        v[:, b] = vb
    return round_to(q, w.dtype), round_to(k, w.dtype), round_to(v, w.dtype)


def tokens(w: Workload, layer: int, t0: int, t1: int):
    """Same as tokens_at with every sequence at stream positions t0..t1-1."""
    return tokens_at(w, layer, [t0] * w.batch, t1 - t0)


def chunk_schedule(w: Workload):
    """List of per-call chunk lengths [n_calls][B] that feeds each sequence its prefill length in chunks of w.chunk."""
    lens = seq_prefill_lens(w)
    if w.chunk <= 0 or w.prefill_len <= 0:
        return []
    n_calls = int((lens.max() + w.chunk - 1) // w.chunk)
    sched = []
    for c in range(n_calls):
        done = c * w.chunk
        sched.append(np.clip(lens - done, 0, w.chunk).astype(np.int32))
    return sched
