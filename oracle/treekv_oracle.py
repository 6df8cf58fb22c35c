"""ctypes face of the C oracle (test infrastructure, see treekv_oracle.c).

`build_oracle()` compiles treekv_oracle.c with gcc into a shared library next
to the source; `Oracle` wraps one cache policy instance.  All arrays are
float64 numpy arrays; inputs are expected to be already rounded to the dtype
under test (bf16 or fp32) and widened.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "treekv_oracle.c")
_LIB = os.path.join(_HERE, "libtreekv_oracle.so")

RULE_SCORES, RULE_KEEP_LEFT, RULE_EVICT_LEFT, RULE_ACCUMULATED = 0, 1, 2, 3
IDX_CYCLE, IDX_LITERAL = 0, 1

_lib = None


def build_oracle(force: bool = False) -> str:
    """Compile the C oracle if the library is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = C.CDLL(build_oracle())
    dp = C.POINTER(C.c_double)
    vp = C.c_void_p
    lib.tkvo_create.restype = vp
    lib.tkvo_create.argtypes = [C.c_int] * 5
    lib.tkvo_destroy.argtypes = [vp]
    lib.tkvo_set_rule.argtypes = [vp, C.c_int]
    lib.tkvo_set_idx_mode.argtypes = [vp, C.c_int]
    lib.tkvo_set_protection.argtypes = [vp, C.c_int, C.c_int]
    lib.tkvo_set_protection.restype = C.c_int
    for name in ("tkvo_decode_attend", "tkvo_decode_step"):
        getattr(lib, name).argtypes = [vp, dp, dp, dp, dp, C.POINTER(C.c_uint8)]
        getattr(lib, name).restype = None
    for name in ("tkvo_prefill_attend", "tkvo_prefill_chunk"):
        getattr(lib, name).argtypes = [vp, dp, dp, dp, dp, C.POINTER(C.c_int32), C.c_int]
        getattr(lib, name).restype = None
    lib.tkvo_evict.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_double]
    lib.tkvo_evict.restype = None
    lib.tkvo_evict_blocks.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_double]
    lib.tkvo_evict_blocks.restype = None
    lib.tkvo_prefill_oneshot_attend.argtypes = [vp, dp, dp, dp, dp, C.POINTER(C.c_int32), C.c_int, C.c_int]
    lib.tkvo_prefill_oneshot_attend.restype = C.c_int
    lib.tkvo_set_rope.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_int, C.c_int]
    lib.tkvo_set_rope.restype = C.c_int
    lib.tkvo_len.argtypes = [vp, C.c_int, C.c_int]
    lib.tkvo_len.restype = C.c_int
    for name in ("tkvo_n_seen", "tkvo_n_evicted"):
        getattr(lib, name).argtypes = [vp, C.c_int]
        getattr(lib, name).restype = C.c_int64
    lib.tkvo_idx.argtypes = [vp, C.c_int]
    lib.tkvo_idx.restype = C.c_int
    for name in ("tkvo_last_near_ties", "tkvo_last_hint_flips", "tkvo_total_near_ties", "tkvo_total_hint_flips"):
        getattr(lib, name).argtypes = [vp]
        getattr(lib, name).restype = C.c_int64
    lib.tkvo_last_min_gap.argtypes = [vp]
    lib.tkvo_last_min_gap.restype = C.c_double
    lib.tkvo_read_unit.argtypes = [vp, C.c_int, C.c_int, C.POINTER(C.c_int64), dp, C.POINTER(C.c_int64), dp]
    lib.tkvo_read_unit.restype = C.c_int
    lib.tkvo_read_kv.argtypes = [vp, C.c_int, C.c_int, dp, dp]
    lib.tkvo_read_kv.restype = C.c_int
    _lib = lib
    return lib


def _f64(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float64)
    if a.shape != tuple(shape):
        raise ValueError("expected shape %s, got %s" % (tuple(shape), a.shape))
    return a


def _dp(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


class Oracle:
    """One TreeKV cache policy (one attention layer) for `batch` sequences."""

    def __init__(self, budget, n_heads, n_kv_heads, head_dim, batch=1, rule=RULE_SCORES, idx_mode=IDX_CYCLE,
                 n_sink=0, n_recent=0):
        self._lib = _load()
        self._h = self._lib.tkvo_create(budget, n_heads, n_kv_heads, head_dim, batch)
        if not self._h:
            raise ValueError("bad oracle configuration")
        self.c, self.Hq, self.Hkv, self.d, self.B = budget, n_heads, n_kv_heads, head_dim, batch
        self._lib.tkvo_set_rule(self._h, rule)
        self._lib.tkvo_set_idx_mode(self._h, idx_mode)
        self.n_sink, self.n_recent = n_sink, n_recent
        if (n_sink or n_recent) and self._lib.tkvo_set_protection(self._h, n_sink, n_recent) != 0:
            raise ValueError("bad protection: the region between sinks and recent tokens needs at least 2 slots")

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            self._lib.tkvo_destroy(h)

    # ---- Algorithm 1, split in its two halves so a test can keep two implementations in lock-step
    def decode_attend(self, q, k, v, active=None):
        q = _f64(q, (self.B, self.Hq, self.d))
        k = _f64(k, (self.B, self.Hkv, self.d))
        v = _f64(v, (self.B, self.Hkv, self.d))
        out = np.zeros_like(q)
        act = None
        if active is not None:
            a = np.ascontiguousarray(active, dtype=np.uint8)
            act = a.ctypes.data_as(C.POINTER(C.c_uint8))
        self._lib.tkvo_decode_attend(self._h, _dp(q), _dp(k), _dp(v), _dp(out), act)
        return out

    def prefill_attend(self, q, k, v, chunk_lens=None):
        q = np.ascontiguousarray(q, dtype=np.float64)
        stride = q.shape[1]
        q = _f64(q, (self.B, stride, self.Hq, self.d))
        k = _f64(k, (self.B, stride, self.Hkv, self.d))
        v = _f64(v, (self.B, stride, self.Hkv, self.d))
        if chunk_lens is None:
            chunk_lens = [stride] * self.B
        cl = np.ascontiguousarray(chunk_lens, dtype=np.int32)
        assert cl.shape == (self.B,) and cl.max() <= stride and cl.min() >= 0
        out = np.zeros_like(q)
        self._lib.tkvo_prefill_attend(self._h, _dp(q), _dp(k), _dp(v), _dp(out),
                                      cl.ctypes.data_as(C.POINTER(C.c_int32)), stride)
        return out

    def evict(self, hint_pos=None, hint_cnt=None, near_tie_tol=1e-4):
        hp = hc = None
        if hint_pos is not None:
            hint_pos = np.ascontiguousarray(hint_pos, dtype=np.int32)
            hint_cnt = np.ascontiguousarray(hint_cnt, dtype=np.int32)
            assert hint_pos.shape == (self.B, self.Hkv, self.c) and hint_cnt.shape == (self.B, self.Hkv)
            hp = hint_pos.ctypes.data_as(C.POINTER(C.c_int32))
            hc = hint_cnt.ctypes.data_as(C.POINTER(C.c_int32))
        self._lib.tkvo_evict(self._h, hp, hc, float(near_tie_tol))
        return self.last_near_ties, self.last_hint_flips

    def _hints(self, hint_pos, hint_cnt):
        hp = hc = None
        if hint_pos is not None:
            hint_pos = np.ascontiguousarray(hint_pos, dtype=np.int32)
            hint_cnt = np.ascontiguousarray(hint_cnt, dtype=np.int32)
            assert hint_pos.shape == (self.B, self.Hkv, self.c) and hint_cnt.shape == (self.B, self.Hkv)
            hp = hint_pos.ctypes.data_as(C.POINTER(C.c_int32))
            hc = hint_cnt.ctypes.data_as(C.POINTER(C.c_int32))
        return hp, hc, hint_pos, hint_cnt

    # ---- Section 4.2: one-shot, block-level prefill of an empty cache
    def prefill_oneshot_attend(self, q, k, v, block, lens=None):
        q = np.ascontiguousarray(q, dtype=np.float64)
        stride = q.shape[1]
        q = _f64(q, (self.B, stride, self.Hq, self.d))
        k = _f64(k, (self.B, stride, self.Hkv, self.d))
        v = _f64(v, (self.B, stride, self.Hkv, self.d))
        if lens is None:
            lens = [stride] * self.B
        cl = np.ascontiguousarray(lens, dtype=np.int32)
        out = np.zeros_like(q)
        rc = self._lib.tkvo_prefill_oneshot_attend(self._h, _dp(q), _dp(k), _dp(v), _dp(out),
                                                   cl.ctypes.data_as(C.POINTER(C.c_int32)), stride, int(block))
        if rc != 0:
            raise ValueError("one-shot prefill needs an empty, unprotected cache and lengths / budget that are multiples of the block")
        return out

    def evict_blocks(self, hint_pos=None, hint_cnt=None, near_tie_tol=1e-4):
        hp, hc, _a, _b = self._hints(hint_pos, hint_cnt)
        self._lib.tkvo_evict_blocks(self._h, hp, hc, float(near_tie_tol))
        return self.last_near_ties, self.last_hint_flips

    def prefill_oneshot(self, q, k, v, block, lens=None):
        out = self.prefill_oneshot_attend(q, k, v, block, lens)
        self.evict_blocks()
        return out

    # ---- Section 4.1 "Position Encoding": in-cache positions
    def set_rope(self, cos, sin, round_bf16):
        """cos, sin: float32 [slots, d/2] tables by cache slot (kept alive by this object); None switches it off."""
        if cos is None:
            self._rope = None
            self._lib.tkvo_set_rope(self._h, None, None, 0, 0)
            return
        cos = np.ascontiguousarray(cos, dtype=np.float32); sin = np.ascontiguousarray(sin, dtype=np.float32)
        assert cos.shape == sin.shape and cos.shape[1] == self.d // 2
        self._rope = (cos, sin)
        fp = C.POINTER(C.c_float)
        assert self._lib.tkvo_set_rope(self._h, cos.ctypes.data_as(fp), sin.ctypes.data_as(fp), cos.shape[0],
                                       1 if round_bf16 else 0) == 0

    def decode_step(self, q, k, v, active=None):
        out = self.decode_attend(q, k, v, active)
        self.evict()
        return out

    def prefill_chunk(self, q, k, v, chunk_lens=None):
        out = self.prefill_attend(q, k, v, chunk_lens)
        self.evict()
        return out

    # ---- read-outs
    def length(self, b=0, kh=0):
        return self._lib.tkvo_len(self._h, b, kh)

    def n_seen(self, b=0):
        return self._lib.tkvo_n_seen(self._h, b)

    def n_evicted(self, b=0):
        return self._lib.tkvo_n_evicted(self._h, b)

    def idx(self, b=0):
        return self._lib.tkvo_idx(self._h, b)

    @property
    def last_near_ties(self):
        return self._lib.tkvo_last_near_ties(self._h)

    @property
    def last_hint_flips(self):
        return self._lib.tkvo_last_hint_flips(self._h)

    @property
    def last_min_gap(self):
        return self._lib.tkvo_last_min_gap(self._h)

    @property
    def total_near_ties(self):
        return self._lib.tkvo_total_near_ties(self._h)

    @property
    def total_hint_flips(self):
        return self._lib.tkvo_total_hint_flips(self._h)

    def unit(self, b=0, kh=0):
        """(pos, S, C, S/C) of one unit in cache order."""
        n = self.length(b, kh)
        pos = np.zeros(n, np.int64); S = np.zeros(n); Cc = np.zeros(n, np.int64); sb = np.zeros(n)
        self._lib.tkvo_read_unit(self._h, b, kh, pos.ctypes.data_as(C.POINTER(C.c_int64)), _dp(S),
                                 Cc.ctypes.data_as(C.POINTER(C.c_int64)), _dp(sb))
        return pos, S, Cc, sb

    def positions(self, b=0, kh=0):
        return self.unit(b, kh)[0]

    def kv(self, b=0, kh=0):
        n = self.length(b, kh)
        K = np.zeros((n, self.d)); V = np.zeros((n, self.d))
        self._lib.tkvo_read_kv(self._h, b, kh, _dp(K), _dp(V))
        return K, V

    def retained_positions(self):
        """[B, Hkv, c] int32 positions (padded with -1) and [B, Hkv] counts."""
        pos = np.full((self.B, self.Hkv, self.c), -1, np.int32)
        cnt = np.zeros((self.B, self.Hkv), np.int32)
        for b in range(self.B):
            for kh in range(self.Hkv):
                p = self.positions(b, kh)
                pos[b, kh, : len(p)] = p
                cnt[b, kh] = len(p)
        return pos, cnt

    def scores(self):
        """[B, Hkv, c] averaged attention weight S/C of every retained slot (0 padding)."""
        sb = np.zeros((self.B, self.Hkv, self.c))
        for b in range(self.B):
            for kh in range(self.Hkv):
                s = self.unit(b, kh)[3]
                sb[b, kh, : len(s)] = s
        return sb
