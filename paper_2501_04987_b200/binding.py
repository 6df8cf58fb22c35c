"""Thin ctypes binding of libtreekv.so: argument marshalling only.

Function names match include/treekv.h.  `TreeKV` is a convenience wrapper that owns the device workspace as a
torch tensor and passes torch tensors' device pointers and the current CUDA stream; every step of the path runs
in the library's kernels.  There is no CPU fallback: if the shared library cannot be loaded the import of this
module fails.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtreekv.so")

TREEKV_OK = 0
TREEKV_F32, TREEKV_BF16 = 0, 1
RULE_SCORES, RULE_KEEP_LEFT, RULE_EVICT_LEFT, RULE_ACCUMULATED = 0, 1, 2, 3
OPT_DECODE_SPLIT, OPT_PREFILL_PATH, OPT_DECODE_PATH, OPT_PREFILL_APPEND, OPT_EVICTION_STREAM = 0, 1, 2, 3, 4
OPT_PREFILL_KEY_SPLIT = 5

# every symbol include/treekv.h declares
EXPORTS = [
    "treekv_workspace_bytes", "treekv_create", "treekv_decode_step", "treekv_prefill_chunk",
    "treekv_decode_step_host", "treekv_prefill_chunk_host", "treekv_prefill_chunk_static_scratch", "treekv_retained_positions", "treekv_scores",
    "treekv_get_stats", "treekv_tokens_seen", "treekv_set_rule", "treekv_set_option", "treekv_reset",
    "treekv_destroy", "treekv_status_string", "treekv_version",
    "treekv_state_bytes", "treekv_export_state", "treekv_import_state", "treekv_selftest_wait_giveup",
    "treekv_set_protection", "treekv_prefill_oneshot", "treekv_set_positions",
]


class TreeKVStats(C.Structure):
    _fields_ = [
        ("evictions", C.c_uint64),
        ("near_ties", C.c_uint64),
        ("kernel_launches", C.c_uint64),
        ("device_error", C.c_uint32),
        ("last_cuda_error", C.c_int32),
    ]


class TreeKVError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (what, status_string(status), status))


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libtreekv.so is missing at %s; build it with `python -m paper_2501_04987_b200._build` "
            "(there is no CPU fallback)" % LIB_PATH
        )
    lib = C.CDLL(LIB_PATH)
    vp, i32 = C.c_void_p, C.c_int
    lib.treekv_workspace_bytes.restype = C.c_size_t
    lib.treekv_workspace_bytes.argtypes = [i32] * 7
    lib.treekv_create.restype = i32
    lib.treekv_create.argtypes = [C.POINTER(vp), i32, i32, i32, i32, i32, i32, i32, vp, C.c_size_t, vp]
    lib.treekv_decode_step.restype = i32
    lib.treekv_decode_step.argtypes = [vp, vp, vp, vp, vp, C.POINTER(C.c_uint8), vp]
    lib.treekv_decode_step_host.restype = i32
    lib.treekv_decode_step_host.argtypes = [vp, vp, vp, vp, vp, C.POINTER(C.c_uint8), vp]
    lib.treekv_prefill_chunk.restype = i32
    lib.treekv_prefill_chunk.argtypes = [vp, vp, vp, vp, vp, C.POINTER(C.c_int32), i32, vp]
    lib.treekv_prefill_chunk_host.restype = i32
    lib.treekv_prefill_chunk_host.argtypes = [vp, vp, vp, vp, vp, C.POINTER(C.c_int32), i32, vp]
    lib.treekv_prefill_chunk_static_scratch.restype = i32
    lib.treekv_prefill_chunk_static_scratch.argtypes = [vp, vp, vp, vp, vp, C.POINTER(C.c_int32), i32, vp]
    lib.treekv_retained_positions.restype = i32
    lib.treekv_retained_positions.argtypes = [vp, vp, vp, vp]
    lib.treekv_scores.restype = i32
    lib.treekv_scores.argtypes = [vp, vp, vp]
    lib.treekv_get_stats.restype = i32
    lib.treekv_get_stats.argtypes = [vp, C.POINTER(TreeKVStats), vp]
    lib.treekv_tokens_seen.restype = C.c_int64
    lib.treekv_tokens_seen.argtypes = [vp, i32]
    lib.treekv_set_rule.restype = i32
    lib.treekv_set_rule.argtypes = [vp, i32]
    lib.treekv_set_option.restype = i32
    lib.treekv_set_option.argtypes = [vp, i32, i32]
    lib.treekv_reset.restype = i32
    lib.treekv_reset.argtypes = [vp, vp]
    lib.treekv_destroy.restype = None
    lib.treekv_destroy.argtypes = [vp]
    lib.treekv_status_string.restype = C.c_char_p
    lib.treekv_status_string.argtypes = [i32]
    lib.treekv_version.restype = C.c_char_p
    lib.treekv_version.argtypes = []
    lib.treekv_state_bytes.restype = C.c_size_t
    lib.treekv_state_bytes.argtypes = [vp]
    lib.treekv_export_state.restype = i32
    lib.treekv_export_state.argtypes = [vp, vp, C.POINTER(C.c_int64), vp]
    lib.treekv_import_state.restype = i32
    lib.treekv_import_state.argtypes = [vp, vp, C.POINTER(C.c_int64), vp]
    lib.treekv_prefill_oneshot.restype = i32
    lib.treekv_prefill_oneshot.argtypes = [vp, vp, vp, vp, vp, C.POINTER(C.c_int32), i32, i32, vp]
    lib.treekv_set_positions.restype = i32
    lib.treekv_set_positions.argtypes = [vp, vp, vp, i32]
    lib.treekv_set_protection.restype = i32
    lib.treekv_set_protection.argtypes = [vp, i32, i32]
    lib.treekv_selftest_wait_giveup.restype = i32
    lib.treekv_selftest_wait_giveup.argtypes = [vp, i32, vp]
    return lib


lib = _load()


def status_string(status: int) -> str:
    return lib.treekv_status_string(status).decode()


def _check(status, what):
    if status != TREEKV_OK:
        raise TreeKVError(status, what)


# ---- the C ABI, same names, raw pointers (ints) ---------------------------------------------------------
def treekv_workspace_bytes(budget, n_heads, n_kv_heads, head_dim, dtype, batch, max_chunk) -> int:
    return lib.treekv_workspace_bytes(budget, n_heads, n_kv_heads, head_dim, dtype, batch, max_chunk)


def treekv_create(budget, n_heads, n_kv_heads, head_dim, dtype, batch, max_chunk, dev_workspace, workspace_bytes, stream=0):
    h = C.c_void_p()
    st = lib.treekv_create(C.byref(h), budget, n_heads, n_kv_heads, head_dim, dtype, batch, max_chunk,
                           dev_workspace, workspace_bytes, stream)
    return st, h


def _u8(active):
    if active is None:
        return None
    arr = (C.c_uint8 * len(active))(*[1 if a else 0 for a in active])
    return arr


def _i32(lens):
    if lens is None:
        return None
    return (C.c_int32 * len(lens))(*[int(x) for x in lens])


def treekv_decode_step(ctx, q, k, v, out, active=None, stream=0) -> int:
    return lib.treekv_decode_step(ctx, q, k, v, out, _u8(active), stream)


def treekv_decode_step_host(ctx, q, k, v, out, active=None, stream=0) -> int:
    return lib.treekv_decode_step_host(ctx, q, k, v, out, _u8(active), stream)


def treekv_prefill_chunk(ctx, q, k, v, out, chunk_lens, chunk_stride, stream=0) -> int:
    return lib.treekv_prefill_chunk(ctx, q, k, v, out, _i32(chunk_lens), chunk_stride, stream)


def treekv_prefill_oneshot(ctx, q, k, v, out, lens, stride, block, stream=0) -> int:
    return lib.treekv_prefill_oneshot(ctx, q, k, v, out, _i32(lens), stride, block, stream)


def treekv_prefill_chunk_host(ctx, q, k, v, out, chunk_lens, chunk_stride, stream=0) -> int:
    return lib.treekv_prefill_chunk_host(ctx, q, k, v, out, _i32(chunk_lens), chunk_stride, stream)


def treekv_prefill_chunk_static_scratch(ctx, q, k, v, out, chunk_lens, chunk_stride, stream=0) -> int:
    """treekv_prefill_chunk with its scratch in the library's fixed 16 MiB device area: for callers that cannot
    allocate device memory where they run.  Calls sharing a GPU must not overlap."""
    return lib.treekv_prefill_chunk_static_scratch(ctx, q, k, v, out, _i32(chunk_lens), chunk_stride, stream)


def treekv_retained_positions(ctx, dev_pos, dev_count, stream=0) -> int:
    return lib.treekv_retained_positions(ctx, dev_pos, dev_count, stream)


def treekv_scores(ctx, dev_sbar, stream=0) -> int:
    return lib.treekv_scores(ctx, dev_sbar, stream)


def treekv_get_stats(ctx, stream=0):
    s = TreeKVStats()
    st = lib.treekv_get_stats(ctx, C.byref(s), stream)
    return st, s


def treekv_tokens_seen(ctx, b) -> int:
    return lib.treekv_tokens_seen(ctx, b)


def treekv_set_rule(ctx, rule) -> int:
    return lib.treekv_set_rule(ctx, rule)


def treekv_set_protection(ctx, n_sink, n_recent) -> int:
    return lib.treekv_set_protection(ctx, n_sink, n_recent)


def treekv_set_positions(ctx, dev_cos, dev_sin, slots) -> int:
    return lib.treekv_set_positions(ctx, dev_cos, dev_sin, slots)


def treekv_set_option(ctx, opt, value) -> int:
    return lib.treekv_set_option(ctx, opt, value)


def treekv_reset(ctx, stream=0) -> int:
    return lib.treekv_reset(ctx, stream)


def treekv_state_bytes(ctx) -> int:
    return lib.treekv_state_bytes(ctx)


def treekv_export_state(ctx, dev_image, batch, stream=0):
    seen = (C.c_int64 * batch)()
    st = lib.treekv_export_state(ctx, dev_image, seen, stream)
    return st, list(seen)


def treekv_import_state(ctx, dev_image, tokens_seen, stream=0) -> int:
    seen = (C.c_int64 * len(tokens_seen))(*[int(x) for x in tokens_seen])
    return lib.treekv_import_state(ctx, dev_image, seen, stream)


def treekv_selftest_wait_giveup(ctx, attempts, stream=0) -> int:
    return lib.treekv_selftest_wait_giveup(ctx, attempts, stream)


def treekv_destroy(ctx) -> None:
    lib.treekv_destroy(ctx)


def treekv_version() -> str:
    return lib.treekv_version().decode()


# ---- convenience wrapper over torch tensors --------------------------------------------------------------
class TreeKV:
    """One attention layer's TreeKV cache on the current CUDA device.  torch supplies memory and streams only."""

    def __init__(self, budget, n_heads, n_kv_heads, head_dim, dtype="bf16", batch=1, max_chunk=0, device=None):
        import torch

        self.torch = torch
        if not torch.cuda.is_available():
            raise RuntimeError("TreeKV needs a CUDA device; there is no CPU fallback")
        self.device = torch.device(device if device is not None else "cuda:%d" % torch.cuda.current_device())
        self.budget, self.n_heads, self.n_kv_heads, self.head_dim = budget, n_heads, n_kv_heads, head_dim
        self.batch, self.max_chunk = batch, max_chunk
        self.dtype_code = TREEKV_F32 if dtype in ("f32", "fp32", torch.float32) else TREEKV_BF16
        self.tdtype = torch.float32 if self.dtype_code == TREEKV_F32 else torch.bfloat16
        nbytes = treekv_workspace_bytes(budget, n_heads, n_kv_heads, head_dim, self.dtype_code, batch, max_chunk)
        if nbytes == 0:
            raise TreeKVError(4, "treekv_workspace_bytes")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        st, h = treekv_create(budget, n_heads, n_kv_heads, head_dim, self.dtype_code, batch, max_chunk, base, nbytes,
                              self._stream())
        _check(st, "treekv_create")
        self._h = h

    def _stream(self):
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def close(self):
        h, self._h = getattr(self, "_h", None), None
        if h and lib is not None and getattr(lib, "treekv_destroy", None) is not None:   # (names vanish at interpreter exit)
            lib.treekv_destroy(h)

    def __del__(self):
        self.close()

    def _chk(self, t, shape):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == self.tdtype and tuple(t.shape) == tuple(shape)):
            raise ValueError("expected contiguous %s CUDA tensor of shape %s, got %s %s" %
                             (self.tdtype, tuple(shape), t.dtype, tuple(t.shape)))

    def decode_step(self, q, k, v, out=None, active=None):
        B, Hq, Hkv, d = self.batch, self.n_heads, self.n_kv_heads, self.head_dim
        self._chk(q, (B, Hq, d)); self._chk(k, (B, Hkv, d)); self._chk(v, (B, Hkv, d))
        if out is None:
            out = self.torch.empty_like(q)
        self._chk(out, (B, Hq, d))
        _check(treekv_decode_step(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), active,
                                  self._stream()), "treekv_decode_step")
        return out

    def prefill_chunk(self, q, k, v, out=None, chunk_lens=None):
        B, Hq, Hkv, d = self.batch, self.n_heads, self.n_kv_heads, self.head_dim
        stride = q.shape[1]
        self._chk(q, (B, stride, Hq, d)); self._chk(k, (B, stride, Hkv, d)); self._chk(v, (B, stride, Hkv, d))
        if out is None:
            out = self.torch.empty_like(q)
        self._chk(out, (B, stride, Hq, d))
        _check(treekv_prefill_chunk(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), chunk_lens,
                                    stride, self._stream()), "treekv_prefill_chunk")
        return out

    def prefill_oneshot(self, q, k, v, block, out=None, lens=None):
        B, Hq, Hkv, d = self.batch, self.n_heads, self.n_kv_heads, self.head_dim
        stride = q.shape[1]
        self._chk(q, (B, stride, Hq, d)); self._chk(k, (B, stride, Hkv, d)); self._chk(v, (B, stride, Hkv, d))
        if out is None:
            out = self.torch.empty_like(q)
        self._chk(out, (B, stride, Hq, d))
        _check(treekv_prefill_oneshot(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lens, stride,
                                      block, self._stream()), "treekv_prefill_oneshot")
        return out

    def prefill_chunk_static_scratch(self, q, k, v, out=None, chunk_lens=None):
        """prefill_chunk through the entry point whose scratch is the library's fixed device area (no allocation)."""
        B, Hq, Hkv, d = self.batch, self.n_heads, self.n_kv_heads, self.head_dim
        stride = q.shape[1]
        self._chk(q, (B, stride, Hq, d)); self._chk(k, (B, stride, Hkv, d)); self._chk(v, (B, stride, Hkv, d))
        if out is None:
            out = self.torch.empty_like(q)
        self._chk(out, (B, stride, Hq, d))
        _check(treekv_prefill_chunk_static_scratch(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                                   chunk_lens, stride, self._stream()),
               "treekv_prefill_chunk_static_scratch")
        return out

    def decode_step_host(self, q, k, v, out, active=None):
        """q,k,v,out: CPU tensors (pinned for asynchronous copies)."""
        _check(treekv_decode_step_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), active,
                                       self._stream()), "treekv_decode_step_host")
        return out

    def prefill_chunk_host(self, q, k, v, out, chunk_lens=None):
        _check(treekv_prefill_chunk_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), chunk_lens,
                                         q.shape[1], self._stream()), "treekv_prefill_chunk_host")
        return out

    def retained_positions(self):
        t = self.torch
        pos = t.empty((self.batch, self.n_kv_heads, self.budget), dtype=t.int32, device=self.device)
        cnt = t.empty((self.batch, self.n_kv_heads), dtype=t.int32, device=self.device)
        _check(treekv_retained_positions(self._h, pos.data_ptr(), cnt.data_ptr(), self._stream()),
               "treekv_retained_positions")
        return pos, cnt

    def scores(self):
        t = self.torch
        sb = t.empty((self.batch, self.n_kv_heads, self.budget), dtype=t.float32, device=self.device)
        _check(treekv_scores(self._h, sb.data_ptr(), self._stream()), "treekv_scores")
        return sb

    def stats(self, check=True):
        """Counters as a dict.  With check=False a device-side give-up (TREEKV_ERR_TIMEOUT) is reported through
        'device_error' and 'status' instead of raising."""
        st, s = treekv_get_stats(self._h, self._stream())
        if check or st not in (TREEKV_OK, 6):
            _check(st, "treekv_get_stats")
        return {"status": st, "evictions": s.evictions, "near_ties": s.near_ties, "kernel_launches": s.kernel_launches,
                "device_error": s.device_error, "last_cuda_error": s.last_cuda_error}

    def tokens_seen(self, b=0):
        return treekv_tokens_seen(self._h, b)

    def set_rule(self, rule):
        _check(treekv_set_rule(self._h, rule), "treekv_set_rule")

    def set_protection(self, n_sink, n_recent):
        _check(treekv_set_protection(self._h, n_sink, n_recent), "treekv_set_protection")

    def set_positions(self, cos, sin):
        """cos, sin: float32 CUDA tensors [slots, head_dim/2] (kept alive by this object), or None, None."""
        if cos is None:
            _check(treekv_set_positions(self._h, None, None, 0), "treekv_set_positions")
            self._rope = None
            return
        t = self.torch
        if not (cos.is_cuda and cos.is_contiguous() and cos.dtype == t.float32 and sin.shape == cos.shape and sin.is_cuda
                and sin.is_contiguous() and sin.dtype == t.float32 and cos.shape[1] == self.head_dim // 2):
            raise ValueError("expected two contiguous float32 CUDA tensors of shape [slots, head_dim/2]")
        _check(treekv_set_positions(self._h, cos.data_ptr(), sin.data_ptr(), cos.shape[0]), "treekv_set_positions")
        self._rope = (cos, sin)

    def set_option(self, opt, value):
        _check(treekv_set_option(self._h, opt, value), "treekv_set_option")

    def reset(self):
        _check(treekv_reset(self._h, self._stream()), "treekv_reset")

    def export_state(self):
        """(image, tokens_seen): a uint8 CUDA tensor holding the state image and the per-sequence token counts."""
        n = treekv_state_bytes(self._h)
        image = self.torch.empty(n + 256, dtype=self.torch.uint8, device=self.device)
        off = (-image.data_ptr()) % 256
        image = image[off:off + n]
        st, seen = treekv_export_state(self._h, image.data_ptr(), self.batch, self._stream())
        _check(st, "treekv_export_state")
        return image, seen

    def import_state(self, image, tokens_seen):
        if not (image.is_cuda and image.dtype == self.torch.uint8 and image.numel() >= treekv_state_bytes(self._h)
                and image.data_ptr() % 16 == 0):
            raise ValueError("expected a uint8 CUDA tensor of at least treekv_state_bytes, 16-byte aligned")
        _check(treekv_import_state(self._h, image.data_ptr(), tokens_seen, self._stream()), "treekv_import_state")
