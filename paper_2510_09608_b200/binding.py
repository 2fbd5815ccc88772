"""Thin ctypes binding of the C ABI in include/svlm.h: argument marshalling only.

Every step of the path runs in the CUDA library; there is no CPU fallback.  If libsvlm.so has not
been built (python -m paper_2510_09608_b200.build), importing this module raises.
torch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
from . import LIB_OVERRIDE as _override

LIB_PATH = _override or os.path.join(_HERE, "libsvlm.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_09608_b200.build`; "
                      "there is no fallback path")
_lib = C.CDLL(LIB_PATH)

TEXT, VISION = 0, 1
ROPE_1D, ROPE_MROPE = 0, 1
OK, ERR_ARG, ERR_CAPACITY, ERR_ORDER, ERR_CUDA, ERR_TIMEOUT, ERR_NOMEM, ERR_TOO_LARGE = 0, -1, -2, -3, -4, -5, -6, -7
NOALLOC_SCRATCH_BYTES = 512 << 10   # SVLM_NOALLOC_SCRATCH_BYTES of include/svlm.h

_vp, _i, _i64p = C.c_void_p, C.c_int, C.POINTER(C.c_int64)
_lib.svlm_cache_create.argtypes = [C.POINTER(_vp), _i, _i, _i, _i, _i, _i, _i]
_lib.svlm_cache_destroy.argtypes = [_vp]
_lib.svlm_cache_destroy.restype = None
_lib.svlm_cache_set_rope.argtypes = [_vp, _i, C.c_double, C.POINTER(C.c_int)]
_lib.svlm_cache_set_policy.argtypes = [_vp, _i, _i]
_lib.svlm_cache_set_stream.argtypes = [_vp, _vp]
_lib.svlm_cache_append.argtypes = [_vp, _i, _vp, _vp, _vp, _vp, _i]
_lib.svlm_cache_evict.argtypes = [_vp]
_lib.svlm_attend.argtypes = [_vp, _i, _vp, _vp, _i, _i, _vp]
_lib.svlm_decode_step.argtypes = [_vp, _i, _vp, _vp, _vp, _vp, _vp, _i, _vp]
_lib.svlm_attend_batched.argtypes = [C.POINTER(_vp), _i, _i, _vp, _vp, _i, _i, _vp]
_lib.svlm_attend_batched_varlen.argtypes = [C.POINTER(_vp), _i, _i, _vp, _vp, C.POINTER(C.c_int32), _i, _vp]
_lib.svlm_qkv_append.argtypes = [_vp, _i, _vp, _vp, _i, _i, _vp, _vp, _i, _vp]
_lib.svlm_out_proj.argtypes = [_vp, _vp, _vp, _i, _i, _i, _vp]
_lib.svlm_decode_step_batched.argtypes = [C.POINTER(_vp), _i, _i, _vp, _vp, _vp, _vp, _vp, _i, _vp]
_lib.svlm_cache_evict_batched.argtypes = [C.POINTER(_vp), _i]
_lib.svlm_cache_append_host.argtypes = [_vp, _i, _vp, _vp, _vp, _vp, _i]
_lib.svlm_attend_host.argtypes = [_vp, _i, _vp, _vp, _i, _i, _vp]
_lib.svlm_decode_step_host.argtypes = [_vp, _i, _vp, _vp, _vp, _vp, _vp, _i, _vp]
_lib.svlm_attend_decode_noalloc.argtypes = [_vp, _i, _vp, _vp, _i, _vp]
_lib.svlm_cache_query.argtypes = [_vp, _i64p, _vp, _vp, _vp, _i64p]
_lib.svlm_cache_read_kv.argtypes = [_vp, _i, _vp, _vp]
_lib.svlm_cache_status.argtypes = [_vp]
_lib.svlm_debug_set_wait_limit.argtypes = [_vp, C.c_uint]
_lib.svlm_launch_count.restype = C.c_int64
_lib.svlm_strerror.restype = C.c_char_p
_lib.svlm_strerror.argtypes = [_i]


class SvlmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {_lib.svlm_strerror(status).decode()} ({status})")


def _check(status: int, where: str):
    if status != OK:
        raise SvlmError(status, where)


def strerror(status: int) -> str:
    return _lib.svlm_strerror(status).decode()


def launch_count() -> int:
    return int(_lib.svlm_launch_count())


def _dev_ptr(t, dtype=None):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return t.data_ptr()


def _host_ptr(a):
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        assert not a.is_cuda and a.is_contiguous()
        return a.data_ptr()
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


class Cache:
    """KV cache of one stream (svlm_cache_*)."""

    def __init__(self, layers, kv_heads, head_dim, n_sink, vision_window, text_window, capacity):
        self.layers, self.kv_heads, self.head_dim, self.capacity = layers, kv_heads, head_dim, capacity
        self.rope_mode = ROPE_1D
        h = _vp()
        _check(_lib.svlm_cache_create(C.byref(h), layers, kv_heads, head_dim, n_sink, vision_window, text_window,
                                      capacity), "svlm_cache_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None) and _lib is not None:      # (at interpreter exit the module may already be torn down)
            _lib.svlm_cache_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def set_rope(self, mode, base, sections=(0, 0, 0)):
        sec = (C.c_int * 3)(*sections)
        _check(_lib.svlm_cache_set_rope(self._h, mode, float(base), sec), "svlm_cache_set_rope")
        self.rope_mode = mode

    def set_policy(self, sink_any_type=False, contiguous=True):
        _check(_lib.svlm_cache_set_policy(self._h, int(sink_any_type), int(contiguous)), "svlm_cache_set_policy")

    def set_stream(self, stream: "torch.cuda.Stream"):
        _check(_lib.svlm_cache_set_stream(self._h, stream.cuda_stream), "svlm_cache_set_stream")

    def append(self, layer, K, V, token_type=None, pos=None):
        """K, V: bf16 CUDA tensors [n, kv_heads, d] (layer >= 0) or [layers, n, kv_heads, d] (layer -1)."""
        n = K.shape[-3]
        rc = _lib.svlm_cache_append(self._h, layer, _dev_ptr(K, torch.bfloat16), _dev_ptr(V, torch.bfloat16),
                                    _dev_ptr(token_type, torch.uint8), _dev_ptr(pos, torch.int32), n)
        _check(rc, "svlm_cache_append")

    def qkv_append(self, layer, X, W, q_heads, token_type=None, pos=None, Q_out=None):
        """Projection with the append as its epilogue: X bf16 CUDA [n, hidden], W [(q_heads + 2 kv_heads) * d, hidden];
        stores the layer's rotated keys and values of the n tokens in the cache and returns Q [n, q_heads, d]."""
        n, hidden = X.shape
        if Q_out is None:
            Q_out = torch.empty(n, q_heads, self.head_dim, dtype=torch.bfloat16, device=X.device)
        rc = _lib.svlm_qkv_append(self._h, layer, _dev_ptr(X, torch.bfloat16), _dev_ptr(W, torch.bfloat16), hidden, q_heads,
                                  _dev_ptr(token_type, torch.uint8), _dev_ptr(pos, torch.int32), n, _dev_ptr(Q_out, torch.bfloat16))
        _check(rc, "svlm_qkv_append")
        return Q_out

    def out_proj(self, A, Wo, Y=None):
        """Y = A Wo^T on the cache's stream: A bf16 CUDA [n, in_dim], Wo [out_dim, in_dim] -> Y [n, out_dim]."""
        n, in_dim = A.shape
        if Y is None:
            Y = torch.empty(n, Wo.shape[0], dtype=torch.bfloat16, device=A.device)
        rc = _lib.svlm_out_proj(self._h, _dev_ptr(A, torch.bfloat16), _dev_ptr(Wo, torch.bfloat16), in_dim, Wo.shape[0], n,
                                _dev_ptr(Y, torch.bfloat16))
        _check(rc, "svlm_out_proj")
        return Y

    def evict(self):
        _check(_lib.svlm_cache_evict(self._h), "svlm_cache_evict")

    def attend(self, layer, Q, q_pos, out=None):
        """Q: bf16 CUDA tensor [n_q, q_heads, d] (layer >= 0) or [layers, n_q, q_heads, d] (layer -1)."""
        if out is None:
            out = torch.empty_like(Q)
        n_q, q_heads = Q.shape[-3], Q.shape[-2]
        rc = _lib.svlm_attend(self._h, layer, _dev_ptr(Q, torch.bfloat16), _dev_ptr(q_pos, torch.int32), n_q, q_heads,
                              _dev_ptr(out, torch.bfloat16))
        _check(rc, "svlm_attend")
        return out

    def decode_step(self, layer, K, V, token_type, pos, Q, out=None):
        """Append one token (K, V: bf16 CUDA [1, kv_heads, d]) and attend with its query (Q: [1, q_heads, d])."""
        if out is None:
            out = torch.empty_like(Q)
        rc = _lib.svlm_decode_step(self._h, layer, _dev_ptr(K, torch.bfloat16), _dev_ptr(V, torch.bfloat16),
                                   _dev_ptr(token_type, torch.uint8), _dev_ptr(pos, torch.int32),
                                   _dev_ptr(Q, torch.bfloat16), Q.shape[-2], _dev_ptr(out, torch.bfloat16))
        _check(rc, "svlm_decode_step")
        return out

    def attend_decode_noalloc(self, layer, Q, q_pos, out=None):
        """Decode attention (Q: bf16 CUDA [1, q_heads, d]) through the entry point that allocates nothing in
        the library: its scratch is a fixed array in the library image.  `out` should be passed by callers
        that must not allocate at all; it is created here only as a convenience when omitted."""
        if out is None:
            out = torch.empty_like(Q)
        assert Q.shape[-3] == 1
        rc = _lib.svlm_attend_decode_noalloc(self._h, layer, _dev_ptr(Q, torch.bfloat16), _dev_ptr(q_pos, torch.int32),
                                             Q.shape[-2], _dev_ptr(out, torch.bfloat16))
        _check(rc, "svlm_attend_decode_noalloc")
        return out

    def append_host(self, layer, K, V, token_type=None, pos=None):
        """Same as append with HOST buffers (numpy uint16 bf16 bits / pinned torch tensors)."""
        n = K.shape[-3]
        rc = _lib.svlm_cache_append_host(self._h, layer, _host_ptr(K), _host_ptr(V), _host_ptr(token_type),
                                         _host_ptr(pos), n)
        _check(rc, "svlm_cache_append_host")

    def attend_host(self, layer, Q, q_pos, out):
        n_q, q_heads = Q.shape[-3], Q.shape[-2]
        rc = _lib.svlm_attend_host(self._h, layer, _host_ptr(Q), _host_ptr(q_pos), n_q, q_heads, _host_ptr(out))
        _check(rc, "svlm_attend_host")
        return out

    def decode_step_host(self, layer, K, V, token_type, pos, Q, out):
        """decode_step with HOST buffers: K, V [layers, 1, kv_heads, d] (layer -1) or [1, kv_heads, d]; fills `out`."""
        rc = _lib.svlm_decode_step_host(self._h, layer, _host_ptr(K), _host_ptr(V), _host_ptr(token_type), _host_ptr(pos),
                                        _host_ptr(Q), Q.shape[-2], _host_ptr(out))
        _check(rc, "svlm_decode_step_host")
        return out

    def query(self):
        """dict(gids int64[n], pos int32[n,3], types uint8[n], shift_total); synchronises."""
        gids = np.zeros(self.capacity, np.int64)
        pos = np.zeros((self.capacity, 3), np.int32)
        types = np.zeros(self.capacity, np.uint8)
        n, shift = C.c_int64(0), C.c_int64(0)
        _check(_lib.svlm_cache_query(self._h, C.byref(n), gids.ctypes.data, pos.ctypes.data, types.ctypes.data,
                                     C.byref(shift)), "svlm_cache_query")
        k = n.value
        return dict(gids=gids[:k].copy(), pos=pos[:k].copy(), types=types[:k].copy(), shift_total=shift.value)

    def read_kv(self, layer, n_kept):
        """Stored (rotated) keys and values of one layer as uint16 bf16 bits [n_kept, kv_heads, d]."""
        K = np.zeros((n_kept, self.kv_heads, self.head_dim), np.uint16)
        V = np.zeros_like(K)
        _check(_lib.svlm_cache_read_kv(self._h, layer, K.ctypes.data, V.ctypes.data), "svlm_cache_read_kv")
        return K, V

    def status(self) -> int:
        return int(_lib.svlm_cache_status(self._h))

    def debug_set_wait_limit(self, polls: int):
        _check(_lib.svlm_debug_set_wait_limit(self._h, int(polls)), "svlm_debug_set_wait_limit")


def attend_batched(caches, layer, Q, q_pos, out=None):
    """Q: [n_caches, n_q, q_heads, d] bf16 CUDA; one launch for all caches (svlm_attend_batched)."""
    if out is None:
        out = torch.empty_like(Q)
    arr = (_vp * len(caches))(*[c._h for c in caches])
    rc = _lib.svlm_attend_batched(arr, len(caches), layer, _dev_ptr(Q, torch.bfloat16), _dev_ptr(q_pos, torch.int32),
                                  Q.shape[1], Q.shape[2], _dev_ptr(out, torch.bfloat16))
    _check(rc, "svlm_attend_batched")
    return out


def attend_batched_varlen(caches, layer, Q, q_pos, n_q, out=None):
    """Chunk prefill of several caches whose chunks differ in length, one launch: Q [sum(n_q), q_heads, d] bf16 CUDA with
    the caches' rows one after another, q_pos likewise, n_q a sequence of ints (svlm_attend_batched_varlen)."""
    if out is None:
        out = torch.empty_like(Q)
    arr = (_vp * len(caches))(*[c._h for c in caches])
    cnt = (C.c_int32 * len(caches))(*[int(x) for x in n_q])
    rc = _lib.svlm_attend_batched_varlen(arr, len(caches), layer, _dev_ptr(Q, torch.bfloat16), _dev_ptr(q_pos, torch.int32), cnt,
                                         Q.shape[1], _dev_ptr(out, torch.bfloat16))
    _check(rc, "svlm_attend_batched_varlen")
    return out


def decode_step_batched(caches, layer, K, V, token_type, pos, Q, out=None):
    """One generated token per cache: K, V [n_caches, kv_heads, d], Q [n_caches, q_heads, d] bf16 CUDA, token_type
    uint8 [n_caches], pos int32 [n_caches] or [n_caches, 3]; one launch for all caches (svlm_decode_step_batched)."""
    if out is None:
        out = torch.empty_like(Q)
    arr = (_vp * len(caches))(*[c._h for c in caches])
    rc = _lib.svlm_decode_step_batched(arr, len(caches), layer, _dev_ptr(K, torch.bfloat16), _dev_ptr(V, torch.bfloat16),
                                       _dev_ptr(token_type, torch.uint8), _dev_ptr(pos, torch.int32),
                                       _dev_ptr(Q, torch.bfloat16), Q.shape[-2], _dev_ptr(out, torch.bfloat16))
    _check(rc, "svlm_decode_step_batched")
    return out


def evict_batched(caches):
    arr = (_vp * len(caches))(*[c._h for c in caches])
    _check(_lib.svlm_cache_evict_batched(arr, len(caches)), "svlm_cache_evict_batched")
