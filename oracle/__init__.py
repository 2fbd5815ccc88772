"""TEST INFRASTRUCTURE: ctypes binding of the fp64 CPU checker in svlm_oracle.cpp.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library never does.  `build()` compiles the checker with g++ (no GPU, no CUDA involved).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "svlm_oracle.cpp")
_LIB = os.path.join(_HERE, "libsvlm_oracle.so")

TEXT, VISION = 0, 1
ROPE_1D, ROPE_MROPE = 0, 1
INF = 2 ** 40   # "infinite" window or sink size


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17", "-o", _LIB, _SRC])
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int
        lib.svlmo_create.restype = vp
        lib.svlmo_create.argtypes = [i32, i32, i32, i64, i64, i64, i32, C.c_double, vp, i32, i32]
        lib.svlmo_destroy.argtypes = [vp]
        lib.svlmo_append.argtypes = [vp, vp, vp, vp, vp, i64]
        lib.svlmo_set_kv.argtypes = [vp, i32, vp, vp, vp, i64]
        lib.svlmo_evict.argtypes = [vp]
        lib.svlmo_count.restype = i64
        lib.svlmo_count.argtypes = [vp]
        lib.svlmo_query.argtypes = [vp, vp, vp, vp, vp, vp]
        lib.svlmo_rotate.argtypes = [vp, vp, vp, vp]
        lib.svlmo_rotated_k.argtypes = [vp, i32, vp]
        lib.svlmo_values.argtypes = [vp, i32, vp]
        lib.svlmo_attend.restype = i32
        lib.svlmo_attend.argtypes = [vp, i32, vp, vp, i64, i32, vp, i64, vp]
        lib.svlmo_threads.restype = i32
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def threads() -> int:
    return int(_load().svlmo_threads())


class Oracle:
    """One stream's cache, followed on the CPU in fp64."""

    def __init__(self, layers, kv_heads, head_dim, n_sink, vision_window, text_window,
                 rope_mode=ROPE_1D, rope_base=1.0e4, sections=(0, 0, 0), sink_any_type=False, contiguous=True):
        self.lib = _load()
        self.layers, self.kv_heads, self.head_dim = layers, kv_heads, head_dim
        self.rope_mode = rope_mode
        sec = np.asarray(sections, dtype=np.int32)
        self.h = self.lib.svlmo_create(layers, kv_heads, head_dim, min(n_sink, INF), min(vision_window, INF),
                                       min(text_window, INF), rope_mode, float(rope_base), _ptr(sec),
                                       int(sink_any_type), int(contiguous))

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.svlmo_destroy(self.h)
            self.h = None

    def _pos(self, pos, n):
        pos = np.ascontiguousarray(pos, dtype=np.int32)
        want = (n,) if self.rope_mode == ROPE_1D else (n, 3)
        assert pos.shape == want, (pos.shape, want)
        return pos

    def append(self, K, V, types, pos):
        """K, V: uint16 bf16 bits [layers, n, kv_heads, head_dim] or None (metadata only)."""
        types = np.ascontiguousarray(types, dtype=np.uint8)
        n = len(types)
        pos = self._pos(pos, n)
        if K is not None:
            K = np.ascontiguousarray(K, dtype=np.uint16)
            V = np.ascontiguousarray(V, dtype=np.uint16)
            assert K.shape == (self.layers, n, self.kv_heads, self.head_dim) == V.shape
        self.lib.svlmo_append(self.h, _ptr(K), _ptr(V), _ptr(types), _ptr(pos), n)

    def set_kv(self, layer, gids, K, V):
        gids = np.ascontiguousarray(gids, dtype=np.int64)
        K = np.ascontiguousarray(K, dtype=np.uint16)
        V = np.ascontiguousarray(V, dtype=np.uint16)
        assert K.shape == (len(gids), self.kv_heads, self.head_dim) == V.shape
        self.lib.svlmo_set_kv(self.h, layer, _ptr(gids), _ptr(K), _ptr(V), len(gids))

    def evict(self):
        self.lib.svlmo_evict(self.h)

    def count(self) -> int:
        return int(self.lib.svlmo_count(self.h))

    def query(self):
        """dict(gids, pos[n,3], types, advances, n_total, n_text, n_vis, cursor, shift_total)."""
        n = self.count()
        gids = np.zeros(n, np.int64)
        pos = np.zeros((n, 3), np.int32)
        types = np.zeros(n, np.uint8)
        adv = np.zeros(n, np.int64)
        cnt = np.zeros(5, np.int64)
        self.lib.svlmo_query(self.h, _ptr(gids), _ptr(pos), _ptr(types), _ptr(adv), _ptr(cnt))
        return dict(gids=gids, pos=pos, types=types, advances=adv, n_total=int(cnt[0]), n_text=int(cnt[1]),
                    n_vis=int(cnt[2]), cursor=int(cnt[3]), shift_total=int(cnt[4]))

    def rotate(self, x, c3):
        x = np.ascontiguousarray(x, dtype=np.float64)
        c3 = np.ascontiguousarray(c3, dtype=np.int64)
        y = np.zeros_like(x)
        self.lib.svlmo_rotate(self.h, _ptr(x), _ptr(c3), _ptr(y))
        return y

    def rotated_k(self, layer):
        out = np.zeros((self.count(), self.kv_heads, self.head_dim), np.float64)
        self.lib.svlmo_rotated_k(self.h, layer, _ptr(out))
        return out

    def values(self, layer):
        out = np.zeros((self.count(), self.kv_heads, self.head_dim), np.float64)
        self.lib.svlmo_values(self.h, layer, _ptr(out))
        return out

    def attend(self, layer, Q, q_pos, rows=None):
        """Q: uint16 bf16 bits [n_q, q_heads, head_dim]; returns fp64 [n_rows, q_heads, head_dim]."""
        Q = np.ascontiguousarray(Q, dtype=np.uint16)
        n_q, q_heads, d = Q.shape
        assert d == self.head_dim and q_heads % self.kv_heads == 0
        q_pos = self._pos(q_pos, n_q)
        if rows is not None:
            rows = np.ascontiguousarray(rows, dtype=np.int64)
            n_rows = len(rows)
        else:
            n_rows = n_q
        out = np.zeros((n_rows, q_heads, d), np.float64)
        rc = self.lib.svlmo_attend(self.h, layer, _ptr(Q), _ptr(q_pos), n_q, q_heads, _ptr(rows), n_rows, _ptr(out))
        if rc != 0:
            raise RuntimeError("attend touched a stored token whose K/V were never supplied")
        return out
