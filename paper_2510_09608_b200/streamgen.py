"""Seeded synthetic streams: the inputs that both the CUDA path and the CPU checker are fed.

This module holds *inputs only*: which tokens arrive in which chunk (type, native position) and the
bf16 bit patterns of their Q/K/V rows.  It contains none of the method's arithmetic (no eviction,
no re-indexing, no rotation, no attention) and imports neither the CUDA binding nor the checker.

Value recipe (integer-only, so every row is regenerable on demand from its coordinates):

    row_key = mix(mix(mix(seed ^ tensor<<56) + (stream<<32 | layer)) + gid)
    elem    = mix(row_key + head*head_dim + dim) >> 48           # 16-bit index
    value   = NORMAL_TABLE[elem]                                   # bf16 bits of Phi^-1((k+.5)/65536)

`mix` is the splitmix64 output function.  Q/K/V are therefore i.i.d. N(0,1) quantised to bf16, the
distribution the workload table asks for, and stand in for the activations of a real decoder layer.

Stream shape: every chunk is one second of video: `frames x grid_h x grid_w` vision tokens followed
by a seeded-uniform number of text tokens, interleaved vision-then-text per second as in the paper's
Section 2.2 layout (a second may carry no text).  Native positions are what a caller of the library
would supply: a running index in 1D mode; in 3D mode a vision block starting at `base` gets
(t,h,w) = (base+frame, base+row, base+col) and advances `base` by max(frames, grid_h, grid_w), a
text token gets (base, base, base) and advances `base` by one (the Qwen-VL family's assignment).
"""
from __future__ import annotations

import dataclasses
from typing import Iterator, Optional

import numpy as np

TEXT = 0
VISION = 1

TENSOR_Q = 1
TENSOR_K = 2
TENSOR_V = 3

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)


def mix64(x):
    """splitmix64 output function on uint64 scalars or arrays (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        z = (np.asarray(x, dtype=np.uint64) + _GOLDEN)
        z = (z ^ (z >> np.uint64(30))) * _C1
        z = (z ^ (z >> np.uint64(27))) * _C2
        return z ^ (z >> np.uint64(31))


def _f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit pattern (uint16)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
    return (rounded >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


_TABLE: Optional[np.ndarray] = None


def normal_table() -> np.ndarray:
    """65,536 bf16 bit patterns: entry k is Phi^-1((k+0.5)/65536) rounded to bf16."""
    global _TABLE
    if _TABLE is None:
        from scipy.special import ndtri

        k = np.arange(65536, dtype=np.float64)
        _TABLE = _f32_to_bf16_bits(ndtri((k + 0.5) / 65536.0).astype(np.float32))
    return _TABLE


def row_keys(seed: int, tensor: int, stream: int, layer: int, gids: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        k0 = mix64(np.uint64(seed) ^ (np.uint64(tensor) << np.uint64(56)))
        k1 = mix64(k0 + ((np.uint64(stream) << np.uint64(32)) | np.uint64(layer)))
        return mix64(k1 + np.asarray(gids, dtype=np.int64).astype(np.uint64))


def rows_bf16(seed: int, tensor: int, stream: int, layer: int, gids, heads: int, head_dim: int) -> np.ndarray:
    """bf16 bit patterns, shape [len(gids), heads, head_dim], for the given token ordinals."""
    gids = np.asarray(gids, dtype=np.int64).reshape(-1)
    keys = row_keys(seed, tensor, stream, layer, gids)
    e = np.arange(heads * head_dim, dtype=np.uint64)
    with np.errstate(over="ignore"):
        idx = (mix64(keys[:, None] + e[None, :]) >> np.uint64(48)).astype(np.int64)
    return normal_table()[idx].reshape(len(gids), heads, head_dim)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One row of the workload table: head geometry, cache policy and stream shape."""

    name: str
    seed: int
    layers: int
    q_heads: int
    kv_heads: int
    head_dim: int
    rope_mode: int            # 0 = 1D, 1 = MRoPE (t,h,w)
    rope_base: float
    sections: tuple           # pair counts per axis (MRoPE); ignored in 1D
    n_sink: int
    vision_window: int        # tokens
    text_window: int          # tokens
    frames: int               # vision block per chunk: frames x grid_h x grid_w tokens
    grid_h: int
    grid_w: int
    text_max: int             # text tokens per chunk ~ U{0..text_max}
    chunks: int
    decode_steps: int         # q=1 steps after each chunk
    streams: int = 1
    text_with_chunk: bool = True   # chunk's text tokens are prefilled together with its vision tokens

    @property
    def vision_per_chunk(self) -> int:
        return self.frames * self.grid_h * self.grid_w

    @property
    def max_chunk_tokens(self) -> int:
        return self.vision_per_chunk + self.text_max

    @property
    def retained(self) -> int:
        return self.n_sink + self.vision_window + self.text_window

    @property
    def capacity(self) -> int:
        """Tokens stored between two evictions, rounded up to a multiple of 128."""
        need = self.retained + self.max_chunk_tokens + self.decode_steps
        return (need + 127) // 128 * 128


def workloads() -> dict:
    """The five workload shapes (synthetic stand-ins for the paper's per-second sports streams)."""
    qwen = dict(q_heads=28, kv_heads=4, head_dim=128, rope_mode=1, rope_base=1.0e6, sections=(16, 24, 24),
                n_sink=512, text_window=512)
    return {
        1: Workload("tiny-1layer", 0x5EED0001, layers=1, q_heads=4, kv_heads=1, head_dim=64, rope_mode=0,
                    rope_base=1.0e4, sections=(32, 0, 0), n_sink=4, vision_window=64, text_window=128,
                    frames=1, grid_h=4, grid_w=8, text_max=8, chunks=20, decode_steps=4),
        2: Workload("qwen7b-1layer", 0x5EED0002, layers=1, vision_window=8192, frames=2, grid_h=16, grid_w=16,
                    text_max=24, chunks=600, decode_steps=16, **qwen),
        3: Workload("qwen7b-28layer", 0x5EED0003, layers=28, vision_window=8192, frames=2, grid_h=16, grid_w=16,
                    text_max=24, chunks=3600, decode_steps=16, **qwen),
        4: Workload("batched-decode-16", 0x5EED0004, layers=1, vision_window=8192, frames=2, grid_h=16, grid_w=16,
                    text_max=24, chunks=64, decode_steps=256, streams=16, **qwen),
        5: Workload("hfr-8stream-28layer", 0x5EED0005, layers=28, vision_window=8192, frames=8, grid_h=8, grid_w=8,
                    text_max=32, chunks=7200, decode_steps=16, streams=8, **qwen),
    }


class Stream:
    """Token schedule of one stream: per chunk the token types, native positions and ordinals (gids)."""

    def __init__(self, wl: Workload, stream: int = 0):
        self.wl = wl
        self.stream = stream
        self.next_gid = 0
        self.base = 0          # native position cursor of the caller
        self.chunk_index = 0

    def text_count(self, chunk: int) -> int:
        with np.errstate(over="ignore"):
            k = mix64(mix64(np.uint64(self.wl.seed) ^ np.uint64(0x7E87 << 40)) +
                      ((np.uint64(self.stream) << np.uint64(32)) | np.uint64(chunk)))
        return int(k % np.uint64(self.wl.text_max + 1))

    def _pos_text(self, n: int) -> np.ndarray:
        p = self.base + np.arange(n, dtype=np.int64)
        self.base += n
        if self.wl.rope_mode == 0:
            return p.astype(np.int32)
        return np.repeat(p[:, None], 3, axis=1).astype(np.int32)

    def _pos_vision(self) -> np.ndarray:
        wl = self.wl
        n = wl.vision_per_chunk
        if wl.rope_mode == 0:
            p = self.base + np.arange(n, dtype=np.int64)
            self.base += n
            return p.astype(np.int32)
        f, r, c = np.meshgrid(np.arange(wl.frames), np.arange(wl.grid_h), np.arange(wl.grid_w), indexing="ij")
        p = np.stack([f.reshape(-1), r.reshape(-1), c.reshape(-1)], axis=1).astype(np.int64) + self.base
        self.base += max(wl.frames, wl.grid_h, wl.grid_w)
        return p.astype(np.int32)

    def next_chunk(self):
        """Returns (gids int64[n], types uint8[n], pos int32[n] or [n,3]) of the next one-second chunk."""
        wl = self.wl
        nv = wl.vision_per_chunk
        nt = self.text_count(self.chunk_index)
        pv = self._pos_vision()
        pt = self._pos_text(nt)
        types = np.concatenate([np.full(nv, VISION, np.uint8), np.full(nt, TEXT, np.uint8)])
        pos = np.concatenate([pv, pt], axis=0)
        gids = self.next_gid + np.arange(nv + nt, dtype=np.int64)
        self.next_gid += nv + nt
        self.chunk_index += 1
        return gids, types, pos

    def next_decode_token(self):
        """One generated text token: (gids[1], types[1], pos[1] or [1,3])."""
        gids = np.array([self.next_gid], dtype=np.int64)
        self.next_gid += 1
        return gids, np.array([TEXT], np.uint8), self._pos_text(1)

    # value accessors -------------------------------------------------------------------------
    def k(self, layer: int, gids) -> np.ndarray:
        return rows_bf16(self.wl.seed, TENSOR_K, self.stream, layer, gids, self.wl.kv_heads, self.wl.head_dim)

    def v(self, layer: int, gids) -> np.ndarray:
        return rows_bf16(self.wl.seed, TENSOR_V, self.stream, layer, gids, self.wl.kv_heads, self.wl.head_dim)

    def q(self, layer: int, gids) -> np.ndarray:
        return rows_bf16(self.wl.seed, TENSOR_Q, self.stream, layer, gids, self.wl.q_heads, self.wl.head_dim)


# ---------------------------------------------------------------------------------------------
# The same generator with torch integer ops, for producing inputs directly in device memory
# (bit-identical to rows_bf16; torch is only the array library here).

def _t_lsr(x, k):
    import torch
    return (x >> k) & ((1 << (64 - k)) - 1)


def _t_const(v: int) -> int:
    return v - (1 << 64) if v >= (1 << 63) else v


def _t_mix64(x):
    z = x + _t_const(0x9E3779B97F4A7C15)
    z = (z ^ _t_lsr(z, 30)) * _t_const(0xBF58476D1CE4E5B9)
    z = (z ^ _t_lsr(z, 27)) * _t_const(0x94D049BB133111EB)
    return z ^ _t_lsr(z, 31)


_T_TABLES = {}


def rows_bf16_torch(seed: int, tensor: int, stream: int, layer: int, gids, heads: int, head_dim: int, device="cuda"):
    """bf16 tensor [len(gids), heads, head_dim] on `device`, bit-identical to rows_bf16."""
    import torch
    key = str(device)
    if key not in _T_TABLES:
        _T_TABLES[key] = torch.from_numpy(normal_table().view(np.int16)).to(device)
    table = _T_TABLES[key]
    g = torch.as_tensor(np.asarray(gids, dtype=np.int64), device=device) if not isinstance(gids, torch.Tensor) else gids
    k0 = int(mix64(np.uint64(seed) ^ (np.uint64(tensor) << np.uint64(56))))
    with np.errstate(over="ignore"):
        k1 = int(mix64(np.uint64(k0) + ((np.uint64(stream) << np.uint64(32)) | np.uint64(layer))))
    keys = _t_mix64(g + _t_const(k1))
    e = torch.arange(heads * head_dim, dtype=torch.int64, device=device)
    idx = _t_lsr(_t_mix64(keys[:, None] + e[None, :]), 48)
    return table[idx].view(torch.bfloat16).reshape(len(g), heads, head_dim)
