"""TEST INFRASTRUCTURE: fp64 statement of the step on the input side of the path, the Q/K/V projection whose
epilogue appends to the cache (plain numpy, no blocking, no fusion).

The paper's cache holds, for every retained token, the key and value of each layer, with the key carrying the
rotary position of the "Contiguous RoPE" paragraph (Section 2.1); a decoder layer obtains them as linear maps of
its input activations.  What is stored for a new token i with input row x_i is therefore

    q_i = W_q x_i,   k_i = R(c_i) W_k x_i,   v_i = W_v x_i,

with R(c) the rotary map of the token's contiguous position c_i (pairs (j, j + d/2), angle c_axis(j) * theta_j,
theta_j = base^(-2j/d); 1D: one axis; MRoPE: pair j uses t for j < s0, h for s0 <= j < s0 + s1, w otherwise).
The query is returned un-rotated: attention rotates it at its own position.

Only tests and the benchmark's CPU leg may import this module; the CUDA library never does.
"""
from __future__ import annotations

import numpy as np


def widen(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float64, exactly."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def project(X_bits: np.ndarray, W_bits: np.ndarray, q_heads: int, kv_heads: int, head_dim: int):
    """X: bf16 bits [n, hidden]; W: bf16 bits [(q_heads + 2 kv_heads) * head_dim, hidden], rows ordered query
    heads, key heads, value heads.  Returns fp64 (Q [n, q_heads, d], K [n, kv_heads, d], V [n, kv_heads, d])."""
    X, W = widen(X_bits), widen(W_bits)
    n = X.shape[0]
    assert W.shape == ((q_heads + 2 * kv_heads) * head_dim, X.shape[1])
    Y = X @ W.T
    nq, nk = q_heads * head_dim, kv_heads * head_dim
    return (Y[:, :nq].reshape(n, q_heads, head_dim), Y[:, nq:nq + nk].reshape(n, kv_heads, head_dim),
            Y[:, nq + nk:].reshape(n, kv_heads, head_dim))


def out_project(A_bits: np.ndarray, Wo_bits: np.ndarray) -> np.ndarray:
    """The projection on the output side, y_i = W_o a_i: A bf16 bits [n, in_dim], Wo [out_dim, in_dim] -> fp64 [n, out_dim]."""
    return widen(A_bits) @ widen(Wo_bits).T


def rotate(x: np.ndarray, c: np.ndarray, rope_mode: int, base: float, sections) -> np.ndarray:
    """R(c) x for x [n, heads, d] and integer positions c [n, 3] (1D mode reads column 0)."""
    n, _, d = x.shape
    half = d // 2
    j = np.arange(half)
    theta = np.power(float(base), -2.0 * j / d)
    c = np.asarray(c, dtype=np.int64).reshape(n, -1)
    if rope_mode == 0:
        pos = np.repeat(c[:, :1], half, axis=1)
    else:
        axis = np.where(j < sections[0], 0, np.where(j < sections[0] + sections[1], 1, 2))
        pos = c[:, axis]
    ang = pos.astype(np.float64) * theta[None, :]
    cs, sn = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * cs - hi * sn, hi * cs + lo * sn], axis=-1)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp64 -> bf16 bit patterns (via fp32; finite inputs of moderate size)."""
    u = np.asarray(x, dtype=np.float64).astype(np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)
