"""TEST INFRASTRUCTURE: brute-force restatements used to pin svlm_oracle.cpp.

Nothing here evicts incrementally.  The kept set is computed from the *whole* history with the
closed-form rule of the paper's "Streaming-aware KV Cache" paragraph; positions are re-assigned
from scratch over the kept sequence (1D: ranks; 3D: the Qwen-VL style block rule run again from
zero, which is what "assemble them by the 3D rule" in the "Contiguous RoPE" paragraph must equal
when whole vision blocks are evicted); attention is dense numpy over the kept set.
"""
from __future__ import annotations

import numpy as np

TEXT, VISION = 0, 1


def kept_mask(types: np.ndarray, n_sink: int, vision_window: int, text_window: int, sink_any_type=False):
    """Boolean mask over the full history: which tokens the policy retains right now.

    The policy is monotone (an evicted token never returns), so the incremental cache after any
    sequence of evictions ending now holds exactly the tokens this mask marks."""
    types = np.asarray(types)
    is_text = types == TEXT
    ord_text = np.cumsum(is_text) - 1
    ord_vis = np.cumsum(~is_text) - 1
    n_text, n_vis = int(is_text.sum()), int((~is_text).sum())
    recent_text = is_text & (ord_text >= n_text - text_window)
    recent_vis = (~is_text) & (ord_vis >= n_vis - vision_window)
    if sink_any_type:
        sink = np.arange(len(types)) < n_sink
    else:
        sink = is_text & (ord_text < n_sink)
    return sink | recent_text | recent_vis


def assign_positions(items):
    """Position assignment from zero over a sequence of items.

    items: list of ("T",) for a text token or ("V", frames, h, w) for a whole vision block.
    Returns int64 [n_tokens, 3].  Text takes (b,b,b) and advances b by one; a block starting at b
    gives token (f,r,c) the index (b+f, b+r, b+c) and advances b by max(frames, h, w)."""
    out = []
    b = 0
    for it in items:
        if it[0] == "T":
            out.append((b, b, b))
            b += 1
        else:
            _, F, H, W = it
            for f in range(F):
                for r in range(H):
                    for c in range(W):
                        out.append((b + f, b + r, b + c))
            b += max(F, H, W)
    return np.asarray(out, dtype=np.int64).reshape(-1, 3)


def rope(x: np.ndarray, c3, base: float, sections=None):
    """Rotate the last axis of x (length d) at position c3 = (t,h,w); sections None means 1D (uses c3[0])."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    half = d // 2
    i = np.arange(half)
    theta = base ** (-2.0 * i / d)
    if sections is None:
        pos = np.full(half, c3[0], dtype=np.float64)
    else:
        axis = np.repeat(np.arange(3), sections)
        pos = np.asarray(c3, dtype=np.float64)[axis]
    ang = pos * theta
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * np.cos(ang) - hi * np.sin(ang), hi * np.cos(ang) + lo * np.sin(ang)], axis=-1)


def attention(q_rot: np.ndarray, k_rot: np.ndarray, v: np.ndarray, visible: np.ndarray):
    """q_rot [n_q,d], k_rot/v [n_k,d], visible bool [n_q,n_k] -> [n_q,d]; empty rows give zeros."""
    d = q_rot.shape[-1]
    s = q_rot @ k_rot.T / np.sqrt(d)
    s = np.where(visible, s, -np.inf)
    out = np.zeros((q_rot.shape[0], v.shape[-1]))
    for r in range(q_rot.shape[0]):
        if not visible[r].any():
            continue
        w = np.exp(s[r] - s[r][visible[r]].max())
        w = np.where(visible[r], w, 0.0)
        out[r] = (w / w.sum()) @ v
    return out
