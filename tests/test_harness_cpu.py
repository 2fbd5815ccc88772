"""CPU checks of the comparison helpers the GPU tests rely on (no device needed)."""
import dataclasses

import numpy as np

import oracle
from paper_2510_09608_b200 import streamgen as sg


def test_rotation_counter_equals_a_per_token_tally():
    """The per-token re-rotation count that bounds the stored-key error: against a dictionary kept by hand."""
    from harness import RotationCounter
    wl = dataclasses.replace(sg.workloads()[2], n_sink=8, vision_window=64, text_window=16, frames=1, grid_h=4,
                             grid_w=4, decode_steps=2)
    st = sg.Stream(wl, 0)
    ref = oracle.Oracle(1, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window,
                        rope_mode=wl.rope_mode, rope_base=wl.rope_base, sections=wl.sections)
    rc, tally = RotationCounter(), {}
    for chunk in range(30):
        _, t, p = st.next_chunk()
        ref.append(None, None, t, p)
        b = ref.query()
        before = {int(g): tuple(c) for g, c in zip(b["gids"], b["pos"])}
        rc.evict(ref)
        a = ref.query()
        tally = {int(g): tally.get(int(g), 0) + (before[int(g)] != tuple(c)) for g, c in zip(a["gids"], a["pos"])}
        assert np.array_equal(rc.of(a["gids"]), [tally[int(g)] for g in a["gids"]]), chunk
        for _ in range(wl.decode_steps):
            _, t, p = st.next_decode_token()
            ref.append(None, None, t, p)
        a = ref.query()
        assert np.array_equal(rc.of(a["gids"]), [tally.get(int(g), 0) for g in a["gids"]])
    vis = a["types"] == sg.VISION
    # a vision token is moved at most once per chunk of its stay in the window
    assert rc.of(a["gids"])[vis].max() <= wl.vision_window // wl.vision_per_chunk


def test_key_rounding_bound_scales_with_the_tokens_own_count():
    from harness import key_rounding_bound
    k = np.zeros((2, 1, 4))
    k[:, 0] = [3.0, 0.0, 4.0, 1.0]          # pairs (0,2) norm 5, (1,3) norm 1
    b = key_rounding_bound(k, [1, 10])
    assert np.allclose(b[0, 0], np.array([5, 1, 5, 1]) * 2.0 ** -8 * 1.05 + 1e-6)
    assert np.allclose(b[1, 0] - 1e-6, 10 * (b[0, 0] - 1e-6))
