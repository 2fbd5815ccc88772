"""CPU pins for the checker's eviction policy and position re-indexing (paper Section 2.1)."""
import os

import numpy as np
import pytest

from oracle import INF, ROPE_1D, ROPE_MROPE, TEXT, VISION, Oracle
from oracle import brute

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _meta_oracle(S, Vw, Tw, mode=ROPE_1D, **kw):
    return Oracle(1, 1, 8, S, Vw, Tw, rope_mode=mode, sections=(2, 1, 1), **kw)


def test_fig3_toy_by_hand():
    rows = []
    for line in open(os.path.join(GOLDEN, "fig3_toy.txt")):
        if line.startswith("#") or not line.strip():
            continue
        sec, gids, pos, shift = [f.strip() for f in line.split("|")]
        rows.append((int(sec), [int(x) for x in gids.split()], [int(x) for x in pos.split()], int(shift)))
    o = _meta_oracle(1, 4, 3)
    o.append(None, None, [TEXT], [0])
    g = 1
    for sec, gids, pos, shift in rows:
        o.append(None, None, [VISION, VISION, TEXT], [g, g + 1, g + 2])
        g += 3
        o.evict()
        q = o.query()
        assert q["gids"].tolist() == gids
        assert q["pos"][:, 0].tolist() == pos
        assert q["shift_total"] == shift


def _random_stream(rng, n_steps, mode):
    """Yields (types, items) per append; items describe blocks for the from-scratch position rule."""
    for _ in range(n_steps):
        types, items = [], []
        for _ in range(rng.integers(1, 4)):
            if rng.random() < 0.5:
                F, H, W = (int(rng.integers(1, 3)), int(rng.integers(1, 4)), int(rng.integers(1, 4)))
                types += [VISION] * (F * H * W)
                items.append(("V", F, H, W))
            else:
                k = int(rng.integers(1, 5))
                types += [TEXT] * k
                items += [("T",)] * k
        yield np.array(types, np.uint8), items


@pytest.mark.parametrize("seed", range(12))
@pytest.mark.parametrize("sink_any", [False, True])
def test_incremental_equals_closed_form_1d(seed, sink_any):
    rng = np.random.default_rng(seed)
    S, Vw, Tw = int(rng.integers(0, 6)), int(rng.integers(0, 20)), int(rng.integers(0, 12))
    o = _meta_oracle(S, Vw, Tw, sink_any_type=sink_any)
    hist = []
    prev_kept = None
    for types, _ in _random_stream(rng, 40, ROPE_1D):
        pos = np.arange(len(hist), len(hist) + len(types), dtype=np.int32)
        hist += types.tolist()
        o.append(None, None, types, pos)
        if rng.random() < 0.7:
            o.evict()
            q = o.query()
            mask = brute.kept_mask(np.array(hist), S, Vw, Tw, sink_any)
            assert q["gids"].tolist() == np.flatnonzero(mask).tolist()
            # contiguous 1D: kept tokens in stream order sit at 0..R-1
            assert q["pos"][:, 0].tolist() == list(range(len(q["gids"])))
            assert q["shift_total"] == len(hist) - len(q["gids"])
            if not sink_any:
                nt = int((np.array(hist) == TEXT).sum())
                nv = len(hist) - nt
                assert int((q["types"] == TEXT).sum()) == min(nt, S + Tw)
                assert int((q["types"] == VISION).sum()) == min(nv, Vw)
                text_gids = np.flatnonzero(np.array(hist) == TEXT)[:S]
                assert set(text_gids.tolist()) <= set(q["gids"].tolist())
            if prev_kept is not None:   # nested over time: nothing evicted comes back
                old = set(g for g in q["gids"].tolist() if g < prev_n)
                assert old <= prev_kept
            prev_kept, prev_n = set(q["gids"].tolist()), len(hist)
    # a token appended after the last evict continues from the last retained position
    o.evict()
    n = o.count()
    o.append(None, None, [TEXT], [len(hist)])
    assert o.query()["pos"][-1, 0] == n


@pytest.mark.parametrize("seed", range(8))
def test_3d_positions_equal_from_scratch_assignment(seed):
    """Whole-block eviction: left-shifted 3D indices == re-running the 3D rule on the kept sequence."""
    rng = np.random.default_rng(100 + seed)
    F, H, W = int(rng.integers(1, 4)), int(rng.integers(1, 5)), int(rng.integers(1, 5))
    blk = F * H * W
    S, Tw, Vw = int(rng.integers(0, 4)), int(rng.integers(0, 6)), blk * int(rng.integers(1, 4))
    o = _meta_oracle(S, Vw, Tw, mode=ROPE_MROPE)
    hist_types, hist_items, item_of_token = [], [], []
    native = []
    for step in range(30):
        items = [("V", F, H, W)] + [("T",)] * int(rng.integers(0, 4))
        if step == 0:
            items = [("T",)] * 2 + items
        types = []
        for it in items:
            k = 1 if it[0] == "T" else blk
            item_of_token += [len(hist_items)] * k
            hist_items.append(it)
            types += [TEXT if it[0] == "T" else VISION] * k
        hist_types += types
        allpos = brute.assign_positions(hist_items)      # native = the rule run over the whole stream
        pos = allpos[len(hist_types) - len(types):].astype(np.int32)
        o.append(None, None, np.array(types, np.uint8), pos)
        o.evict()
        q = o.query()
        mask = brute.kept_mask(np.array(hist_types), S, Vw, Tw)
        assert q["gids"].tolist() == np.flatnonzero(mask).tolist()
        kept_items = sorted(set(np.array(item_of_token)[mask].tolist()))
        expect = brute.assign_positions([hist_items[i] for i in kept_items])
        assert np.array_equal(q["pos"].astype(np.int64), expect)
        assert q["cursor"] == allpos.max() + 1
        # the next text token lands right after the last retained index
        assert q["cursor"] - q["shift_total"] == expect.max() + 1


def test_positions_stay_bounded_on_a_long_stream():
    """'effective RoPE indices stop growing and remain within a bounded range' (Contiguous RoPE paragraph)."""
    S, Vw, Tw = 4, 64, 16
    o = _meta_oracle(S, Vw, Tw, mode=ROPE_MROPE)
    rng = np.random.default_rng(7)
    items = []
    seen_max = 0
    for step in range(400):
        new = [("V", 2, 4, 4)] + [("T",)] * int(rng.integers(0, 5))
        n_before = len(brute.assign_positions(items))
        items += new
        allpos = brute.assign_positions(items)
        types = [VISION] * 32 + [TEXT] * (len(new) - 1)
        o.append(None, None, np.array(types, np.uint8), allpos[n_before:].astype(np.int32))
        o.evict()
        seen_max = max(seen_max, int(o.query()["pos"].max()))
    # S + Tw text spans, two blocks of span 4 in the window, nothing else
    assert seen_max <= S + Tw + (Vw // 32) * 4
    assert o.query()["cursor"] > 10 * seen_max      # native indices kept growing meanwhile


@pytest.mark.parametrize("S,Vw,Tw", [(0, 8, 4), (4, 0, 4), (4, 8, 0), (0, 0, 0), (INF, INF, INF)])
def test_degenerate_windows(S, Vw, Tw):
    o = _meta_oracle(S, Vw, Tw)
    types = np.array(([VISION] * 4 + [TEXT] * 3) * 6, np.uint8)
    o.append(None, None, types, np.arange(len(types), dtype=np.int32))
    o.evict()
    q = o.query()
    assert q["gids"].tolist() == np.flatnonzero(brute.kept_mask(types, S, Vw, Tw)).tolist()
    if S == INF:
        assert o.count() == len(types) and q["shift_total"] == 0
    if (S, Vw, Tw) == (0, 0, 0):
        assert o.count() == 0 and q["shift_total"] == len(types)


def test_native_rope_switch_never_shifts():
    o = _meta_oracle(1, 4, 3, contiguous=False)
    for s in range(6):
        o.append(None, None, [VISION, VISION, TEXT], [3 * s, 3 * s + 1, 3 * s + 2])
        o.evict()
    q = o.query()
    assert q["pos"][:, 0].tolist() == q["gids"].tolist() and q["shift_total"] == 0
