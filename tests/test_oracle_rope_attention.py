"""CPU pins for the checker's rotation and attention (closed forms, a library routine, special cases)."""
import math

import numpy as np
import pytest
import torch

from oracle import INF, ROPE_1D, ROPE_MROPE, TEXT, VISION, Oracle
from oracle import brute
from paper_2510_09608_b200 import streamgen as sg


def _bits(x):
    return sg._f32_to_bf16_bits(np.asarray(x, np.float32))


def test_rotation_closed_forms():
    o = Oracle(1, 1, 2, 0, INF, INF, rope_base=10000.0)
    # d=2: one pair, theta=1: plain planar rotation by c radians
    y = o.rotate([1.0, 0.0], [3, 3, 3])
    assert np.allclose(y, [math.cos(3), math.sin(3)], atol=1e-15)
    y = o.rotate([0.0, 1.0], [3, 3, 3])
    assert np.allclose(y, [-math.sin(3), math.cos(3)], atol=1e-15)
    # d=4: pairs (0,2) and (1,3); theta_1 = base^(-1/2) = 0.01
    o4 = Oracle(1, 1, 4, 0, INF, INF, rope_base=10000.0)
    y = o4.rotate([0.0, 1.0, 0.0, 0.0], [50, 50, 50])
    assert np.allclose(y, [0.0, math.cos(0.5), 0.0, math.sin(0.5)], atol=1e-15)
    y = o4.rotate([2.0, 0.0, 0.0, 0.0], [5, 5, 5])
    assert np.allclose(y, [2 * math.cos(5), 0.0, 2 * math.sin(5), 0.0], atol=1e-15)


@pytest.mark.parametrize("mode", [ROPE_1D, ROPE_MROPE])
def test_rotation_group_identities(mode):
    rng = np.random.default_rng(0)
    d = 16
    o = Oracle(1, 1, d, 0, INF, INF, rope_mode=mode, rope_base=1.0e6, sections=(2, 3, 3))
    x = rng.standard_normal(d)
    a = rng.integers(-50, 900, 3)
    b = rng.integers(-50, 900, 3)
    if mode == ROPE_1D:
        a[:] = a[0]
        b[:] = b[0]
    assert np.allclose(o.rotate(o.rotate(x, a), b), o.rotate(x, a + b), atol=1e-11)
    assert np.allclose(o.rotate(x, [0, 0, 0]), x, atol=0)
    assert abs(np.linalg.norm(o.rotate(x, a)) - np.linalg.norm(x)) < 1e-12
    # logits depend on position differences only
    y = rng.standard_normal(d)
    s0 = o.rotate(x, a) @ o.rotate(y, b)
    s1 = o.rotate(x, a + 37) @ o.rotate(y, b + 37)
    assert abs(s0 - s1) < 1e-10


def test_mrope_sections_select_the_axis():
    d, sections = 16, (2, 3, 3)
    o = Oracle(1, 1, d, 0, INF, INF, rope_mode=ROPE_MROPE, rope_base=100.0, sections=sections)
    axis = np.repeat(np.arange(3), sections)
    for i in range(d // 2):
        x = np.zeros(d)
        x[i] = 1.0
        c = np.array([11, 23, 37])
        theta = 100.0 ** (-2.0 * i / d)
        y = o.rotate(x, c)
        want = np.zeros(d)
        want[i], want[i + d // 2] = math.cos(c[axis[i]] * theta), math.sin(c[axis[i]] * theta)
        assert np.allclose(y, want, atol=1e-14)
    # and the separately written numpy rotation agrees on random input
    x = np.random.default_rng(1).standard_normal(d)
    assert np.allclose(o.rotate(x, [5, 9, 2]), brute.rope(x, [5, 9, 2], 100.0, sections), atol=1e-13)


def test_incremental_rerotation_equals_fresh_rotation():
    """Rotating stored (already rotated) keys by -delta equals rotating raw keys at the new position."""
    rng = np.random.default_rng(3)
    d = 32
    o = Oracle(1, 1, d, 0, INF, INF, rope_mode=ROPE_MROPE, rope_base=1.0e6, sections=(4, 6, 6))
    x = rng.standard_normal(d)
    c = np.array([700, 650, 712])
    y = o.rotate(x, c)
    for delta in (3, 16, 44, 129):
        y = o.rotate(y, [-delta] * 3)
        c = c - delta
        assert np.allclose(y, o.rotate(x, c), atol=1e-12)


@pytest.mark.parametrize("hq,hkv,d", [(4, 1, 16), (6, 2, 8), (4, 4, 32)])
def test_no_eviction_equals_library_causal_attention(hq, hkv, d):
    rng = np.random.default_rng(5)
    n0, nq = 9, 7
    o = Oracle(1, hkv, d, 0, INF, INF, rope_base=10000.0)
    K = _bits(rng.standard_normal((1, n0 + nq, hkv, d)))
    V = _bits(rng.standard_normal((1, n0 + nq, hkv, d)))
    Q = _bits(rng.standard_normal((nq, hq, d)))
    types = rng.integers(0, 2, n0 + nq).astype(np.uint8)
    pos = np.arange(n0 + nq, dtype=np.int32)
    o.append(K[:, :n0], V[:, :n0], types[:n0], pos[:n0])
    o.evict()
    o.append(K[:, n0:], V[:, n0:], types[n0:], pos[n0:])
    o.evict()
    assert o.count() == n0 + nq
    got = o.attend(0, Q, pos[n0:])
    kf, vf, qf = sg.bf16_bits_to_f64(K[0]), sg.bf16_bits_to_f64(V[0]), sg.bf16_bits_to_f64(Q)
    krot = np.stack([brute.rope(kf[j], [pos[j]] * 3, 10000.0) for j in range(n0 + nq)])
    qrot = np.stack([brute.rope(qf[r], [pos[n0 + r]] * 3, 10000.0) for r in range(nq)])
    g = hq // hkv
    kt = torch.from_numpy(krot).permute(1, 0, 2).repeat_interleave(g, dim=0)     # [hq, n, d]
    vt = torch.from_numpy(vf).permute(1, 0, 2).repeat_interleave(g, dim=0)
    qt = torch.from_numpy(qrot).permute(1, 0, 2)                                # [hq, nq, d]
    mask = torch.ones(nq, n0 + nq, dtype=torch.bool).tril(diagonal=n0)          # bottom-right causal
    want = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask).permute(1, 0, 2).numpy()
    assert np.allclose(got, want, atol=1e-12)


def test_attention_special_cases():
    rng = np.random.default_rng(6)
    d = 8
    # a single visible key: the output is its value
    o = Oracle(1, 1, d, 0, INF, INF)
    K, V = _bits(rng.standard_normal((1, 1, 1, d))), _bits(rng.standard_normal((1, 1, 1, d)))
    o.append(K, V, [TEXT], [0])
    out = o.attend(0, _bits(rng.standard_normal((1, 2, d))), [0])
    assert np.allclose(out[0, 0], sg.bf16_bits_to_f64(V[0, 0, 0]), atol=1e-15)
    assert np.allclose(out[0, 1], sg.bf16_bits_to_f64(V[0, 0, 0]), atol=1e-15)
    # identical keys at the same position: the output is the mean of the values
    o = Oracle(1, 1, d, 0, INF, INF, rope_mode=ROPE_MROPE, sections=(2, 1, 1))
    k1 = _bits(rng.standard_normal((1, 1, 1, d)))
    K = np.repeat(k1, 5, axis=1)
    V = _bits(rng.standard_normal((1, 5, 1, d)))
    o.append(K, V, [VISION] * 5, np.tile([[4, 4, 4]], (5, 1)))
    out = o.attend(0, _bits(rng.standard_normal((1, 1, d))), [[9, 9, 9]])
    assert np.allclose(out[0, 0], sg.bf16_bits_to_f64(V[0, :, 0]).mean(0), atol=1e-14)
    # a query that was appended but whose own token (and everything else) was evicted sees nothing
    o = Oracle(1, 1, d, 0, 0, 0)
    o.append(_bits(rng.standard_normal((1, 3, 1, d))), _bits(rng.standard_normal((1, 3, 1, d))), [VISION] * 3, [0, 1, 2])
    o.evict()
    assert np.all(o.attend(0, _bits(rng.standard_normal((3, 1, d))), [0, 1, 2]) == 0)


@pytest.mark.parametrize("mode", [ROPE_1D, ROPE_MROPE])
def test_tiny_stream_equals_brute_force_over_kept_set(mode):
    """Evicting cache + checker attention == dense attention restricted to the closed-form kept set."""
    rng = np.random.default_rng(11 + mode)
    hq, hkv, d, S, Vw, Tw = 4, 2, 8, 2, 8, 3
    sections = (2, 1, 1)
    o = Oracle(1, hkv, d, S, Vw, Tw, rope_mode=mode, rope_base=100.0, sections=sections)
    items, types_hist = [], []
    Ks, Vs = [], []
    for step in range(9):
        new = [("V", 1, 2, 2)] + [("T",)] * int(rng.integers(0, 3))
        n_before = len(types_hist)
        items += new
        tnew = [VISION] * 4 + [TEXT] * (len(new) - 1)
        types_hist += tnew
        n = len(tnew)
        if mode == ROPE_MROPE:
            native = brute.assign_positions(items)
            pos = native[n_before:].astype(np.int32)
        else:
            native = np.repeat(np.arange(len(types_hist))[:, None], 3, 1)
            pos = native[n_before:, 0].astype(np.int32)
        K, V = _bits(rng.standard_normal((1, n, hkv, d))), _bits(rng.standard_normal((1, n, hkv, d)))
        Q = _bits(rng.standard_normal((n, hq, d)))
        Ks.append(K[0]); Vs.append(V[0])
        o.append(K, V, np.array(tnew, np.uint8), pos)
        o.evict()
        got = o.attend(0, Q, pos)
        # brute force: closed-form kept set, positions = native minus the span freed before each token
        mask = brute.kept_mask(np.array(types_hist), S, Vw, Tw)
        kall, vall = sg.bf16_bits_to_f64(np.concatenate(Ks)), sg.bf16_bits_to_f64(np.concatenate(Vs))
        adv = np.diff(np.maximum.accumulate(np.concatenate([[0], native.max(1) + 1])))
        freed_before = np.cumsum(np.where(mask, 0, adv)) - np.where(mask, 0, adv)
        cpos = native - freed_before[:, None]
        total_freed = int(np.where(mask, 0, adv).sum())
        kept = np.flatnonzero(mask)
        sec = sections if mode == ROPE_MROPE else None
        qf = sg.bf16_bits_to_f64(Q)
        for h in range(hq):
            g = h // (hq // hkv)
            krot = np.stack([brute.rope(kall[j, g], cpos[j], 100.0, sec) for j in kept])
            qrot = np.stack([brute.rope(qf[r, h], native[n_before + r] - total_freed, 100.0, sec) for r in range(n)])
            vis = kept[None, :] <= (n_before + np.arange(n))[:, None]
            want = brute.attention(qrot, krot, vall[kept, g], vis)
            assert np.allclose(got[:, h], want, atol=1e-12), (step, h)


@pytest.mark.parametrize("mode", [ROPE_1D, ROPE_MROPE])
def test_late_values_and_row_subsets_equal_brute_force(mode):
    """The two entry points the long-stream GPU tests lean on: values handed over after the fact by
    stream ordinal (`set_kv`, shuffled, with ordinals that are no longer stored mixed in) and the
    `rows` subset of `attend`.  Pinned against dense numpy attention over the closed-form kept set,
    against the same stream fed with values at append time, and against the full-row result."""
    rng = np.random.default_rng(23 + mode)
    hq, hkv, d, S, Vw, Tw, L = 6, 2, 8, 2, 8, 3, 2
    sections = (2, 1, 1)
    kw = dict(rope_mode=mode, rope_base=100.0, sections=sections)
    early = Oracle(L, hkv, d, S, Vw, Tw, **kw)     # K/V supplied with the append
    late = Oracle(L, hkv, d, S, Vw, Tw, **kw)      # metadata only; K/V by set_kv before attending
    items, types_hist, Ks, Vs = [], [], [], []
    for step in range(10):
        new = [("V", 1, 2, 2)] + [("T",)] * int(rng.integers(0, 4))
        n_before = len(types_hist)
        items += new
        tnew = [VISION] * 4 + [TEXT] * (len(new) - 1)
        types_hist += tnew
        n = len(tnew)
        if mode == ROPE_MROPE:
            native = brute.assign_positions(items)
            pos = native[n_before:].astype(np.int32)
        else:
            native = np.repeat(np.arange(len(types_hist))[:, None], 3, 1)
            pos = native[n_before:, 0].astype(np.int32)
        K, V = _bits(rng.standard_normal((L, n, hkv, d))), _bits(rng.standard_normal((L, n, hkv, d)))
        Q = _bits(rng.standard_normal((n, hq, d)))
        Ks.append(K); Vs.append(V)
        early.append(K, V, np.array(tnew, np.uint8), pos)
        late.append(None, None, np.array(tnew, np.uint8), pos)
        early.evict(); late.evict()
        kall, vall = np.concatenate(Ks, axis=1), np.concatenate(Vs, axis=1)    # [L, history, hkv, d]
        mask = brute.kept_mask(np.array(types_hist), S, Vw, Tw)
        kept = np.flatnonzero(mask)
        assert np.array_equal(late.query()["gids"], kept)
        if step < 2:
            continue
        layer = step % L
        # before any value arrives (or with one stored token left out) attention must refuse
        if step in (2, 3):
            with pytest.raises(RuntimeError):
                late.attend(layer, Q, pos)
            hole = kept[kept != kept[len(kept) // 2]]
            late.set_kv(layer, hole, kall[layer, hole], vall[layer, hole])
            with pytest.raises(RuntimeError):
                late.attend(layer, Q, pos)
        # every ordinal of the history in shuffled order: the evicted ones must be skipped silently
        order = rng.permutation(len(types_hist))
        late.set_kv(layer, order, kall[layer, order], vall[layer, order])
        assert np.array_equal(late.query()["gids"], kept), "set_kv must not change what is stored"
        full_early = early.attend(layer, Q, pos)
        full_late = late.attend(layer, Q, pos)
        assert np.allclose(full_late, full_early, atol=1e-12)
        rows = rng.permutation(n)[: max(1, n // 2)]
        sub = late.attend(layer, Q, pos, rows=rows)
        assert sub.shape == (len(rows), hq, d)
        assert np.allclose(sub, full_late[rows], atol=1e-12)
        assert np.allclose(early.attend(layer, Q, pos, rows=rows[::-1]), full_early[rows[::-1]], atol=1e-12)
        # dense numpy over the closed-form kept set, for the chosen rows only
        adv = np.diff(np.maximum.accumulate(np.concatenate([[0], native.max(1) + 1])))
        freed = np.where(mask, 0, adv)
        cpos = native - (np.cumsum(freed) - freed)[:, None]
        total_freed = int(freed.sum())
        sec = sections if mode == ROPE_MROPE else None
        kf, vf, qf = sg.bf16_bits_to_f64(kall[layer]), sg.bf16_bits_to_f64(vall[layer]), sg.bf16_bits_to_f64(Q)
        for h in range(hq):
            g = h // (hq // hkv)
            krot = np.stack([brute.rope(kf[j, g], cpos[j], 100.0, sec) for j in kept])
            qrot = np.stack([brute.rope(qf[r, h], native[n_before + r] - total_freed, 100.0, sec) for r in rows])
            vis = kept[None, :] <= (n_before + rows)[:, None]
            want = brute.attention(qrot, krot, vf[kept, g], vis)
            assert np.allclose(sub[:, h], want, atol=1e-12), (step, h)
