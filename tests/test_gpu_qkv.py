"""GPU parity of the projection whose epilogue appends to the cache (svlm_qkv_append) against oracle/qkv.py."""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _check_step(wl, hidden, n_warm, seed):
    """A few ordinary chunks (so that positions are shifted), then one chunk through svlm_qkv_append on every layer:
    queries, stored keys (rotated at the contiguous positions) and values against the fp64 statement, then the
    chunk's attention against the cache checker fed with the fp64 projection rounded to bf16."""
    from harness import SideBySide, assert_close, bits_to_dev, dev_to_f64
    from oracle import qkv
    from paper_2510_09608_b200 import binding, streamgen as sg
    rng = np.random.default_rng(seed)
    s = SideBySide(wl)
    for _ in range(n_warm):
        s.append_chunk()
        s.evict()
    gids, types, pos = s.stream.next_chunk()
    n = len(gids)
    n_out = (wl.q_heads + 2 * wl.kv_heads) * wl.head_dim
    ty, ps = torch.from_numpy(types).cuda(), torch.from_numpy(np.ascontiguousarray(pos)).cuda()
    s.ref.append(None, None, types, pos)
    Xs, Ws, Qg = [], [], []
    for l in range(wl.layers):
        Xs.append(qkv.to_bf16_bits(rng.standard_normal((n, hidden))))
        Ws.append(qkv.to_bf16_bits(rng.standard_normal((n_out, hidden)) / np.sqrt(hidden)))
        Qg.append(s.cache.qkv_append(l, bits_to_dev(Xs[l]), bits_to_dev(Ws[l]), wl.q_heads, ty if l == 0 else None, ps if l == 0 else None))
    assert s.cache.status() == binding.OK
    s.check_metadata()
    meta = s.ref.query()
    c_new = meta["pos"][-n:]
    assert np.array_equal(meta["gids"][-n:], gids)
    half = wl.head_dim // 2
    for l in range(wl.layers):
        Q64, K64, V64 = qkv.project(Xs[l], Ws[l], wl.q_heads, wl.kv_heads, wl.head_dim)
        # one rounding to bf16 (2^-8 relative, 2^-9 nominal) on top of fp32 accumulation over `hidden` terms
        acc = 1e-5 * np.sqrt(hidden)
        assert np.all(np.abs(dev_to_f64(Qg[l]) - Q64) <= 2.0 ** -8 * np.abs(Q64) + acc), "queries"
        Kb, Vb = s.cache.read_kv(l, len(meta["gids"]))
        assert np.all(np.abs(sg.bf16_bits_to_f64(Vb[-n:]) - V64) <= 2.0 ** -8 * np.abs(V64) + acc), "values"
        Kr = qkv.rotate(K64, c_new, wl.rope_mode, wl.rope_base, wl.sections)
        pn = np.sqrt(Kr[..., :half] ** 2 + Kr[..., half:] ** 2)
        pn = np.concatenate([pn, pn], axis=-1)
        assert np.all(np.abs(sg.bf16_bits_to_f64(Kb[-n:]) - Kr) <= 2.0 ** -8 * 1.05 * pn + acc), "rotated keys"
        # the checker's cache gets the fp64 projection rounded to bf16 (never anything the GPU produced)
        s.ref.set_kv(l, gids, qkv.to_bf16_bits(K64), qkv.to_bf16_bits(V64))
    s.evict()
    kept = s.ref.query()["gids"]
    old = kept[kept < gids[0]]
    for l in range(wl.layers):
        s.ref.set_kv(l, old, s.stream.k(l, old), s.stream.v(l, old))
        Q64 = qkv.project(Xs[l], Ws[l], wl.q_heads, wl.kv_heads, wl.head_dim)[0]
        out = dev_to_f64(s.cache.attend(l, Qg[l], ps))
        assert_close(s._stats(out, s.ref.attend(l, qkv.to_bf16_bits(Q64), pos)), tight=False)
    return n


def test_projection_with_append_small_mrope_and_1d():
    from paper_2510_09608_b200 import streamgen as sg
    wl = dataclasses.replace(sg.workloads()[2], layers=2, n_sink=16, vision_window=448, text_window=32, frames=3, grid_h=8, grid_w=8)
    n = _check_step(wl, hidden=192, n_warm=3, seed=11)
    assert n > 128                                  # two row tiles, the second ragged
    wl1 = dataclasses.replace(wl, rope_mode=0, rope_base=1.0e4, q_heads=8, kv_heads=1, frames=1)
    _check_step(wl1, hidden=64, n_warm=2, seed=12)


def test_projection_with_append_full_size_layer():
    """The Qwen2.5-VL-7B layer shape: hidden 3584 -> 28 query, 4 key, 4 value heads of 128, one steady-size chunk."""
    from paper_2510_09608_b200 import streamgen as sg
    wl = dataclasses.replace(sg.workloads()[2], layers=1, vision_window=1024, text_window=64, n_sink=32)
    n = _check_step(wl, hidden=3584, n_warm=2, seed=13)
    assert n >= 512


@pytest.mark.parametrize("n,in_dim,out_dim", [(70, 128, 384), (300, 192, 128), (524, 3584, 3584),
                                              (1, 3584, 4608), (3, 192, 128), (8, 3584, 3584), (16, 1024, 640)])
def test_output_projection(n, in_dim, out_dim):
    """svlm_out_proj against the fp64 product: ragged row tiles, an odd number of 128-column blocks, the full layer."""
    from harness import bits_to_dev, dev_to_f64
    from oracle import qkv
    from paper_2510_09608_b200 import binding
    rng = np.random.default_rng(n)
    A = qkv.to_bf16_bits(rng.standard_normal((n, in_dim)))
    W = qkv.to_bf16_bits(rng.standard_normal((out_dim, in_dim)) / np.sqrt(in_dim))
    c = binding.Cache(1, 1, 128, 4, 64, 16, 256)
    Y = dev_to_f64(c.out_proj(bits_to_dev(A), bits_to_dev(W)))
    want = qkv.out_project(A, W)
    assert c.status() == binding.OK
    assert np.all(np.abs(Y - want) <= 2.0 ** -8 * np.abs(want) + 1e-5 * np.sqrt(in_dim))
    with pytest.raises(binding.SvlmError) as e:
        c.out_proj(bits_to_dev(A), bits_to_dev(W[:out_dim - 64]))        # out_dim must be a multiple of 128
    assert e.value.status == binding.ERR_ARG


def test_decode_step_fed_by_the_projection():
    """One generated token the way a decoder layer runs it: [q | k | v] = W_qkv x through svlm_out_proj (the
    bandwidth kernel for a single row), then svlm_decode_step on the three slices; against the fp64 projection
    rounded to bf16 and the cache checker."""
    from harness import SideBySide, assert_close, bits_to_dev, dev_to_f64
    from oracle import qkv
    from paper_2510_09608_b200 import streamgen as sg
    wl = dataclasses.replace(sg.workloads()[2], layers=2, n_sink=16, vision_window=256, text_window=32, frames=1, grid_h=8, grid_w=8)
    hidden, d = 256, wl.head_dim
    rng = np.random.default_rng(21)
    s = SideBySide(wl)
    for _ in range(3):
        s.append_chunk()
        s.evict()
    nq, nk = wl.q_heads * d, wl.kv_heads * d
    for step in range(2):
        gids, types, pos = s.stream.next_decode_token()
        ty, ps = torch.from_numpy(types).cuda(), torch.from_numpy(np.ascontiguousarray(pos)).cuda()
        s.ref.append(None, None, types, pos)
        for l in range(wl.layers):
            x = qkv.to_bf16_bits(rng.standard_normal((1, hidden)))
            W = qkv.to_bf16_bits(rng.standard_normal((nq + 2 * nk, hidden)) / np.sqrt(hidden))
            y = s.cache.out_proj(bits_to_dev(x), bits_to_dev(W))                       # [1, (Hq + 2 Hkv) d]
            Q, K, V = y[:, :nq].view(1, wl.q_heads, d), y[:, nq:nq + nk].view(1, wl.kv_heads, d), y[:, nq + nk:].view(1, wl.kv_heads, d)
            out = dev_to_f64(s.cache.decode_step(l, K.contiguous(), V.contiguous(), ty if l == 0 else None, ps, Q.contiguous()))
            Q64, K64, V64 = qkv.project(x, W, wl.q_heads, wl.kv_heads, d)
            old = s.ref.query()["gids"][:-1]
            s.ref.set_kv(l, old, s.stream.k(l, old), s.stream.v(l, old)) if step == 0 else None
            s.ref.set_kv(l, gids, qkv.to_bf16_bits(K64), qkv.to_bf16_bits(V64))
            assert_close(s._stats(out, s.ref.attend(l, qkv.to_bf16_bits(Q64), pos)), tight=False)
    s.check_metadata()


def test_projection_argument_errors():
    from paper_2510_09608_b200 import binding
    c = binding.Cache(1, 2, 128, 4, 64, 16, 256)
    X = torch.zeros(8, 96, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((4 + 4) * 128, 96, dtype=torch.bfloat16, device="cuda")
    ty = torch.zeros(8, dtype=torch.uint8, device="cuda")
    pos = torch.arange(8, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.SvlmError) as e:          # hidden must be a multiple of 64
        c.qkv_append(0, X, W, 4, ty, pos)
    assert e.value.status == binding.ERR_ARG
    c64 = binding.Cache(1, 2, 64, 4, 64, 16, 256)
    with pytest.raises(binding.SvlmError) as e:          # head_dim 128 only
        c64.qkv_append(0, torch.zeros(8, 128, dtype=torch.bfloat16, device="cuda"),
                       torch.zeros(8 * 64, 128, dtype=torch.bfloat16, device="cuda"), 4, ty, pos)
    assert e.value.status == binding.ERR_ARG
