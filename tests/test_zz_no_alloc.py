"""The decode entry point that allocates nothing (svlm_attend_decode_noalloc) against svlm_attend.

Some users of the library cannot call the CUDA allocator at the time they attend (all device memory
already belongs to their own pool, or they run where allocation is not allowed), so one entry point
keeps its split-KV scratch in a fixed array inside the library.  This file checks that it returns
what the regular entry point returns, twice in a row, since every call reuses the same array and
must clean up after the previous one.  It is named to be collected last.
"""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_noalloc_decode_matches_regular_entry_point_twice():
    import oracle
    from harness import MAX_ABS, MEAN_ABS, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding, streamgen as sg

    wl = dataclasses.replace(sg.workloads()[2], layers=2, n_sink=40, vision_window=5 * 128, text_window=70,
                             frames=2, grid_h=8, grid_w=8, text_max=24)
    stream = sg.Stream(wl, 0)
    cache = binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
    cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
    ref = oracle.Oracle(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window,
                        rope_mode=wl.rope_mode, rope_base=wl.rope_base, sections=wl.sections)

    def append(gids, types, pos):
        K = np.stack([stream.k(l, gids) for l in range(wl.layers)])
        V = np.stack([stream.v(l, gids) for l in range(wl.layers)])
        cache.append(-1, bits_to_dev(K), bits_to_dev(V), torch.from_numpy(types).cuda(),
                     torch.from_numpy(np.ascontiguousarray(pos)).cuda())
        ref.append(K, V, types, pos)

    for _ in range(8):                      # past the point where both windows are full
        append(*stream.next_chunk())
        cache.evict()
        ref.evict()
    for call in range(2):                   # two calls in a row share the library's scratch array
        gids, types, pos = stream.next_decode_token()
        append(gids, types, pos)
        layer = call % wl.layers
        Q = bits_to_dev(stream.q(layer, gids))
        qp = torch.from_numpy(np.ascontiguousarray(pos)).cuda()
        want = dev_to_f64(cache.attend(layer, Q, qp))
        out = torch.full_like(Q, float("nan"))
        got = dev_to_f64(cache.attend_decode_noalloc(layer, Q, qp, out))
        assert cache.status() == binding.OK
        assert np.isfinite(got).all()
        err = np.abs(got - want)
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (call, err.max(), err.mean())
        assert np.abs(want).max() > 0
        # and against the CPU checker directly, in the band the other decode tests use
        exact = ref.attend(layer, stream.q(layer, gids), pos)
        err = np.abs(got - exact)
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (call, err.max(), err.mean())


def _scratch_need(layers, kv_heads, head_dim, splits):
    """Bytes of the library's fixed array a call needs: one 4-byte arrival counter per (layer, KV head), rounded up
    to 16 bytes, then per (KV head, split) one record of 8 x head_dim bf16 partial outputs + 8 maxima + 8 sums."""
    up4 = lambda x: (x + 3) // 4 * 4  # noqa: E731
    return up4(layers * kv_heads) * 4 + kv_heads * splits * (16 * head_dim + 64)


def test_noalloc_limit_both_sides():
    """The largest problem that fits the fixed array runs and agrees with the regular entry point; problems
    beyond it are refused with SVLM_ERR_TOO_LARGE before anything is launched."""
    from harness import MAX_ABS, dev_to_f64
    from paper_2510_09608_b200 import binding
    limit = binding.NOALLOC_SCRATCH_BYTES
    # with more KV heads than SMs every KV head gets a single split
    fits = max(h for h in range(149, 400) if _scratch_need(1, h, 128, 1) <= limit)
    assert _scratch_need(1, fits + 1, 128, 1) > limit
    g = torch.Generator(device="cuda").manual_seed(7)
    rnd = lambda *shape: torch.randn(*shape, generator=g, device="cuda").to(torch.bfloat16)  # noqa: E731
    for kv_heads, ok in ((fits, True), (fits + 1, False), (2 * fits, False)):
        cache = binding.Cache(1, kv_heads, 128, 4, 64, 32, 256)
        n = 150
        cache.append(0, rnd(n, kv_heads, 128), rnd(n, kv_heads, 128), torch.zeros(n, dtype=torch.uint8, device="cuda"),
                     torch.arange(n, dtype=torch.int32, device="cuda"))
        Q, qp = rnd(1, kv_heads, 128), torch.full((1,), n - 1, dtype=torch.int32, device="cuda")
        if ok:
            want = dev_to_f64(cache.attend(0, Q, qp))
            got = dev_to_f64(cache.attend_decode_noalloc(0, Q, qp))
            assert cache.status() == binding.OK
            assert np.abs(got - want).max() <= MAX_ABS and np.abs(want).max() > 0
        else:
            with pytest.raises(binding.SvlmError) as e:
                cache.attend_decode_noalloc(0, Q, qp)
            assert e.value.status == binding.ERR_TOO_LARGE
        cache.close()


def test_noalloc_between_fused_decode_steps_changes_nothing():
    """The no-allocation call enqueued between two layers' fused decode steps: the steps must give what they give
    without it (the regular entry points start reading a layer's pages early only behind a decode of another layer of
    the same cache, and the no-allocation call is not one of those)."""
    from harness import bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding, streamgen as sg

    wl = dataclasses.replace(sg.workloads()[2], layers=3, n_sink=40, vision_window=5 * 128, text_window=70,
                             frames=2, grid_h=8, grid_w=8, text_max=24)

    def run(interleave):
        stream = sg.Stream(wl, 0)
        cache = binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
        cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
        for _ in range(6):
            gids, types, pos = stream.next_chunk()
            K = np.stack([stream.k(l, gids) for l in range(wl.layers)])
            V = np.stack([stream.v(l, gids) for l in range(wl.layers)])
            cache.append(-1, bits_to_dev(K), bits_to_dev(V), torch.from_numpy(types).cuda(), torch.from_numpy(np.ascontiguousarray(pos)).cuda())
            cache.evict()
        outs = []
        for _ in range(2):
            gids, types, pos = stream.next_decode_token()
            ty, ps = torch.from_numpy(types).cuda(), torch.from_numpy(np.ascontiguousarray(pos)).cuda()
            for l in range(wl.layers):
                outs.append(dev_to_f64(cache.decode_step(l, bits_to_dev(stream.k(l, gids)), bits_to_dev(stream.v(l, gids)),
                                                         ty if l == 0 else None, ps, bits_to_dev(stream.q(l, gids)))))
                if interleave:      # attention of the same token over another layer, through the fixed scratch array
                    other = (l + 2) % wl.layers
                    if other < l:   # only layers whose K/V of this token are already in the cache
                        cache.attend_decode_noalloc(other, bits_to_dev(stream.q(other, gids)), ps)
        assert cache.status() == binding.OK
        cache.close()
        return outs

    plain, mixed = run(False), run(True)
    for a, b in zip(plain, mixed):
        assert np.array_equal(a, b)
