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
    from harness import MAX_ABS, MEAN_ABS, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding, streamgen as sg

    wl = dataclasses.replace(sg.workloads()[2], layers=2, n_sink=40, vision_window=5 * 128, text_window=70,
                             frames=2, grid_h=8, grid_w=8, text_max=24)
    stream = sg.Stream(wl, 0)
    cache = binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
    cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)

    def append(gids, types, pos):
        K = np.stack([stream.k(l, gids) for l in range(wl.layers)])
        V = np.stack([stream.v(l, gids) for l in range(wl.layers)])
        cache.append(-1, bits_to_dev(K), bits_to_dev(V), torch.from_numpy(types).cuda(),
                     torch.from_numpy(np.ascontiguousarray(pos)).cuda())

    for _ in range(8):                      # past the point where both windows are full
        append(*stream.next_chunk())
        cache.evict()
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


def test_noalloc_rejects_what_does_not_fit():
    from paper_2510_09608_b200 import binding
    # 256 KV heads x (8*128+16) floats of partial results do not fit the 1 MiB array
    cache = binding.Cache(1, 256, 128, 4, 64, 32, 128)
    K = torch.zeros(1, 256, 128, dtype=torch.bfloat16, device="cuda")
    cache.append(0, K, K, torch.zeros(1, dtype=torch.uint8, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda"))
    with pytest.raises(binding.SvlmError) as e:
        cache.attend_decode_noalloc(0, torch.zeros(1, 256, 128, dtype=torch.bfloat16, device="cuda"),
                                    torch.zeros(1, dtype=torch.int32, device="cuda"))
    assert e.value.status == binding.ERR_TOO_LARGE
