"""The give-up paths of the kernels' bounded waits, walked without anything hanging.

Every device-side wait in the library is bounded by a poll limit that lives in the cache's control block.  With the
limit at 0 every wait gives up at once: the kernels must then record SVLM_ERR_TIMEOUT, release what they hold (shared
memory copies in flight, tensor memory, cluster barriers) and return by themselves; nothing may trap, fault or spin.
Afterwards, with the limit restored, the same caches must compute correctly again (only the sticky status remembers)
and so must a fresh cache.
"""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _small(d128=True, layers=1):
    from paper_2510_09608_b200 import streamgen as sg
    base = sg.workloads()[2] if d128 else sg.workloads()[1]
    return dataclasses.replace(base, layers=layers, n_sink=16, vision_window=3 * 64, text_window=40, frames=1, grid_h=8, grid_w=8,
                               text_max=12, decode_steps=1)


def _filled(wl, stream_id=0, chunks=5):
    from harness import SideBySide
    s = SideBySide(wl, stream=stream_id)
    for _ in range(chunks):
        s.append_chunk()
        s.evict()
    return s


@pytest.mark.parametrize("d128", [True, False])
def test_chunk_prefill_gives_up_and_recovers(d128):
    from harness import assert_close, bits_to_dev
    from paper_2510_09608_b200 import binding
    wl = _small(d128)
    s = _filled(wl)
    s.append_chunk()
    gids, _, pos = s.last
    Q = bits_to_dev(s.stream.q(0, gids))
    qp = torch.from_numpy(np.ascontiguousarray(pos)).cuda()
    s.cache.debug_set_wait_limit(0)
    s.cache.attend(0, Q, qp)                              # tcgen05 kernel: every CTA gives up, frees TMEM, meets its partner
    assert s.cache.status() == binding.ERR_TIMEOUT
    s.cache.debug_set_wait_limit(1 << 20)
    from harness import dev_to_f64                        # (the harness's own attend insists on an OK status: compare by hand)
    out = dev_to_f64(s.cache.attend(0, Q, qp))
    s._give_values_to_ref(0)
    assert_close(s._stats(out, s.ref.attend(0, s.stream.q(0, gids), pos)))
    assert s.cache.status() == binding.ERR_TIMEOUT        # sticky
    fresh = _filled(wl, stream_id=1, chunks=3)            # and a new cache is untouched by all this
    fresh.append_chunk()
    assert_close(fresh.attend(0))
    assert fresh.cache.status() == binding.OK


def test_batched_decode_gives_up_counter_returns_to_zero():
    """The streaming split-KV kernel (several caches per launch): CTAs that give up still count themselves as
    arrived, so the arrival counters are back at zero and the next launch combines correctly."""
    from harness import assert_close, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding
    wl = _small(True)
    sides = [_filled(wl, stream_id=i) for i in range(2)]
    for s in sides:
        s.append_decode_token()
    caches = [s.cache for s in sides]
    Q = bits_to_dev(np.stack([s.stream.q(0, s.last[0]) for s in sides]))
    qp = torch.from_numpy(np.ascontiguousarray(np.stack([s.last[2] for s in sides]))).cuda()
    for c in caches:
        c.debug_set_wait_limit(0)
    binding.attend_batched(caches, 0, Q, qp)
    for c in caches:
        assert c.status() == binding.ERR_TIMEOUT
        c.debug_set_wait_limit(1 << 20)
    for _ in range(2):                                    # twice: the second launch starts from what the first left
        out = dev_to_f64(binding.attend_batched(caches, 0, Q, qp))
        for i, s in enumerate(sides):
            s._give_values_to_ref(0)
            assert_close(s._stats(out[i], s.ref.attend(0, s.stream.q(0, s.last[0]), s.last[2])))


def test_layer_decode_combiners_give_up_and_the_next_launch_is_right():
    """The per-layer split-KV kernel (one cache, one layer): its copies are cp.async and cannot time out, but the first
    splits of a KV head combine all the splits' records and read a record's words again until they carry the launch's
    tag.  With the limit at 0 they give up before a first try: time-out recorded, their shares of the output
    undefined; the KV head's epoch moves on all the same, so that with the limit restored the next launches look for
    fresh tags and combine correctly."""
    from harness import assert_close, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding
    wl = _small(True)
    one = _filled(wl, stream_id=5)
    one.append_decode_token()
    gids, _, pos = one.last
    Q = bits_to_dev(one.stream.q(0, gids))
    qp = torch.from_numpy(np.ascontiguousarray(pos)).cuda()
    one.cache.debug_set_wait_limit(0)
    for _ in range(3):
        one.cache.attend(0, Q, qp)
    assert one.cache.status() == binding.ERR_TIMEOUT
    one.cache.debug_set_wait_limit(1 << 20)
    one._give_values_to_ref(0)
    want = one.ref.attend(0, one.stream.q(0, gids), pos)
    for _ in range(2):
        assert_close(one._stats(dev_to_f64(one.cache.attend(0, Q, qp)), want))
    assert one.cache.status() == binding.ERR_TIMEOUT        # sticky


def test_projection_gives_up_and_recovers():
    from harness import bits_to_dev, dev_to_f64
    from oracle import qkv
    from paper_2510_09608_b200 import binding
    wl = _small(True)
    hidden = 256
    rng = np.random.default_rng(3)
    s = _filled(wl)
    gids, types, pos = s.stream.next_chunk()
    n = len(gids)
    X = qkv.to_bf16_bits(rng.standard_normal((n, hidden)))
    W = qkv.to_bf16_bits(rng.standard_normal(((wl.q_heads + 2 * wl.kv_heads) * wl.head_dim, hidden)) / np.sqrt(hidden))
    ty, ps = torch.from_numpy(types).cuda(), torch.from_numpy(np.ascontiguousarray(pos)).cuda()
    s.cache.debug_set_wait_limit(0)
    s.cache.qkv_append(0, bits_to_dev(X), bits_to_dev(W), wl.q_heads, ty, ps)
    assert s.cache.status() == binding.ERR_TIMEOUT
    s.ref.append(None, None, types, pos)
    got, want = s.cache.query(), s.ref.query()           # the metadata append itself stood
    assert np.array_equal(got["gids"], want["gids"]) and np.array_equal(got["pos"], want["pos"])
    # a fresh cache with the default limit: the same projection is right
    t = _filled(wl, stream_id=2)
    g2, ty2, p2 = t.stream.next_chunk()
    Qg = t.cache.qkv_append(0, bits_to_dev(X[:len(g2)]), bits_to_dev(W), wl.q_heads, torch.from_numpy(ty2).cuda(),
                            torch.from_numpy(np.ascontiguousarray(p2)).cuda())
    assert t.cache.status() == binding.OK
    Q64 = qkv.project(X[:len(g2)], W, wl.q_heads, wl.kv_heads, wl.head_dim)[0]
    assert np.all(np.abs(dev_to_f64(Qg) - Q64) <= 2.0 ** -8 * np.abs(Q64) + 1e-5 * np.sqrt(hidden))
