"""GPU parity: the CUDA library against the CPU checker, through the C ABI, on seeded streams."""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _wl(n):
    from paper_2510_09608_b200 import streamgen as sg
    return sg.workloads()[n]


def test_config1_every_output():
    """Workload 1: the whole 20-chunk stream; every kept index, position, key and output is compared."""
    from harness import SideBySide, assert_close
    wl = _wl(1)
    s = SideBySide(wl)
    worst = [0.0, 0.0]
    for chunk in range(wl.chunks):
        s.append_chunk()
        s.evict()
        n = s.check_metadata()
        assert n <= wl.retained
        s.check_kv(0)
        st = s.attend(0)
        assert_close(st)
        worst = [max(worst[0], st[0]), max(worst[1], st[1])]
        for d in range(wl.decode_steps):
            if d % 2:
                for st in s.decode_step_fused():      # append + attention in one launch
                    assert_close(st)
            else:
                s.append_decode_token()
                assert_close(s.attend(0))
        s.check_metadata()
        s.check_kv(0)
    print("config 1 worst max/mean abs error", worst)


@pytest.mark.parametrize("sink_any,contiguous", [(False, True), (True, True), (False, False)])
def test_scaled_mrope_stream_multi_layer(sink_any, contiguous):
    """A shrunk workload-2 shape (MRoPE, GQA 28/4, d=128, 3 layers) that crosses several pages,
    partial pages and a ragged tail; every chunk fully compared, per-layer and all-layer calls."""
    from harness import SideBySide, assert_close
    wl = dataclasses.replace(_wl(2), layers=3, n_sink=40, vision_window=3 * 128, text_window=70,
                             frames=2, grid_h=8, grid_w=8, text_max=24, decode_steps=3)
    s = SideBySide(wl, sink_any=sink_any, contiguous=contiguous)
    for chunk in range(12):
        s.append_chunk(per_layer_calls=(chunk % 2 == 1))
        s.evict()
        s.check_metadata()
        layer = chunk % 3
        s.check_kv(layer)
        assert_close(s.attend(layer, all_layers=(chunk % 3 == 0)))
        for d in range(wl.decode_steps):
            if (chunk + d) % 2:
                for st in s.decode_step_fused():
                    assert_close(st)
            else:
                s.append_decode_token()
                assert_close(s.attend((layer + 1) % 3))
        s.check_kv((layer + 2) % 3)
    s.evict()
    s.evict()      # a second evict with nothing new must change nothing
    s.check_metadata()
    s.check_kv(1)


def test_layer_sequential_appends_after_the_evict():
    """A decoder computes layer l's K/V only after layer l-1 has attended: the chunk's metadata and
    layer 0 go in first, the eviction runs, and layers 1.. are appended afterwards."""
    from harness import SideBySide, assert_close
    wl = dataclasses.replace(_wl(2), layers=3, n_sink=20, vision_window=256, text_window=40,
                             frames=2, grid_h=8, grid_w=8, text_max=24, decode_steps=2)
    s = SideBySide(wl)
    for chunk in range(8):
        s.append_chunk_first_layer()
        s.evict()
        s.check_metadata()
        assert_close(s.attend(0))
        for l in (1, 2):
            s.append_later_layer(l)
            assert_close(s.attend(l))
        s.check_kv(chunk % 3)
        for _ in range(wl.decode_steps):
            for st in s.decode_step_fused():
                assert_close(st)
        s.check_kv((chunk + 1) % 3)


@pytest.mark.parametrize("S,Vw,Tw", [(0, 64, 16), (8, 0, 16), (8, 64, 0), (0, 0, 0), (300, 64, 16)])
def test_degenerate_policies(S, Vw, Tw):
    """Window and sink sizes of zero (the paper's ablation grid has 0-sized sinks and windows), and
    sinks spanning several pages."""
    from harness import SideBySide, assert_close
    wl = dataclasses.replace(_wl(1), n_sink=S, vision_window=Vw, text_window=Tw, text_max=30)
    s = SideBySide(wl, capacity=512)
    for chunk in range(14):
        s.append_chunk()
        s.evict()
        s.check_metadata()
        s.check_kv(0)
        st = s.attend(0)
        assert_close(st)
        s.append_decode_token()
        assert_close(s.attend(0))


def test_eight_query_heads_per_kv_head_and_all_layers_decode():
    """The widest group the tensor-core decode kernel packs (8 query heads per KV head), through single-layer,
    fused and all-layers (one launch, one CTA streaming many sub-tiles) decode calls."""
    from harness import SideBySide, assert_close
    wl = dataclasses.replace(_wl(2), layers=3, q_heads=16, kv_heads=2, n_sink=24, vision_window=5 * 128, text_window=90,
                             frames=2, grid_h=8, grid_w=8, text_max=24, decode_steps=3)
    s = SideBySide(wl)
    for chunk in range(9):
        s.append_chunk()
        s.evict()
        s.check_metadata()
        assert_close(s.attend(chunk % 3))
        for st in s.decode_step_fused():
            assert_close(st)
        s.append_decode_token()
        assert_close(s.attend(1))
        assert_close(s.attend(2, all_layers=True))


def test_fused_decode_step_all_layers_in_one_launch():
    """svlm_decode_step with layer -1: one token's append and attention for all layers at once."""
    from harness import SideBySide, assert_close, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding
    wl = dataclasses.replace(_wl(2), layers=3, n_sink=16, vision_window=256, text_window=32, frames=1, grid_h=8, grid_w=8)
    s = SideBySide(wl)
    for _ in range(4):
        s.append_chunk()
        s.evict()
    for step in range(3):
        gids, types, pos = s.stream.next_decode_token()
        K = np.stack([s.stream.k(l, gids)[0] for l in range(wl.layers)])
        V = np.stack([s.stream.v(l, gids)[0] for l in range(wl.layers)])
        Q = np.stack([s.stream.q(l, gids)[0] for l in range(wl.layers)])
        out = dev_to_f64(s.cache.decode_step(-1, bits_to_dev(K), bits_to_dev(V), torch.from_numpy(types).cuda(),
                                             torch.from_numpy(np.ascontiguousarray(pos)).cuda(), bits_to_dev(Q)))
        assert s.cache.status() == binding.OK
        s.ref.append(None, None, types, pos)
        s.last = (gids, types, pos)
        for l in range(wl.layers):
            s._give_values_to_ref(l)
            assert_close(s._stats(out[l][None], s.ref.attend(l, Q[l][None], pos)))
    s.check_metadata()
    for l in range(wl.layers):
        s.check_kv(l)


def test_batched_streams_match_single_calls():
    from harness import SideBySide, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding
    wl = dataclasses.replace(_wl(2), n_sink=16, vision_window=256, text_window=32, frames=1, grid_h=8, grid_w=8)
    sides = [SideBySide(wl, stream=i) for i in range(3)]
    for s in sides:
        for _ in range(4 + sides.index(s)):
            s.append_chunk()
            s.evict()
        s.append_decode_token()
    Q = np.stack([s.stream.q(0, s.last[0]) for s in sides])
    qpos = torch.from_numpy(np.stack([s.last[2] for s in sides])).cuda()
    out = dev_to_f64(binding.attend_batched([s.cache for s in sides], 0, bits_to_dev(Q), qpos))
    for i, s in enumerate(sides):
        s._give_values_to_ref(0)
        want = s.ref.attend(0, Q[i], s.last[2])
        err = np.abs(out[i] - want)
        assert err.max() <= 1e-2 and err.mean() <= 1e-3


@pytest.mark.parametrize("rope_1d", [False, True])
def test_batched_decode_steps_and_batched_evict(rope_1d):
    """Three streams at different fill levels advance in lock step through svlm_decode_step_batched (two layers,
    one launch per layer for all streams) with svlm_cache_evict_batched every four tokens: outputs of every
    stream, layer and step against the checker, metadata bit-exact after every eviction, stored K/V at the end."""
    from harness import SideBySide, assert_close, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding
    wl = dataclasses.replace(_wl(2), layers=2, n_sink=16, vision_window=256, text_window=24, frames=1, grid_h=8, grid_w=8)
    if rope_1d:
        wl = dataclasses.replace(_wl(1), layers=2, q_heads=8, kv_heads=2)
    sides = [SideBySide(wl, stream=i) for i in range(3)]
    for i, s in enumerate(sides):
        for _ in range(3 + 2 * i):
            s.append_chunk()
            s.evict()
    caches = [s.cache for s in sides]
    for step in range(10):
        toks = [s.stream.next_decode_token() for s in sides]
        ty = torch.from_numpy(np.concatenate([t[1] for t in toks])).cuda()
        ps = torch.from_numpy(np.ascontiguousarray(np.stack([t[2][0] for t in toks]))).cuda()
        outs, Qs = [], []
        for l in range(wl.layers):
            K = np.stack([s.stream.k(l, t[0])[0] for s, t in zip(sides, toks)])
            V = np.stack([s.stream.v(l, t[0])[0] for s, t in zip(sides, toks)])
            Qs.append(np.stack([s.stream.q(l, t[0])[0] for s, t in zip(sides, toks)]))
            outs.append(dev_to_f64(binding.decode_step_batched(caches, l, bits_to_dev(K), bits_to_dev(V),
                                                               ty if l == 0 else None, ps, bits_to_dev(Qs[-1]))))
        for i, (s, t) in enumerate(zip(sides, toks)):
            assert s.cache.status() == binding.OK
            s.ref.append(None, None, t[1], t[2])
            s.last = t
            for l in range(wl.layers):
                s._give_values_to_ref(l)
                assert_close(s._stats(outs[l][i][None], s.ref.attend(l, Qs[l][i][None], t[2])))
        if step % 4 == 3:
            binding.evict_batched(caches)
            for s in sides:
                s.rot.evict(s.ref)
                s.check_metadata()
    for s in sides:
        s.check_metadata()
        for l in range(wl.layers):
            s.check_kv(l)
    with pytest.raises(binding.SvlmError) as e:          # a cache may appear only once in a batch
        binding.evict_batched([caches[0], caches[0]])
    assert e.value.status == binding.ERR_ARG
    side = torch.cuda.Stream()
    caches[1].set_stream(side)                           # caches of a batch must sit on one stream
    with pytest.raises(binding.SvlmError) as e:
        binding.evict_batched(caches)
    assert e.value.status == binding.ERR_ARG
    caches[1].set_stream(torch.cuda.current_stream())


def test_batched_chunk_prefill_with_chunks_of_different_lengths():
    """svlm_attend_batched_varlen: four streams whose new chunks differ in length (one contributes a single row)
    attend in one launch per layer; every output row of every stream against the checker."""
    from harness import SideBySide, assert_close, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding
    wl = dataclasses.replace(_wl(2), layers=2, n_sink=16, vision_window=320, text_window=40, frames=1, grid_h=8, grid_w=8)
    sides = [SideBySide(wl, stream=i) for i in range(4)]
    for i, s in enumerate(sides):
        for _ in range(2 + 2 * i):
            s.append_chunk()
            s.evict()
        s.append_chunk()
        s.evict()
    sides[3].append_decode_token()                       # this stream attends with one row only
    n_q = [len(s.last[0]) for s in sides]
    assert len(set(n_q)) > 2 and n_q[3] == 1
    pos = torch.from_numpy(np.ascontiguousarray(np.concatenate([s.last[2] for s in sides]))).cuda()
    for l in range(wl.layers):
        Q = np.concatenate([s.stream.q(l, s.last[0]) for s in sides])
        out = dev_to_f64(binding.attend_batched_varlen([s.cache for s in sides], l, bits_to_dev(Q), pos, n_q))
        o = 0
        for s, n in zip(sides, n_q):
            assert s.cache.status() == binding.OK
            s._give_values_to_ref(l)
            assert_close(s._stats(out[o:o + n], s.ref.attend(l, Q[o:o + n], s.last[2])))
            o += n
    with pytest.raises(binding.SvlmError) as e:
        binding.attend_batched_varlen([s.cache for s in sides], 0, bits_to_dev(Q), pos, [n_q[0], n_q[1], n_q[2], 0])
    assert e.value.status == binding.ERR_ARG


@pytest.mark.parametrize("sink_any", [False, True])
def test_one_token_appends_equal_bulk_appends(sink_any):
    """The single-token append (its own short kernel path, which edits the list of active pages) against the
    general append of the same tokens in one call and against the checker: mixed types, sinks filling up, pages
    opening in the sink area and in both rings, evictions in between; metadata bit-exact at every check."""
    import oracle
    from paper_2510_09608_b200 import binding
    rng = np.random.default_rng(7 + sink_any)
    args = (1, 1, 64, 150, 200, 140, 1024)       # layers, kv heads, d, sinks, vision window, text window, capacity
    one, bulk = binding.Cache(*args), binding.Cache(*args)
    ref = oracle.Oracle(1, 1, 64, 150, 200, 140, sink_any_type=sink_any)
    for c in (one, bulk):
        c.set_policy(sink_any, True)
    z = lambda n: torch.zeros(n, 1, 64, dtype=torch.bfloat16, device="cuda")  # noqa: E731
    nxt = 0
    for rnd in range(12):
        n = int(rng.integers(40, 300))
        types = (rng.random(n) < (0.7 if rnd % 3 else 0.2)).astype(np.uint8)        # mostly vision, sometimes mostly text
        pos = np.arange(nxt, nxt + n, dtype=np.int32)
        nxt += n
        ty, ps = torch.from_numpy(types).cuda(), torch.from_numpy(pos).cuda()
        bulk.append(0, z(n), z(n), ty, ps)
        for i in range(n):
            one.append(0, z(1), z(1), ty[i:i + 1], ps[i:i + 1])
        ref.append(None, None, types, pos)
        for check in (False, True):
            a, b, w = one.query(), bulk.query(), ref.query()
            assert one.status() == binding.OK and bulk.status() == binding.OK
            for k in ("gids", "types", "pos"):
                assert np.array_equal(a[k], b[k]) and np.array_equal(a[k], w[k]), (rnd, check, k)
            assert a["shift_total"] == b["shift_total"] == w["shift_total"]
            if not check:
                one.evict(); bulk.evict(); ref.evict()
    # a single-token append beyond the capacity is dropped on the device and reported
    small = binding.Cache(1, 1, 64, 4, 8, 8, 16)
    for i in range(17):
        small.append(0, z(1), z(1), torch.zeros(1, dtype=torch.uint8, device="cuda"), torch.full((1,), i, dtype=torch.int32, device="cuda"))
        assert small.status() == (binding.OK if i < 16 else binding.ERR_CAPACITY)
    assert len(small.query()["gids"]) == 16


def test_host_buffer_entry_points_equal_the_device_ones():
    """svlm_cache_append_host / svlm_attend_host (pinned host buffers, all layers per call; the chunk prefill runs as a
    copy/attend pipeline over the layers) against the device-pointer calls on a twin cache: same bits out."""
    from harness import bits_to_dev
    from paper_2510_09608_b200 import binding, streamgen as sg
    wl = dataclasses.replace(_wl(2), layers=3, n_sink=16, vision_window=256, text_window=32, frames=2, grid_h=8, grid_w=8)
    stream = sg.Stream(wl, 0)
    mk = lambda: binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)  # noqa: E731
    dev, host = mk(), mk()
    for c in (dev, host):
        c.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()  # noqa: E731
    for step in range(4):
        for gids, types, pos in [stream.next_chunk()] + [stream.next_decode_token() for _ in range(2)]:
            K = np.stack([stream.k(l, gids) for l in range(wl.layers)])
            V = np.stack([stream.v(l, gids) for l in range(wl.layers)])
            Q = np.stack([stream.q(l, gids) for l in range(wl.layers)])
            ty, ps = torch.from_numpy(types), torch.from_numpy(np.ascontiguousarray(pos))
            got = torch.empty(Q.shape, dtype=torch.int16).pin_memory()
            if len(gids) > 1:
                dev.append(-1, bits_to_dev(K), bits_to_dev(V), ty.cuda(), ps.cuda())
                host.append_host(-1, pin(K.view(np.int16)), pin(V.view(np.int16)), ty.pin_memory(), ps.pin_memory())
                dev.evict()
                host.evict()
                want = dev.attend(-1, bits_to_dev(Q), ps.cuda())
                host.attend_host(-1, pin(Q.view(np.int16)), ps.pin_memory(), got)
            else:       # a generated token: the fused step, device pointers against host buffers
                want = dev.decode_step(-1, bits_to_dev(K[:, 0]), bits_to_dev(V[:, 0]), ty.cuda(), ps.cuda(), bits_to_dev(Q[:, 0]))[:, None]
                host.decode_step_host(-1, pin(K.view(np.int16)), pin(V.view(np.int16)), ty.pin_memory(), ps.pin_memory(),
                                      pin(Q.view(np.int16)), got)
            assert host.status() == binding.OK
            assert np.array_equal(got.numpy().view(np.uint16), want.view(torch.int16).cpu().numpy().view(np.uint16)), step
        # a generated token layer by layer: pinned buffers (the kernels read them in place) and, every other step,
        # pageable ones (staged through device memory) against the device-pointer calls
        gids, types, pos = stream.next_decode_token()
        ty, ps = torch.from_numpy(types), torch.from_numpy(np.ascontiguousarray(pos))
        for l in range(wl.layers):
            K, V, Q = stream.k(l, gids), stream.v(l, gids), stream.q(l, gids)
            want = dev.decode_step(l, bits_to_dev(K), bits_to_dev(V), ty.cuda() if l == 0 else None, ps.cuda(), bits_to_dev(Q))
            if step % 2:
                got = np.zeros(Q.shape, dtype=np.uint16)
                host.decode_step_host(l, np.ascontiguousarray(K), np.ascontiguousarray(V), types if l == 0 else None,
                                      np.ascontiguousarray(pos), np.ascontiguousarray(Q), got)
            else:
                got_t = torch.zeros(Q.shape, dtype=torch.int16).pin_memory()
                host.decode_step_host(l, pin(K.view(np.int16)), pin(V.view(np.int16)), ty.pin_memory() if l == 0 else None,
                                      ps.pin_memory(), pin(Q.view(np.int16)), got_t)
                got = got_t.numpy().view(np.uint16)
            assert host.status() == binding.OK
            assert np.array_equal(got, want.view(torch.int16).cpu().numpy().view(np.uint16)), (step, l)
    a, b = dev.query(), host.query()
    assert np.array_equal(a["gids"], b["gids"]) and np.array_equal(a["pos"], b["pos"])


def test_errors_and_capacity():
    from paper_2510_09608_b200 import binding
    with pytest.raises(binding.SvlmError):
        binding.Cache(1, 1, 96, 4, 8, 8, 64)          # head_dim must be 64 or 128
    c = binding.Cache(1, 1, 64, 4, 8, 8, 64)
    K = torch.zeros(40, 1, 64, dtype=torch.bfloat16, device="cuda")
    ty = torch.zeros(40, dtype=torch.uint8, device="cuda")
    pos = torch.arange(40, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.SvlmError) as e:
        c.attend(0, K[:1], pos[:1])
    assert e.value.status == binding.ERR_ORDER           # nothing appended yet
    c.append(0, K, K, ty, pos)
    c2 = binding.Cache(1, 2, 64, 4, 8, 8, 64)
    c2.append(0, torch.zeros(4, 2, 64, dtype=torch.bfloat16, device="cuda"),
              torch.zeros(4, 2, 64, dtype=torch.bfloat16, device="cuda"), ty[:4], pos[:4])
    with pytest.raises(binding.SvlmError) as e:          # 3 query heads over 2 kv heads
        c2.attend(0, torch.zeros(1, 3, 64, dtype=torch.bfloat16, device="cuda"), pos[:1])
    assert e.value.status == binding.ERR_ARG
    assert c.status() == binding.OK
    before = c.query()
    c.append(0, K, K, ty, pos + 40)                       # 80 > capacity 64: dropped on the device
    assert c.status() == binding.ERR_CAPACITY
    after = c.query()
    assert np.array_equal(before["gids"], after["gids"])
    with pytest.raises(binding.SvlmError) as e:
        c.append(0, torch.zeros(100, 1, 64, dtype=torch.bfloat16, device="cuda"),
                 torch.zeros(100, 1, 64, dtype=torch.bfloat16, device="cuda"),
                 torch.zeros(100, dtype=torch.uint8, device="cuda"), torch.arange(100, dtype=torch.int32, device="cuda"))
    assert e.value.status == binding.ERR_CAPACITY


@pytest.mark.parametrize("contiguous", [True, False])
def test_mrope_vision_window_that_cuts_a_block(contiguous):
    """A vision window that is not a whole number of blocks: each chunk is one 2x8x8 block of 128 tokens and
    the window holds 200, so the oldest retained block is always partly evicted.  The rule is applied
    literally: a kept token moves left by the cursor advances of the evicted tokens before it, whatever
    block they belong to, so a partly evicted block keeps its internal offsets."""
    from harness import SideBySide, assert_close
    wl = dataclasses.replace(_wl(2), layers=2, n_sink=24, vision_window=200, text_window=50,
                             frames=2, grid_h=8, grid_w=8, text_max=24, decode_steps=2)
    s = SideBySide(wl, contiguous=contiguous)
    for chunk in range(10):
        s.append_chunk(per_layer_calls=(chunk % 2 == 0))
        s.evict()
        n = s.check_metadata()
        if chunk >= 2:
            q = s.ref.query()
            assert int((q["types"] == 1).sum()) == 200 and n == len(q["gids"])
        s.check_kv(chunk % 2)
        assert_close(s.attend(chunk % 2))
        for _ in range(wl.decode_steps):
            for st in s.decode_step_fused():
                assert_close(st)
    s.check_kv(0)
    s.check_kv(1)


@pytest.mark.parametrize("d,hq,hkv", [(128, 28, 2), (64, 12, 1)])
def test_wide_gqa_group_decode_takes_the_general_kernel(d, hq, hkv):
    """More than 8 query heads per KV head at n_q = 1 is outside the split-KV decode kernel: svlm_attend then runs
    the general row-at-a-time kernel, and the fused decode step refuses the shape."""
    from harness import SideBySide, assert_close, bits_to_dev
    from paper_2510_09608_b200 import binding
    base = _wl(2) if d == 128 else _wl(1)
    wl = dataclasses.replace(base, layers=2, q_heads=hq, kv_heads=hkv, n_sink=10, vision_window=3 * 64, text_window=40,
                             frames=1, grid_h=8, grid_w=8, text_max=12, decode_steps=2, head_dim=d)
    s = SideBySide(wl)
    for chunk in range(6):
        s.append_chunk()
        s.evict()
        s.check_metadata()
        assert_close(s.attend(chunk % 2))                   # chunk prefill: the tensor-core kernel takes any group
        for _ in range(wl.decode_steps):
            s.append_decode_token()
            assert_close(s.attend(chunk % 2))               # n_q = 1, group 14 / 12: general kernel
            assert_close(s.attend(0, all_layers=True))
    gids, types, pos = s.stream.next_decode_token()
    with pytest.raises(binding.SvlmError) as e:
        s.cache.decode_step(0, bits_to_dev(s.stream.k(0, gids)), bits_to_dev(s.stream.v(0, gids)),
                            torch.from_numpy(types).cuda(), torch.from_numpy(np.ascontiguousarray(pos)).cuda(),
                            bits_to_dev(s.stream.q(0, gids)))
    assert e.value.status == binding.ERR_ARG
    s.check_metadata()                                       # the refused call changed nothing


def test_cache_with_more_pages_than_the_fast_kernels_list():
    """A capacity beyond 512 pages (no-eviction or full-attention style use): one-token attention over all of
    it must not stop at the 512th page.  svlm_attend takes the general kernel for both shapes; the fused decode
    step and the no-allocation entry point refuse."""
    from harness import SideBySide, assert_close, bits_to_dev
    from paper_2510_09608_b200 import binding
    n_chunk = 4 * 32 * 32                                    # 4096 vision tokens per chunk
    wl = dataclasses.replace(_wl(1), layers=1, q_heads=2, kv_heads=1, n_sink=0, vision_window=1 << 20, text_window=1 << 20,
                             frames=4, grid_h=32, grid_w=32, text_max=8, decode_steps=1)
    s = SideBySide(wl, capacity=66 * 1024 + 512)
    for chunk in range(16):                                  # 65.5k vision tokens + text: 513+ pages in use
        s.append_chunk()
    s.evict()
    n = s.check_metadata()
    assert n > 512 * 128
    rows = np.array([0, n_chunk // 2, len(s.last[0]) - 1])
    assert_close(s.attend(0, rows=rows))                     # n_q >= 2 over more than 512 pages
    s.append_decode_token()
    assert_close(s.attend(0))                                # n_q = 1 over more than 512 pages
    gids, types, pos = s.stream.next_decode_token()
    args = (bits_to_dev(s.stream.k(0, gids)), bits_to_dev(s.stream.v(0, gids)), torch.from_numpy(types).cuda(),
            torch.from_numpy(np.ascontiguousarray(pos)).cuda(), bits_to_dev(s.stream.q(0, gids)))
    with pytest.raises(binding.SvlmError) as e:
        s.cache.decode_step(0, *args)
    assert e.value.status == binding.ERR_ARG
    with pytest.raises(binding.SvlmError) as e:
        s.cache.attend_decode_noalloc(0, args[4], args[3])
    assert e.value.status == binding.ERR_TOO_LARGE
    s.check_metadata()


@pytest.mark.parametrize("d", [64, 128])
def test_per_layer_decode_with_several_rounds_per_cta(d):
    """A cache large enough, over few enough CTAs, that a CTA of the per-layer decode kernel holds more 16-key units
    than its six warps take in one round (8 KV heads: 18 CTAs per head; more than 40 pages in use): the second round
    reuses the warps' slots and carries the running maximum.  Plain and fused decode steps of every layer."""
    from harness import SideBySide, assert_close
    base = _wl(2) if d == 128 else _wl(1)
    wl = dataclasses.replace(base, layers=2, q_heads=16, kv_heads=8, head_dim=d, n_sink=100, vision_window=6 * 1024, text_window=300,
                             frames=4, grid_h=16, grid_w=16, text_max=24, decode_steps=2)
    s = SideBySide(wl)
    for chunk in range(8):
        s.append_chunk()
        s.evict()
    n = s.check_metadata()
    assert n > 48 * 128          # 8 units per page over 18 CTAs: more than the 18 units of one round
    for step in range(3):
        if step % 2:
            for st in s.decode_step_fused():
                assert_close(st)
        else:
            s.append_decode_token()
            assert_close(s.attend(0))
            assert_close(s.attend(1))
    s.check_kv(1)


@pytest.mark.parametrize("d", [64, 128])
def test_per_layer_decode_many_launches_in_a_row(d):
    """The per-layer decode kernel hands its splits' partial results over in words that carry the launch's tag (the KV
    head's epoch + 1) and a launch trusts a word by its tag alone: several hundred launches on one cache, every one with
    another query and a few of them replayed from a CUDA graph (where nothing on the host changes between launches), must
    each give that query's result, never a word left by an earlier launch."""
    from harness import SideBySide, assert_close, bits_to_dev, dev_to_f64
    base = _wl(2) if d == 128 else _wl(1)
    wl = dataclasses.replace(base, layers=2, q_heads=8, kv_heads=2, head_dim=d, n_sink=16, vision_window=5 * 128, text_window=100,
                             frames=1, grid_h=8, grid_w=8, text_max=12, decode_steps=1)
    s = SideBySide(wl)
    for _ in range(6):
        s.append_chunk()
        s.evict()
    s.append_decode_token()
    gids, _, pos = s.last
    qp = torch.from_numpy(np.ascontiguousarray(pos)).cuda()
    rng = np.random.default_rng(11)
    for l in range(wl.layers):
        s._give_values_to_ref(l)
    from oracle import qkv
    Qs = [qkv.to_bf16_bits(rng.standard_normal((1, wl.q_heads, d))) for _ in range(6)]
    Qd = [bits_to_dev(q) for q in Qs]
    want = [[s.ref.attend(l, Qs[i], pos) for i in range(len(Qs))] for l in range(wl.layers)]
    for it in range(240):
        i, l = it % len(Qs), (it // 7) % wl.layers
        out = s.cache.attend(l, Qd[i], qp)
        if it % 17 == 0 or it >= 236:
            assert_close(s._stats(dev_to_f64(out), want[l][i]))
    # the same from a graph: six launches per replay, replayed five times, outputs in fixed buffers
    outs = [torch.empty_like(Qd[0]) for _ in Qd]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        s.cache.set_stream(side)
        for i in range(len(Qd)):
            s.cache.attend(i % wl.layers, Qd[i], qp, out=outs[i])      # warm-up outside the capture
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for i in range(len(Qd)):
                s.cache.attend(i % wl.layers, Qd[i], qp, out=outs[i])
        for _ in range(5):
            for o in outs:
                o.zero_()
            g.replay()
            side.synchronize()
            for i in range(len(Qd)):
                assert_close(s._stats(dev_to_f64(outs[i]), want[i % wl.layers][i]))
    torch.cuda.current_stream().wait_stream(side)
    s.cache.set_stream(torch.cuda.current_stream())
    assert s.cache.status() == 0
