"""GPU parity at the full workload sizes, in the launch configuration the benchmark times.

The streams are too long to compare every value, so the CPU checker follows the *metadata* of every
token (cheap) and receives keys/values only for the layers that are compared; every input value is
regenerable from its coordinates.  Compared: kept ordinals, positions and total shift bit-exactly;
stored keys of sampled layers within the re-rotation rounding bound, values bit-exactly; attention
outputs of sampled query rows (the first, the last and a seeded random set) of sampled layers for the
chunk prefill, and every decode output of those layers, within the acceptance band.
"""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _setup(wl, stream_id=0):
    import oracle
    from paper_2510_09608_b200 import binding, streamgen as sg
    stream = sg.Stream(wl, stream_id)
    cache = binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
    cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
    ref = oracle.Oracle(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window,
                        rope_mode=wl.rope_mode, rope_base=wl.rope_base, sections=wl.sections)
    return stream, cache, ref


def _fill(cache, ref, wl, stream, rot):
    """Stream chunks (append + evict, decode tokens appended in bulk) through both sides until every window is
    full; the checker only follows the metadata."""
    from paper_2510_09608_b200 import streamgen as sg
    gen = lambda tensor, g: torch.stack(  # noqa: E731
        [sg.rows_bf16_torch(wl.seed, tensor, stream.stream, l, g, wl.kv_heads, wl.head_dim) for l in range(wl.layers)])
    n_text, chunks = 0, 0
    while n_text < wl.n_sink + wl.text_window + 64 or chunks * wl.vision_per_chunk < wl.vision_window + 1:
        gids, types, pos = stream.next_chunk()
        extra = [stream.next_decode_token() for _ in range(wl.decode_steps)]
        cache.append(-1, gen(sg.TENSOR_K, gids), gen(sg.TENSOR_V, gids), torch.from_numpy(types).cuda(),
                     torch.from_numpy(np.ascontiguousarray(pos)).cuda())
        cache.evict()
        ref.append(None, None, types, pos)
        rot.evict(ref)
        if extra:
            g = np.concatenate([e[0] for e in extra]); t = np.concatenate([e[1] for e in extra])
            p = np.concatenate([e[2] for e in extra])
            cache.append(-1, gen(sg.TENSOR_K, g), gen(sg.TENSOR_V, g), torch.from_numpy(t).cuda(),
                         torch.from_numpy(np.ascontiguousarray(p)).cuda())
            ref.append(None, None, t, p)
        n_text += int((types == sg.TEXT).sum()) + len(extra)
        chunks += 1


def _same_metadata(cache, ref):
    from paper_2510_09608_b200 import binding
    got, want = cache.query(), ref.query()
    assert cache.status() == binding.OK
    assert np.array_equal(got["gids"], want["gids"]), "kept set differs"
    assert np.array_equal(got["types"], want["types"])
    assert np.array_equal(got["pos"], want["pos"]), "positions differ"
    assert got["shift_total"] == want["shift_total"]


def _give(ref, stream, layer):
    gids = ref.query()["gids"]
    ref.set_kv(layer, gids, stream.k(layer, gids), stream.v(layer, gids))


def _give_new(ref, stream, layer, gids):
    """Values of freshly appended tokens only (the kept history already has them)."""
    ref.set_kv(layer, gids, stream.k(layer, gids), stream.v(layer, gids))


def _check_kv(cache, ref, stream, wl, layer, rot, one_evict_per_chunk=True):
    """Values bit-exact; every stored key within the rounding bound of ITS OWN history: the first rotation plus
    one re-rotation per eviction that moved the token (a vision token lives 16 chunks, so at most 17 roundings
    however long the stream; text-window tokens a few dozen; sinks only the first)."""
    from harness import key_rounding_bound
    from paper_2510_09608_b200 import streamgen as sg
    _give(ref, stream, layer)
    Kb, Vb = cache.read_kv(layer, ref.count())
    want_k, want_v = ref.rotated_k(layer), ref.values(layer)
    assert np.array_equal(sg.bf16_bits_to_f64(Vb), want_v), "values must be bit-exact"
    q = ref.query()
    roundings = 1 + rot.of(q["gids"])
    vis = q["types"] == sg.VISION
    if vis.any() and one_evict_per_chunk:
        assert roundings[vis].max() <= 1 + -(-wl.vision_window // wl.vision_per_chunk), "a vision key outlived its window"
    err = np.abs(sg.bf16_bits_to_f64(Kb) - want_k)
    over = err - key_rounding_bound(want_k, roundings)
    assert np.all(over <= 0), f"key error {err.max()} exceeds the token's rounding bound by {over.max()}"


def _close(got, want, what):
    from harness import MAX_ABS, MEAN_ABS, TIGHT_RMS_REL
    err = np.abs(got - want)
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, f"{what}: max {err.max()}, mean {err.mean()}"
    rms = np.sqrt((err ** 2).mean()) / max(np.sqrt((want ** 2).mean()), 1e-30)
    assert rms <= TIGHT_RMS_REL, f"{what}: rms error is {rms:.4f} of the rms signal"


def test_config3_full_stack_steady_state_step_as_benchmarked():
    """28 layers at the deployed policy (512 sinks / 8192 vision / 512 text), steady state, two steps run exactly
    as bench.py runs them: layer-sequential C-ABI calls replayed from a CUDA graph (append + evict + per-layer
    append/prefill + 16 fused decode steps per layer)."""
    import bench
    from harness import dev_to_f64
    from paper_2510_09608_b200 import streamgen as sg
    wl = sg.workloads()[3]
    from harness import RotationCounter
    stream, cache, ref = _setup(wl)
    rot = RotationCounter()
    _fill(cache, ref, wl, stream, rot)
    _same_metadata(cache, ref)
    layers = (0, 13, 27)
    rng = np.random.default_rng(wl.seed)
    for step in range(2):
        chunk, decode = bench.next_step_schedule(stream, wl)
        inp = bench.StepInputs(wl, stream, chunk, decode)
        if step == 0:      # one plain step on a scratch cache sets the kernels' one-time attributes outside the capture
            _, scratch, _ = _setup(wl)
            bench.run_step(scratch, wl, inp)
            torch.cuda.synchronize()
            scratch.close()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            cache.set_stream(torch.cuda.current_stream())
            bench.run_step(cache, wl, inp)
        cache.set_stream(torch.cuda.current_stream())
        g.replay()
        torch.cuda.synchronize()
        # the checker walks the same step and produces the expected values at each point
        gids, types, pos = chunk
        ref.append(None, None, types, pos)
        rot.evict(ref)
        rows = np.unique(np.concatenate([[0, len(gids) - 1], rng.integers(0, len(gids), 16)]))
        for l in layers:
            _give(ref, stream, l)
            want = ref.attend(l, stream.q(l, gids), pos, rows)
            _close(dev_to_f64(inp.out[l])[rows], want, f"step {step} prefill layer {l}")
        for d, (g1, t1, p1) in zip(inp.dec, decode):
            ref.append(None, None, t1, p1)
            for l in layers:
                _give_new(ref, stream, l, g1)
                _close(dev_to_f64(d["out"][l]), ref.attend(l, stream.q(l, g1), p1), f"step {step} decode layer {l}")
        _same_metadata(cache, ref)
    for l in layers:
        _check_kv(cache, ref, stream, wl, l, rot)


def test_config4_batched_decode_16_streams_with_interleaved_eviction():
    """16 independent streams at the full retained size, 48 batched q=1 steps (svlm_decode_step_batched), a batched
    eviction every 16 steps; every stream's output compared at sampled steps, metadata after every eviction."""
    from harness import RotationCounter, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding, streamgen as sg
    wl = dataclasses.replace(sg.workloads()[4], decode_steps=16)
    sides, rots = [], []
    for sid in range(wl.streams):
        stream, cache, ref = _setup(wl, sid)
        rots.append(RotationCounter())
        _fill(cache, ref, wl, stream, rots[-1])
        _give(ref, stream, 0)
        sides.append((stream, cache, ref))
    caches = [c for _, c, _ in sides]
    for step in range(48):
        toks = [s.next_decode_token() for s, _, _ in sides]
        for (s, c, r), (g1, t1, p1) in zip(sides, toks):
            r.append(None, None, t1, p1)
            _give_new(r, s, 0, g1)
        gen = lambda f: bits_to_dev(np.stack([f(s, g1)[0] for (s, _, _), (g1, _, _) in zip(sides, toks)]))  # noqa: E731
        Q = np.stack([s.q(0, g1) for (s, _, _), (g1, _, _) in zip(sides, toks)])
        ty = torch.from_numpy(np.concatenate([t1 for _, t1, _ in toks])).cuda()
        qpos = torch.from_numpy(np.ascontiguousarray(np.stack([p1[0] for _, _, p1 in toks]))).cuda()
        # as benchmarked: one fused step for all streams (metadata launch + attention launch)
        out = dev_to_f64(binding.decode_step_batched(caches, 0, gen(lambda s, g: s.k(0, g)), gen(lambda s, g: s.v(0, g)), ty,
                                                     qpos, bits_to_dev(Q[:, 0])))
        if step % 16 in (0, 15):
            for i, ((s, c, r), (g1, t1, p1)) in enumerate(zip(sides, toks)):
                _close(out[i][None], r.attend(0, Q[i], p1), f"stream {i} step {step}")
        if step % 16 == 15:
            binding.evict_batched(caches)
            for (s, c, r), rot in zip(sides, rots):
                rot.evict(r)
                _same_metadata(c, r)
    for (s, c, r), rot in list(zip(sides, rots))[::5]:
        _check_kv(c, r, s, wl, 0, rot, one_evict_per_chunk=False)


def test_config5_high_frame_rate_streams_sampled():
    """The 8 frames/s x 8x8-grid shape (vision blocks of span 8, text bursts up to 32): three of the eight streams,
    four of the 28 layers, one steady-state step run as benchmarked: the streams advance in lock step (per-stream
    appends, one batched eviction, one chunk-prefill launch per layer for all streams' different-length chunks, one
    batched decode launch per layer and token)."""
    import bench
    from harness import RotationCounter, dev_to_f64
    from paper_2510_09608_b200 import streamgen as sg
    wl = dataclasses.replace(sg.workloads()[5], layers=4)
    rng = np.random.default_rng(wl.seed)
    sides, rots = [], []
    for sid in (0, 3, 7):
        stream, cache, ref = _setup(wl, sid)
        rots.append(RotationCounter())
        _fill(cache, ref, wl, stream, rots[-1])
        _same_metadata(cache, ref)
        sides.append((stream, cache, ref))
    scheds = [bench.next_step_schedule(s, wl) for s, _, _ in sides]
    inps = [bench.StepInputs(wl, s, chunk, decode) for (s, _, _), (chunk, decode) in zip(sides, scheds)]
    dec = bench.stack_decode_inputs(inps)
    pre = bench.stack_prefill_inputs(inps)
    bench.run_step_multi([c for _, c, _ in sides], wl, inps, dec, None, pre)
    offs = np.concatenate([[0], np.cumsum(pre["n_q"])])
    torch.cuda.synchronize()
    for i, ((stream, cache, ref), (chunk, decode), inp) in enumerate(zip(sides, scheds, inps)):
        gids, types, pos = chunk
        ref.append(None, None, types, pos)
        rots[i].evict(ref)
        rows = np.unique(np.concatenate([[0, len(gids) - 1], rng.integers(0, len(gids), 16)]))
        for l in (0, 3):
            _give(ref, stream, l)
            _close(dev_to_f64(pre["out"][l][offs[i]:offs[i + 1]])[rows], ref.attend(l, stream.q(l, gids), pos, rows), f"stream {i} prefill layer {l}")
        for g1, t1, p1 in decode:
            ref.append(None, None, t1, p1)
            for l in (0, 3):
                _give_new(ref, stream, l, g1)
        for l in (0, 3):
            g1, t1, p1 = decode[-1]
            _close(dev_to_f64(dec[-1]["out"][l][i])[None], ref.attend(l, stream.q(l, g1), p1), f"stream {i} last decode layer {l}")
        _same_metadata(cache, ref)
        _check_kv(cache, ref, stream, wl, 3, rots[i])


def test_config2_whole_600_chunk_stream_metadata_and_final_outputs():
    """The complete 600-chunk single-layer stream (ten minutes at one chunk per second, 16 generated tokens per
    chunk): ring ordinals, page tables and positions run far past their first wrap.  Kept ordinals, positions
    and total shift are compared bit-exactly every 50 chunks; stored keys and attention outputs at the end."""
    from harness import RotationCounter, bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import streamgen as sg
    wl = sg.workloads()[2]
    stream, cache, ref = _setup(wl)
    gen = lambda tensor, g, heads: sg.rows_bf16_torch(wl.seed, tensor, 0, 0, g, heads, wl.head_dim)  # noqa: E731
    rot = RotationCounter()
    max_pos = 0
    for chunk in range(wl.chunks):
        gids, types, pos = stream.next_chunk()
        cache.append(0, gen(sg.TENSOR_K, gids, wl.kv_heads), gen(sg.TENSOR_V, gids, wl.kv_heads),
                     torch.from_numpy(types).cuda(), torch.from_numpy(np.ascontiguousarray(pos)).cuda())
        cache.evict()
        ref.append(None, None, types, pos)
        rot.evict(ref)
        toks = [stream.next_decode_token() for _ in range(wl.decode_steps)]
        g = np.concatenate([t[0] for t in toks]); ty = np.concatenate([t[1] for t in toks]); p = np.concatenate([t[2] for t in toks])
        last = chunk == wl.chunks - 1
        if not last:      # generated tokens in bulk: the same metadata as sixteen single appends
            cache.append(0, gen(sg.TENSOR_K, g, wl.kv_heads), gen(sg.TENSOR_V, g, wl.kv_heads), torch.from_numpy(ty).cuda(),
                         torch.from_numpy(np.ascontiguousarray(p)).cuda())
            ref.append(None, None, ty, p)
        if chunk % 50 == 49 or last:
            _same_metadata(cache, ref)
            max_pos = max(max_pos, int(ref.query()["pos"].max()))
    # bounded positions (contiguous RoPE): never beyond retained tokens + one chunk's span
    assert max_pos < wl.n_sink + wl.text_window + wl.vision_window + wl.max_chunk_tokens + wl.decode_steps
    # the last chunk: prefill rows and fused decode steps against the checker
    _give(ref, stream, 0)
    rng = np.random.default_rng(wl.seed)
    rows = np.unique(np.concatenate([[0, len(gids) - 1], rng.integers(0, len(gids), 16)]))
    qp = torch.from_numpy(np.ascontiguousarray(pos)).cuda()
    out = dev_to_f64(cache.attend(0, gen(sg.TENSOR_Q, gids, wl.q_heads), qp))
    _close(out[rows], ref.attend(0, stream.q(0, gids), pos, rows), "last chunk prefill")
    for g1, t1, p1 in toks:
        o = dev_to_f64(cache.decode_step(0, bits_to_dev(stream.k(0, g1)), bits_to_dev(stream.v(0, g1)),
                                         torch.from_numpy(t1).cuda(), torch.from_numpy(np.ascontiguousarray(p1)).cuda(),
                                         bits_to_dev(stream.q(0, g1))))
        ref.append(None, None, t1, p1)
        _give_new(ref, stream, 0, g1)
        _close(o, ref.attend(0, stream.q(0, g1), p1), "decode after 600 chunks")
    _same_metadata(cache, ref)
    _check_kv(cache, ref, stream, wl, 0, rot)


def test_overlap_workload_whole_window_reprefilled():
    """The sliding-window-with-overlap shape of the benchmark's second workload: all 9216 tokens of one second's
    window are appended and chunk-prefilled at once (Lq = Lk, every page causal), twice in a row with an eviction
    that drops everything in between (more evicted tokens than the metadata kernel keeps in shared memory).
    Sampled rows of the second pass against the checker; metadata bit-exact."""
    import bench
    import oracle
    from harness import bits_to_dev, dev_to_f64
    from paper_2510_09608_b200 import binding, streamgen as sg
    wl = dataclasses.replace(sg.workloads()[3], layers=1)
    gids, types, pos = bench.overlap_window(wl)
    n = len(gids)
    assert n == wl.retained          # the window after the second's eviction: the new chunk plus the retained history
    span = int(pos.max()) + 1
    cap = (n + 127) // 128 * 128
    cache = binding.Cache(1, wl.kv_heads, wl.head_dim, 0, 0, 0, cap)
    cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
    ref = oracle.Oracle(1, wl.kv_heads, wl.head_dim, 0, 0, 0, rope_mode=wl.rope_mode, rope_base=wl.rope_base, sections=wl.sections)
    stream = sg.Stream(wl, 0)
    K, V, Q = stream.k(0, gids), stream.v(0, gids), stream.q(0, gids)
    ty = torch.from_numpy(types).cuda()
    for t in range(2):
        p = np.ascontiguousarray(pos + t * span)
        cache.evict()
        ref.evict()
        cache.append(0, bits_to_dev(K), bits_to_dev(V), ty, torch.from_numpy(p).cuda())
        ref.append(K[None], V[None], types, p)
        out = cache.attend(0, bits_to_dev(Q), torch.from_numpy(p).cuda())
        assert cache.status() == binding.OK
        _same_metadata(cache, ref)
    rng = np.random.default_rng(wl.seed)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, n - 1], rng.integers(0, n, 16)]))
    _close(dev_to_f64(out)[rows], ref.attend(0, Q, p, rows), "whole-window prefill")
