"""Pins of the fp64 statement of the projection-with-append step (oracle/qkv.py); no GPU."""
import numpy as np

import oracle
from oracle import qkv
from paper_2510_09608_b200 import streamgen as sg


def _bits(rng, shape, scale=1.0):
    return qkv.to_bf16_bits(rng.standard_normal(shape) * scale)


def test_selector_weights_copy_input_columns():
    """With 0/1 weights that pick input columns the projection is a gather: every output is exactly an input."""
    rng = np.random.default_rng(1)
    n, hidden, qh, kh, d = 5, 64, 2, 1, 8
    X = _bits(rng, (n, hidden))
    W = np.zeros(((qh + 2 * kh) * d, hidden))
    cols = rng.permutation(hidden)[:W.shape[0]]
    W[np.arange(W.shape[0]), cols] = 1.0
    Q, K, V = qkv.project(X, qkv.to_bf16_bits(W), qh, kh, d)
    Y = qkv.widen(X)[:, cols]
    assert np.array_equal(Q.reshape(n, -1), Y[:, :qh * d])
    assert np.array_equal(K.reshape(n, -1), Y[:, qh * d:(qh + kh) * d])
    assert np.array_equal(V.reshape(n, -1), Y[:, (qh + kh) * d:])


def test_output_projection_selector_and_loop():
    rng = np.random.default_rng(5)
    A, W = _bits(rng, (4, 12)), _bits(rng, (7, 12))
    Y = qkv.out_project(A, W)
    Af, Wf = qkv.widen(A), qkv.widen(W)
    for i in range(4):
        for o in range(7):
            want = sum(float(Af[i, k]) * float(Wf[o, k]) for k in range(12))
            assert abs(Y[i, o] - want) <= 1e-12 * max(1.0, abs(want))
    S = np.zeros((5, 12))
    S[np.arange(5), [3, 0, 11, 7, 7]] = 1.0
    assert np.array_equal(qkv.out_project(A, qkv.to_bf16_bits(S)), Af[:, [3, 0, 11, 7, 7]])


def test_projection_is_the_triple_loop():
    rng = np.random.default_rng(2)
    n, hidden, qh, kh, d = 3, 16, 2, 1, 4
    X, W = _bits(rng, (n, hidden)), _bits(rng, ((qh + 2 * kh) * d, hidden))
    Q, K, V = qkv.project(X, W, qh, kh, d)
    Xf, Wf = qkv.widen(X), qkv.widen(W)
    for i in range(n):
        for o in range(W.shape[0]):
            want = sum(float(Xf[i, k]) * float(Wf[o, k]) for k in range(hidden))
            got = np.concatenate([Q.reshape(n, -1), K.reshape(n, -1), V.reshape(n, -1)], axis=1)[i, o]
            assert abs(got - want) <= 1e-12 * max(1.0, abs(want))


def test_rotation_identities_and_sections():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((4, 2, 16))
    a = rng.integers(0, 5000, (4, 3))
    b = rng.integers(0, 5000, (4, 3))
    sec = (2, 3, 3)
    for mode in (0, 1):
        ra = qkv.rotate(x, a, mode, 1e4, sec)
        assert np.allclose(qkv.rotate(ra, b, mode, 1e4, sec), qkv.rotate(x, a + b, mode, 1e4, sec), atol=1e-9)   # R(a)R(b)=R(a+b)
        assert np.allclose(np.linalg.norm(ra, axis=-1), np.linalg.norm(x, axis=-1))                             # isometry
        assert np.array_equal(qkv.rotate(x, np.zeros_like(a), mode, 1e4, sec), x)                                # R(0) = I
    # pair 0 has theta = 1: position pi/2 is not an integer, so check the closed form on one pair directly
    y = qkv.rotate(x, np.array([[1, 0, 0]] * 4), 1, 1e4, sec)
    assert np.allclose(y[..., 0], x[..., 0] * np.cos(1.0) - x[..., 8] * np.sin(1.0))      # pair 0 follows the t axis
    assert np.allclose(y[..., 2:8], x[..., 2:8]) and np.allclose(y[..., 10:], x[..., 10:])  # h and w pairs: position 0


def test_rotation_agrees_with_the_cache_checker():
    """The stored-key rotation of the C++ checker (pinned on its own in test_oracle_*.py) and this numpy statement
    are separate code; on bf16-exact raw keys they must give the same rotated keys."""
    wl = sg.workloads()[2]
    ref = oracle.Oracle(1, wl.kv_heads, wl.head_dim, 4, 64, 16, rope_mode=wl.rope_mode, rope_base=wl.rope_base, sections=wl.sections)
    stream = sg.Stream(wl, 0)
    for _ in range(2):
        gids, types, pos = stream.next_chunk()
        ref.append(stream.k(0, gids)[None], stream.v(0, gids)[None], types, pos)
        ref.evict()
    q = ref.query()
    want = ref.rotated_k(0)
    got = qkv.rotate(qkv.widen(stream.k(0, q["gids"])), q["pos"], wl.rope_mode, wl.rope_base, wl.sections)
    assert np.allclose(got, want, atol=1e-9)


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0])
    assert np.array_equal(qkv.widen(qkv.to_bf16_bits(x)), np.array([1.0, 1.0, 1.0 + 2.0 ** -6, -2.5, 0.0]))
