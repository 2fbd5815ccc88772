"""The synthetic input generator: determinism, addressability and the stated distribution."""
import numpy as np

from paper_2510_09608_b200 import streamgen as sg


def test_rows_are_addressable_and_deterministic():
    a = sg.rows_bf16(0x5EED0002, sg.TENSOR_K, 0, 3, np.arange(100, 140), 4, 128)
    b = sg.rows_bf16(0x5EED0002, sg.TENSOR_K, 0, 3, np.array([117]), 4, 128)
    assert a.dtype == np.uint16 and a.shape == (40, 4, 128)
    assert np.array_equal(a[17], b[0])
    c = sg.rows_bf16(0x5EED0002, sg.TENSOR_V, 0, 3, np.array([117]), 4, 128)
    assert not np.array_equal(b, c)


def test_values_are_standard_normal():
    x = sg.bf16_bits_to_f64(sg.rows_bf16(1, sg.TENSOR_Q, 0, 0, np.arange(2000), 4, 64))
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    assert abs((np.abs(x) < 1.0).mean() - 0.6827) < 0.01
    t = sg.bf16_bits_to_f64(sg.normal_table())
    assert np.all(np.diff(t) >= 0) and t[0] < -4 and t[-1] > 4


def test_chunk_schedule_shapes():
    wl = sg.workloads()[2]
    s = sg.Stream(wl)
    gids, types, pos = s.next_chunk()
    assert (types[:512] == sg.VISION).all() and (types[512:] == sg.TEXT).all()
    assert pos.shape == (len(gids), 3) and 512 <= len(gids) <= 536
    assert pos[:512].max() == 15 and pos[0].tolist() == [0, 0, 0] and pos[511].tolist() == [1, 15, 15]
    if len(gids) > 512:
        assert pos[512].tolist() == [16, 16, 16]
    g2, t2, p2 = s.next_decode_token()
    assert g2[0] == len(gids) and t2[0] == sg.TEXT
    counts = [sg.Stream(wl).text_count(c) for c in range(400)]
    assert min(counts) == 0 and max(counts) == 24
    wl1 = sg.workloads()[1]
    g, t, p = sg.Stream(wl1).next_chunk()
    assert p.ndim == 1 and (t[:32] == sg.VISION).all() and 32 <= len(g) <= 40


def test_torch_generator_is_bit_identical():
    import torch
    gids = np.array([0, 1, 17, 123456789, 2 ** 40 + 5])
    for tensor, heads, d in ((sg.TENSOR_K, 4, 128), (sg.TENSOR_Q, 28, 128), (sg.TENSOR_V, 1, 64)):
        a = sg.rows_bf16(0x5EED0003, tensor, 5, 27, gids, heads, d)
        b = sg.rows_bf16_torch(0x5EED0003, tensor, 5, 27, gids, heads, d, device="cpu")
        assert np.array_equal(a, b.view(torch.int16).numpy().view(np.uint16))
