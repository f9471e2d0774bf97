"""The seeded input generator: layouts, shapes, determinism.  CPU only."""
import numpy as np

import hkv_inputs as hi


def test_layouts_match_the_recipes():
    m = hi.layout_sandwich(64, 1920, 64)
    assert m.size == 2048 and m.sum() == 128 and m[:64].all() and m[-64:].all() and not m[64:-64].any()
    m = hi.layout_image_blocks(16384)
    assert m.size == 16384 and int(m.sum()) == 320 and m[-64:].all() and m[:16].all()
    m = hi.layout_image_blocks(50000)
    assert int(m.sum()) == 848
    m = hi.layout_image_blocks(32768)
    assert int(m.sum()) == 576
    m, f = hi.layout_video(64)
    assert m.size == 32768 and int(m.sum()) == 64 + 64 * 11 and f.max() == 63
    m, _ = hi.layout_video(48)
    assert m.size >= 24576


def test_generation_is_deterministic_and_thread_independent():
    a = hi.cfg2(layer=3, B=2, n_frames=4, min_frames=3, frame_visual=50, threads=1)
    b = hi.cfg2(layer=3, B=2, n_frames=4, min_frames=3, frame_visual=50, threads=4)
    for x, y in [(a.k, b.k), (a.v, b.v), (a.q_obs, b.q_obs), (a.q[0], b.q[0]), (a.head_type, b.head_type)]:
        assert np.array_equal(x, y)
    c = hi.cfg2(layer=4, B=2, n_frames=4, min_frames=3, frame_visual=50)
    assert not np.array_equal(a.k, c.k)
    assert np.array_equal(a.seq_lens, c.seq_lens)          # lengths are a property of the batch, not the layer
    assert a.seq_lens[0] == a.max_seq_len


def test_cfg0_geometry_and_values():
    L = hi.cfg0()
    assert (L.batch, L.n_q_heads, L.n_kv_heads, L.head_dim, L.max_seq_len) == (1, 28, 4, 128, 2048)
    assert L.budgets.tolist() == [[205] * 4] and L.chunk_size == 32 and L.obs_window == 32
    assert sorted(L.head_type[0].tolist()) == [0, 0, 1, 1]
    k = hi.bf16_bits_to_f32(L.k[0, 0])
    var = k.var(axis=0)
    assert (var > 30).sum() == 4 and (var < 2).sum() == 124     # 4 outlier channels x8
    assert np.array_equal(var > 30, hi.bf16_bits_to_f32(L.v[0, 0]).var(axis=0) > 30)


def test_static_fraction_counts():
    for f, n in [(0.0, 0), (0.25, 16), (0.5, 32), (0.75, 48), (1.0, 64)]:
        ht = hi._choose_static(4, 0, 16, 4, f)
        assert int((ht == 0).sum()) == n
    assert int((hi._choose_static(2, 5, 4, 4, 0.6) == 0).sum()) == 10
    assert int((hi._choose_static(3, 5, 8, 4, 0.4) == 0).sum()) == 13


def test_bf16_round_trip():
    x = np.array([1.0, -2.5, 0.1, 3.0e-3, 1 + 2.0 ** -8], dtype=np.float32)
    b = hi.f32_to_bf16_bits(x)
    assert b[0] == 0x3F80 and b[4] == 0x3F80
    assert np.allclose(hi.bf16_bits_to_f32(b), x, rtol=2 ** -8)
