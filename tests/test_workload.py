"""The seeded generator: determinism, shapes, bf16 rounding and the stated structure."""
import numpy as np

from paper_2607_27692_b200 import workload as wl


def test_bf16_round_trip_and_rounding():
    x = np.array([1.0, -2.5, 1.00390625, 1.01171875, 3.0e-3, 0.0], dtype=np.float32)
    b = wl.f32_to_bf16_bits(x)
    back = wl.bf16_bits_to_f32(b)
    assert back[0] == 1.0 and back[1] == -2.5 and back[5] == 0.0
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: nearest even keeps 1.0
    assert back[2] == 1.0
    # 1 + 3*2^-8 ties between 1 + 2^-7 and 1 + 2^-6: nearest even is 1 + 2^-6
    assert back[3] == 1.015625
    assert abs(back[4] - 3.0e-3) <= 3.0e-3 * 2.0 ** -8
    assert np.array_equal(wl.bf16_bits_to_f64(b), back.astype(np.float64))


def test_stream_is_deterministic_and_shaped():
    cfg = wl.CONFIGS["tiny"].replace(context=128, steps=12, B=2, H_q=4, H_kv=2)
    a = wl.make_stream(cfg, steps=12, workers=1)
    b = wl.make_stream(cfg, steps=12, workers=4)
    assert a.k.shape == (2, 2, 140, 64) and a.q.shape == (12, 2, 4, 64)
    for x, y in ((a.k, b.k), (a.v, b.v), (a.q, b.q)):
        assert x.dtype == np.uint16 and np.array_equal(x, y)
    assert a.seq_len(0) == 129
    # a sampled sequence equals the same row of the full batch
    one = wl.make_stream(cfg, steps=12, sequences=range(1, 2))
    assert np.array_equal(one.k[0], a.k[1]) and np.array_equal(one.q[:, 0], a.q[:, 1])
    # other layers are independent draws
    other = wl.make_stream(cfg, steps=12, layer=1)
    assert not np.array_equal(other.k, a.k)


def test_queries_are_a_slow_walk_on_the_sphere():
    cfg = wl.CONFIGS["llama16k"].replace(context=64, steps=200, B=1, p_jump=0.0)
    st = wl.make_stream(cfg, steps=200)
    q = wl.bf16_bits_to_f64(st.q[:, 0, 0])
    n = np.linalg.norm(q, axis=1)
    assert np.allclose(n, 1.0, atol=5e-3)
    cos = (q[1:] * q[:-1]).sum(1) / (n[1:] * n[:-1])
    assert 0.88 < cos.mean() < 0.915


def test_quarter_of_keys_sit_near_a_centre():
    cfg = wl.CONFIGS["tiny"].replace(context=8192, steps=4)
    st = wl.make_stream(cfg, steps=4)
    k = wl.bf16_bits_to_f64(st.k[0, 0, :8192])
    # centred keys have norm about 2*sqrt(d), plain ones about sqrt(d)
    frac = (np.linalg.norm(k, axis=1) > 1.5 * np.sqrt(cfg.d)).mean()
    assert 0.22 < frac < 0.28
