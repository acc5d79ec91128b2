"""The seeded generator: reproducible, slice-addressable, plausible N(0,1)."""
import numpy as np

from paper_2609_20734_b200 import synth


def test_slices_match_whole_tensor():
    whole = synth.gauss_bf16_tensor(5, synth.STREAM_K, (1000,))
    part = synth.gauss_bf16(synth.stream_key(5, synth.STREAM_K), np.arange(100, 200))
    np.testing.assert_array_equal(whole[100:200], part)
    assert (synth.gauss_bf16_tensor(5, synth.STREAM_V, (1000,)) != whole).mean() > 0.9
    assert (synth.gauss_bf16_tensor(6, synth.STREAM_K, (1000,)) != whole).mean() > 0.9


def test_distribution():
    x = synth.bf16_bits_to_f32(synth.gauss_bf16_tensor(1, synth.STREAM_Q, (200000,)))
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    assert np.isfinite(x).all() and np.abs(x).max() < 5
    w = synth.gauss_f32_tensor(1, synth.STREAM_W1, (100000,), std=0.02)
    assert abs(w.std() - 0.02) < 5e-4


def test_bf16_round_trip():
    x = np.array([0.0, 1.0, -1.5, 3.140625, 1e-3], dtype=np.float32)
    b = synth.f32_to_bf16_bits(x)
    y = synth.bf16_bits_to_f32(b)
    assert (np.abs(y - x) <= np.abs(x) * 2.0 ** -8).all()
    np.testing.assert_array_equal(synth.f32_to_bf16_bits(y), b)
    # ties round to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(np.array([1 + 2.0 ** -8], np.float32)))[0] == 1.0


def test_block_tables():
    need = np.array([3, 5, 1])
    t, pool = synth.block_tables(3, need, 6, shuffled=True, num_blocks=12)
    used = t[t >= 0]
    assert len(used) == 9 and len(set(used.tolist())) == 9 and used.max() < 12
    assert (t[0, 3:] == -1).all()
    t2, _ = synth.block_tables(3, need, 6, shuffled=False)
    np.testing.assert_array_equal(t2[1, :5], np.arange(3, 8))
    lens = synth.uniform_lengths(4, 1000, 8192, 65536)
    assert lens.min() >= 8192 and lens.max() <= 65536 and lens.std() > 10000
