"""The seeded generator: deterministic, right moments, exact bf16 rounding."""
import numpy as np

from paper_1708_08917_b200 import synth


def test_deterministic_and_stream_separated():
    a = synth.normal((1000,), 1.0, synth.stream_id("c", "w"))
    b = synth.normal((1000,), 1.0, synth.stream_id("c", "w"))
    c = synth.normal((1000,), 1.0, synth.stream_id("c", "x"))
    assert np.array_equal(a, b) and not np.array_equal(a, c) and a.dtype == np.float32


def test_moments():
    z = synth.normal((200_000,), 1.0 / 4096, 7).astype(np.float64)
    assert abs(z.mean()) < 3e-4 and abs(z.std() - 1 / 64) < 2e-4      # second argument is the variance
    u = synth.uniform((200_000,), -1.0, 1.0, 9).astype(np.float64)
    assert u.min() > -1 and u.max() < 1 and abs(u.mean()) < 5e-3 and abs(u.var() - 1 / 3) < 5e-3
    assert synth.normal((1000,), 1.0, 3, absolute=True).min() >= 0


def test_bf16_rounding_ties_to_even():
    f = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -0.3, 3.1415926], dtype=np.float32)
    r = synth.round_to_bf16(f)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2 ** -7 and r[3] == 1.0 + 2 ** -6
    import torch
    ref = torch.from_numpy(f).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(r, ref)
    big = synth.normal((4096,), 1.0, 11)
    assert np.array_equal(synth.round_to_bf16(big), torch.from_numpy(big).to(torch.bfloat16).float().numpy())
    assert np.array_equal(synth.bf16_bits_to_f32(synth.bf16_bits(synth.round_to_bf16(big))), synth.round_to_bf16(big))


def test_config_shapes():
    c1 = synth.config1()
    assert c1.w.shape == (16, 16, 16) and c1.x.shape == (1, 256) and c1.bias is None and not c1.relu
    c2 = synth.config2(16)
    assert c2.w.shape == (64, 64, 64) and c2.x.shape == (16, 4096) and c2.bias.shape == (4096,) and c2.relu
    l = synth.config3_layers(4)
    assert [c.w.shape for c in l] == [(32, 72, 128), (32, 32, 128), (8, 32, 128)] and l[0].x.shape == (4, 9216)
    c4 = synth.config4(2, 5, 5)
    assert c4.w.shape == (3, 3, 16, 16, 16) and c4.x.shape == (2, 5, 5, 256)
    assert np.array_equal(c4.x, synth.round_to_bf16(c4.x)) and c4.x.min() >= 0
