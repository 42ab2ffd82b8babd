"""The seeded input generators: reproducible, and bf16 rounding is round-to-nearest-even."""
import numpy as np
import torch

from paper_2609_32814_b200 import synth


def test_bf16_rounding_matches_torch():
    x = synth.normal(123, (4096,), 3.0)
    bits = synth.to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(bits.view(np.int16), want.view(torch.int16).numpy())
    assert np.array_equal(synth.from_bf16_bits(bits), want.float().numpy())
    ties = np.array([1.00390625, 1.01171875, -1.00390625], dtype=np.float32)  # exact halves
    assert np.array_equal(synth.bf16_round(ties), np.array([1.0, 1.015625, -1.0], dtype=np.float32))


def test_workloads_are_reproducible_and_shaped():
    a, b = synth.config2(M=256, seq=128), synth.config2(M=256, seq=128)
    assert np.array_equal(a.X, b.X) and np.array_equal(a.W_up, b.W_up)
    assert a.d_widths == [384, 384] and a.f_widths == [1536, 1536]
    assert a.types.tolist()[:4] == [0, 1, 0, 1] and a.types[128] == 0
    assert np.array_equal(synth.bf16_round(a.X), a.X)
    c1 = synth.config1(integer=True)
    assert c1.X.shape == (512, 256) and c1.W_up.shape == (256, 1024)
    assert set(np.unique(c1.X)) <= set(range(-3, 4))
    w = synth.config3(4, M=512)
    assert w.d_widths == [128] * 4 and w.f_widths == [512] * 4 and w.types.max() == 3
    d = synth.config4(8)
    assert d.M == 8 and set(np.unique(d.types)) <= {0, 1}
    assert abs(float(a.W_up.std()) - 0.02) < 2e-3
