"""The seeded input generator: shapes, determinism, padding structure, bf16 rounding."""
import numpy as np

from paper_2506_02939_b200 import synth


def test_c1_shape_and_padding():
    a = synth.make_inputs("c1")
    b_ = synth.make_inputs("c1")
    assert a.X.shape == (2048, 512) and a.dY.shape == (2048, 1536) and a.X.dtype == np.float32
    assert np.array_equal(a.X, b_.X) and np.array_equal(a.dY, b_.dY)
    frac = len(a.pad_rows) / 2048
    assert 0.03 < frac < 0.2
    assert np.all(a.X[a.pad_rows] == a.X[a.pad_rows[0]])         # exact duplicates
    assert abs(float(a.dY.std()) - 1e-3) < 1e-4


def test_c2_reduced_has_zero_and_duplicate_padding():
    a = synth.make_inputs("c2", num_seqs=8)
    assert a.X.shape == (8 * 256, 768) and a.X.dtype == np.uint16 and a.dY.dtype == np.uint16
    pads = a.X[a.pad_rows]
    zero = np.all((pads & 0x7FFF) == 0, axis=1)
    assert zero.any() and (~zero).any()
    nz = pads[~zero]
    assert np.all(nz == nz[0])


def test_seed_override_changes_data():
    a = synth.make_inputs("c2", num_seqs=2, seed=5)
    b_ = synth.make_inputs("c2", num_seqs=2, seed=6)
    assert not np.array_equal(a.X, b_.X)


def test_c3_reduced_unit_rms_heavy_tail():
    a = synth.make_inputs("c3", num_seqs=4)
    x = synth.bf16_bits_to_f32(a.X).astype(np.float64)
    assert abs(np.sqrt(np.mean(x * x)) - 1.0) < 0.01
    kurt = np.mean(x ** 4) / np.mean(x ** 2) ** 2
    assert kurt > 4.0                                             # heavier than Gaussian (3)


def test_bf16_round_to_nearest_even():
    import torch
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 3.0e38]        # exact halves -> even
    ours = synth.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    assert np.array_equal(synth.bf16_bits_to_f32(ours), torch.from_numpy(x).to(torch.bfloat16).float().numpy())
