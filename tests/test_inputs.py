"""The seeded input recipes: shapes, dtypes, determinism and the structure each configuration states."""
import numpy as np
import torch

import luvc_inputs as gi


def test_config0_is_fp32_and_reproducible():
    a, b = gi.oim_input(0), gi.oim_input(0)
    assert a.shape == (1, 24, 24, 1024) and a.dtype == torch.float32
    assert torch.equal(a, b)
    # 8 unit-variance cosines per channel (variance 8 * 1/2 = 4) plus N(0, 0.1) noise
    assert 1.7 < a.std().item() < 2.3


def test_config1_has_high_norm_outliers():
    x = gi.oim_input(1, batch=2)
    assert x.shape == (2, 24, 24, 1024) and x.dtype == torch.bfloat16
    norms = x.float().reshape(2, 576, 1024).norm(dim=-1)
    for b in range(2):
        big = (norms[b] > 4 * norms[b].median()).sum().item()
        assert big == round(0.02 * 576)
    assert not torch.equal(x[0], x[1])           # a fresh seed per image


def test_config3_frames_drift_slowly():
    x = gi.oim_input(3, batch=3, hw=(12, 12), dim=64).float()
    d01 = (x[0] - x[1]).norm() / x[0].norm()
    assert 0.0 < d01 < 0.6                       # consecutive frames are similar, not identical


def test_reduced_cases_and_projection():
    x = gi.oim_input(2, batch=1, hw=(16, 16), dim=32)
    assert x.shape == (1, 16, 16, 32) and x.dtype == torch.bfloat16
    merged = torch.randn(4, 9, 32)
    y = gi.spu_input_from_tokens(2, merged, dim_out=48)
    assert y.shape == (4, 9, 48) and y.dtype == torch.bfloat16
    assert torch.equal(y, gi.spu_input_from_tokens(2, merged, dim_out=48))
    v = gi.spu_input_from_tokens(3, torch.randn(32, 5, 32), dim_out=16)
    assert v.shape == (2, 80, 16)                # 16 frames of each video concatenated in time order


def test_stress_sequence_is_low_frequency_plus_noise():
    x = gi.spu_stress_input(batch=1, n_tokens=512, dim=64)
    assert x.shape == (1, 512, 64) and x.dtype == torch.bfloat16
    spec = np.abs(np.fft.rfft(x[0].float().numpy(), axis=0)) ** 2
    low, high = spec[:10].sum(), spec[10:].sum()
    assert low > high                            # most energy sits below 8 cycles per sequence
    assert gi.keep_count(0.25, 1296) == 324 and gi.keep_count(0.1, 1296) == 130 and gi.keep_count(0.05, 1296) == 65
    assert gi.keep_count(0.1, 16384) == 1638
