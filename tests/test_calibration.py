"""Calibration of the equalization vector with positional interpolation (Sec. 3.3, Eq. 10-12): pins for
the oracle on CPU, parity of the device kernel on GPU."""
import math

import numpy as np
import pytest
import torch

from oracle import pmkvq_oracle as O
from paper_2505_18610_b200 import synth


def test_rotation_keeps_pair_norms_and_matches_the_generator():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((50, 2, 3, 128))
    pos = np.arange(50) * 7
    y = O.rope_interpolated(x, pos, pos_scale=2.5)
    assert np.allclose(x[..., :64] ** 2 + x[..., 64:] ** 2, y[..., :64] ** 2 + y[..., 64:] ** 2)
    # the input generator's RoPE (Eq. 11/12, written independently on torch) agrees
    z = synth.apply_rope(torch.tensor(x, dtype=torch.float32), torch.tensor(pos), pos_scale=2.5).numpy()
    assert np.allclose(y, z, atol=2e-5)


def test_single_pair_closed_form_and_interpolation_identity():
    n, a, b, i = 300, 0.6, -1.3, 10
    k = np.zeros((n, 1, 1, 128)); k[..., i] = a; k[..., i + 64] = b
    th = 10000.0 ** (-2.0 * i / 128)
    r, phi = math.hypot(a, b), math.atan2(b, a)
    for s in (1.0, 4.0):
        lam = O.calibrate_lambda(k, pos_scale=s, alpha=1.0)
        m = np.arange(n)
        assert np.isclose(lam[0, i], np.abs(r * np.cos(m * s * th + phi)).max())
        assert np.isclose(lam[0, i + 64], np.abs(r * np.sin(m * s * th + phi)).max())
        assert np.allclose(np.delete(lam[0], [i, i + 64]), 1e-5)        # untouched channels sit at the floor
    # s = 4 on n tokens sees the angles of positions 0, 4, 8, ... of plain RoPE (Eq. 12 vs Eq. 11)
    rng = np.random.default_rng(1)
    kk = rng.standard_normal((64, 2, 2, 128))
    direct = np.abs(O.rope_interpolated(kk, np.arange(64) * 4, 1.0)).max(axis=(0, 1)) ** 0.5
    assert np.allclose(O.calibrate_lambda(kk, pos_scale=4.0), direct)


def test_short_calibration_needs_interpolation_for_the_slow_pair():
    """Sec. 3.3: the lowest-frequency pair has a period of 54,410 tokens; 2,048 tokens of plain RoPE sweep
    13.5 degrees of it, positional interpolation widens the sweep by its factor."""
    i = 63
    th = 10000.0 ** (-2.0 * i / 128)
    assert round(2 * math.pi / th) == 54410
    k = np.zeros((2048, 1, 1, 128)); k[..., i] = 1.0          # amplitude sits in the cosine channel at position 0
    plain = O.calibrate_lambda(k, pos_scale=1.0, alpha=1.0)[0, i + 64]
    interp = O.calibrate_lambda(k, pos_scale=4.0, alpha=1.0)[0, i + 64]
    assert np.isclose(plain, math.sin(2047 * th)) and np.isclose(interp, math.sin(2047 * 4 * th))
    assert interp > 3.4 * plain and interp < 1.0          # sin(4x) / sin(x) at x = 13.5 degrees


@pytest.mark.gpu
@pytest.mark.parametrize("n_tokens,n_seq,kv_heads,scale", [(1, 1, 1, 1.0), (333, 3, 4, 1.0), (2048, 2, 8, 4.0), (700, 1, 12, 2.0)])
def test_device_calibration_matches_oracle(n_tokens, n_seq, kv_heads, scale):
    from paper_2505_18610_b200 import binding as B
    g = torch.Generator().manual_seed(n_tokens)
    k = torch.randn(n_tokens, n_seq, kv_heads, 128, generator=g)
    k[..., 5] *= 15.0
    k[:, :, 0, 100] *= 20.0
    k = k.to(torch.bfloat16)
    want = O.calibrate_lambda(k.float().numpy(), pos_scale=scale, alpha=0.5)
    got = B.calibrate_lambda(k.cuda().contiguous(), pos_scale=scale, alpha=0.5).cpu().numpy()
    assert got.shape == want.shape
    assert np.allclose(got, want, rtol=2e-6 * 8, atol=0)      # fp32 rotation: a few ulp on |K_rot|, halved by the root
