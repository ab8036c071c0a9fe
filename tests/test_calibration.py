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


# ---- Sec. 4.1.1: alpha by grid search on the attention reconstruction loss ----
def _calib_tensors(n, n_seq, kv_heads, group, seed, outlier=None):
    g = torch.Generator().manual_seed(seed)
    k = torch.randn(n, n_seq, kv_heads, 128, generator=g)
    q = torch.randn(n, n_seq, kv_heads * group, 128, generator=g)
    v = torch.randn(n, n_seq, kv_heads, 128, generator=g)
    if outlier:
        ch, gain = outlier
        k[..., ch] *= gain
        k[..., ch + 64] *= gain
    return tuple(t.to(torch.bfloat16).float().numpy() for t in (k, q, v))


def test_causal_attention_against_loops_and_head_map():
    rng = np.random.default_rng(3)
    n, group, kvh = 5, 2, 2
    q = rng.standard_normal((n, 1, kvh * group, 128)); k = rng.standard_normal((n, 1, kvh, 128))
    v = rng.standard_normal((n, 1, kvh, 128))
    got = O.causal_self_attention(q, k, v, group)
    for t in range(n):
        for h in range(kvh * group):
            w = [math.exp(float(q[t, 0, h] @ k[j, 0, h // group]) / math.sqrt(128.0)) for j in range(t + 1)]
            want = sum(w[j] * v[j, 0, h // group] for j in range(t + 1)) / sum(w)
            assert np.allclose(got[t, 0, h], want, rtol=1e-12, atol=1e-14)
    # a later token changes nothing before it
    k2, v2 = k.copy(), v.copy(); k2[3:] += 1.0; v2[3:] -= 2.0
    assert np.array_equal(O.causal_self_attention(q, k2, v2, group)[:3], got[:3])


def test_loss_vanishes_at_16_bit_for_every_alpha():
    """(Q Lambda)(K Lambda^-1)^T = Q K^T: with a 16-bit quantizer only its tiny rounding is left, for every
    alpha; a Lambda applied on one side only, or twice, leaves a loss of the order of the output itself."""
    k, q, v = _calib_tensors(40, 2, 2, 3, seed=5, outlier=(7, 30.0))
    ref = O.causal_self_attention(O.rope_interpolated(q, np.arange(40)), O.rope_interpolated(k, np.arange(40)), v, 3)
    losses = O.attention_reconstruction_losses(k, q, v, 3, 16, [0.0, 0.3, 0.7, 1.0])
    assert np.all(losses < 1e-7 * np.mean(ref ** 2))
    assert np.all(O.attention_reconstruction_losses(k, q, v, 3, 2, [0.0, 0.3, 0.7, 1.0]) > 1e-3 * np.mean(ref ** 2))


def test_single_token_loss_is_the_value_error_alone():
    k, q, v = _calib_tensors(1, 3, 2, 2, seed=6)
    for bits in (2, 4, 8):
        losses = O.attention_reconstruction_losses(k, q, v, 2, bits, O.alpha_grid(5))
        # softmax over one key is 1: every head returns its KV head's quantized Value; the cache oracle
        # (n_sink = window = 0, budget of a cache at `bits`) supplies that Value independently
        err = 0.0
        for b in range(3):
            pol = O.Policy(bits, 1, 2, n_sink=0, window=0)
            lo = O.LayerOracle(pol, 2)
            lo.append(k[:, b], v[:, b])
            while pol.cur_bits > bits:
                lo.reduce()
            for h in range(2):
                cv, sv, zv, _b = lo.export_slice(h, True)
                err += 2 * float(((O.dequantize(cv, sv, zv)[0] - v[0, b, h]) ** 2).sum())   # group = 2 heads each
        assert np.allclose(losses, err / (3 * 4 * 128), rtol=1e-12)


@pytest.mark.parametrize("bits", [2, 4])
def test_last_query_row_equals_decode_attention_of_the_cache_oracle(bits):
    n, group, kvh = 37, 3, 2
    k, q, v = _calib_tensors(n, 1, kvh, group, seed=8, outlier=(20, 12.0))
    pos = np.arange(n)
    k_rot = O.rope_interpolated(k, pos, 2.0).astype(np.float32)
    q_rot = O.rope_interpolated(q, pos, 2.0).astype(np.float32)
    ref = O.causal_self_attention(q_rot, k_rot, v, group)
    alpha = 0.6
    lam = (np.maximum(np.abs(k_rot.astype(np.float64)).max(axis=(0, 1)), 1e-5) ** alpha).astype(np.float32)
    pol = O.Policy(bits, n, kvh, n_sink=0, window=0)
    lo = O.LayerOracle(pol, kvh, lam=lam)
    lo.append_bulk(k_rot[:, 0], v[:, 0])
    while pol.cur_bits > bits:
        lo.reduce()
    last = lo.decode_attention(q_rot[n - 1, 0].reshape(kvh, group, 128)).reshape(kvh * group, 128)
    # the last row of the quantized operator, assembled as the loss function assembles it
    lam64 = np.repeat(lam.astype(np.float64), group, axis=0)
    k_hat = O.quantize_progressively((k_rot * (np.float32(1.0) / lam)[None, None]).astype(np.float32), bits)
    got = O.causal_self_attention(q_rot.astype(np.float64) * lam64[None, None], k_hat, O.quantize_progressively(v, bits), group)
    assert np.allclose(got[n - 1, 0], last, rtol=0, atol=2e-6)
    # and the loss is the mean squared difference of exactly these two operators
    loss = O.attention_reconstruction_losses(k, q, v, group, bits, [alpha], pos_scale=2.0)[0]
    ref64 = O.causal_self_attention(O.rope_interpolated(q, pos, 2.0), O.rope_interpolated(k, pos, 2.0), v, group)
    got64 = O.causal_self_attention(O.rope_interpolated(q, pos, 2.0) * lam64[None, None], k_hat, O.quantize_progressively(v, bits), group)
    assert np.isclose(loss, np.mean((got64 - ref64) ** 2), rtol=1e-9)
    assert np.mean((ref - ref64) ** 2) < 1e-10


def test_alpha_one_loss_ignores_power_of_two_rescaling_of_a_channel_pair():
    """At alpha = 1, K Lambda^-1 has unit abs-max per channel whatever the channel's gain: scaling a rotated
    pair (i, i + 64) of K by 2^e and of Q by 2^-e changes neither factor of Eq. 9, so the loss stays put;
    with alpha = 0 (no equalization) the same rescaling changes it."""
    k, q, v = _calib_tensors(48, 1, 1, 2, seed=9)
    k2, q2 = k.copy(), q.copy()
    for ch, e in ((3, 4), (40, -3)):
        for c in (ch, ch + 64):
            k2[..., c] *= 2.0 ** e
            q2[..., c] *= 2.0 ** -e
    a = O.attention_reconstruction_losses(k, q, v, 2, 2, [1.0, 0.0])
    b = O.attention_reconstruction_losses(k2, q2, v, 2, 2, [1.0, 0.0])
    assert np.isclose(a[0], b[0], rtol=1e-6)
    assert abs(a[1] - b[1]) > 0.05 * a[1]


def test_outlier_channels_move_the_best_alpha_off_zero():
    """Sec. 3.3: a channel pair with large magnitude eats the range of every token's group; moving part of it
    into the Queries (alpha > 0) lowers the reconstruction loss at low width."""
    k, q, v = _calib_tensors(64, 2, 2, 2, seed=10, outlier=(11, 40.0))
    best, losses = O.grid_search_alpha(k, q, v, 2, 2, n_grid=10)
    assert np.allclose(O.alpha_grid(10), np.arange(10) / 10.0) and len(losses) == 10
    assert best >= 0.3 and losses.min() < 0.7 * losses[0]
    assert best == O.alpha_grid(10)[int(np.argmin(losses))]


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


@pytest.mark.gpu
@pytest.mark.parametrize("n_tokens,n_seq,kv_heads,group,bits,scale",
                         [(1, 1, 1, 1, 2, 1.0), (45, 2, 2, 3, 2, 1.0), (130, 1, 2, 7, 4, 4.0), (97, 2, 1, 2, 8, 2.0),
                          (300, 2, 2, 4, 4, 1.0), (257, 1, 1, 8, 2, 2.0)])   # several query blocks and key tiles, ragged ends
def test_device_alpha_grid_matches_oracle(n_tokens, n_seq, kv_heads, group, bits, scale):
    from paper_2505_18610_b200 import binding as B
    k, q, v = _calib_tensors(n_tokens, n_seq, kv_heads, group, seed=100 + n_tokens, outlier=(9, 25.0))
    alphas = O.alpha_grid(8)
    want = O.attention_reconstruction_losses(k, q, v, group, bits, alphas, pos_scale=scale)
    dev = [torch.tensor(t).to(torch.bfloat16).cuda().contiguous() for t in (k, q, v)]
    best, got = B.alpha_grid_search(dev[0], dev[1], dev[2], bits, alphas=alphas, pos_scale=scale)
    # fp32-like attention on both operators (operands of 22 significant bits, fp32 sums): the loss is a squared
    # difference of two such outputs, so its
    # relative error grows as the quantization error shrinks (2e-2 covers 8 bit)
    assert np.allclose(got, want, rtol=2e-2 if bits == 8 else 2e-3, atol=0)
    order = np.sort(want)
    if len(order) > 1 and order[1] > 1.05 * order[0]:      # a clear winner must be found
        assert best == pytest.approx(float(alphas[int(np.argmin(want))]))


@pytest.mark.gpu
def test_device_alpha_grid_argument_checks():
    from paper_2505_18610_b200 import binding as B
    k, q, v = (torch.zeros(4, 1, 1, 128, dtype=torch.bfloat16, device="cuda") for _ in range(3))
    with pytest.raises(B.PmkvqError):
        B.alpha_grid_search(k, q, v, 3)
    with pytest.raises(B.PmkvqError):
        B.alpha_grid_search(k, q, v, 2, alphas=np.zeros(65))
    # constant tensors: every group has S = 0, nothing is lost, every loss is 0
    best, losses = B.alpha_grid_search(k, q, v, 2)
    assert best == 0.0 and np.all(losses == 0.0) and len(losses) == 20
