"""Pins for the oracle's progressive policy (Sec. 3.1), its cache bookkeeping and its decode
attention (Eq. 9 + softmax attention).  Checked against what the paper fixes (halving thresholds,
Table 1 shapes, RoPE period), closed forms, brute-force loops and a library attention routine."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import pmkvq_oracle as O
from paper_2505_18610_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def _bf16(a):
    return torch.tensor(a).to(torch.bfloat16).float().numpy()


# ------------------------------------------------------------------ policy ----
def test_halving_thresholds_from_paper():
    """With code-bit accounting and no sink/window, the width is halved exactly when the cache
    holds max_len*Fbit/16, /8, /4 tokens and one more arrives (Fig. 2a, App. C.7)."""
    for row in _rows("halving_thresholds.txt"):
        fbit, max_len, want = int(row[0]), int(row[1]), [int(v) for v in row[2:]]
        pol = O.Policy(fbit, max_len, n_slices=3, n_sink=0, window=0, count_metadata=False)
        fired, bits_seen = [], [16]
        for n in range(max_len):
            k, ok = pol.reduces_needed_for(n + 1)
            assert ok
            for _ in range(k):
                fired.append(n)
                pol.cur_bits //= 2
            pol.n_tokens = n + 1
            assert pol.bytes_used() <= pol.budget
        assert fired == want
        assert pol.cur_bits == fbit
        # the cache is exactly full at max_len and nothing more fits
        assert pol.bytes_used() == pol.budget
        assert pol.reduces_needed_for(max_len + 1)[1] is False


def test_default_budget_and_accounting():
    pol = O.Policy(4, 4096, n_slices=1, n_sink=1, window=128)
    # 129 INT16 tokens + 3967 4-bit tokens, K and V, codes + fp32 scale + fp32 zero
    assert pol.budget == 2 * (129 * (256 + 8) + 3967 * (64 + 8))
    assert O.tokbytes(2) == 40 and O.tokbytes(16) == 264 and O.tokbytes(8, False) == 128
    # eviction granularity: the window floats in [W, W + C)
    polc = O.Policy(2, 1000, 1, n_sink=1, window=128, evict_chunk=16)
    assert [polc.n_body_at(n) for n in (0, 1, 129, 144, 145, 160, 161)] == [0, 0, 0, 0, 16, 16, 32]
    assert [pol.n_body_at(n) for n in (129, 130, 131)] == [0, 1, 2]


def test_table1_shapes():
    """Table 1: 2 (K,V) x layers x kv_heads x 128 x 2 bytes x 32K tokens x batch 16."""
    for name, layers, kvh, hd, gb in _rows("table1_kv_memory.txt"):
        size = 2 * int(layers) * int(kvh) * int(hd) * 2 * 32768 * 16
        assert size == int(gb) * 2 ** 30


def test_rope_period_pins_generator_frequencies():
    hd, theta, period = (float(v) for v in _rows("rope_period.txt")[0])
    cos, sin = synth.rope_tables(torch.tensor([1.0], dtype=torch.float64), theta)
    lowest = math.atan2(float(sin[0, -1]), float(cos[0, -1]))      # angle per token of the last pair
    assert round(2 * math.pi / lowest) == period
    # rotate-half pairing (i, i + d/2): rotating e_0 by position 1 moves energy into channel 64
    x = torch.zeros(1, 1, 128); x[0, 0, 0] = 1.0
    y = synth.apply_rope(x, torch.tensor([1]))
    assert abs(float(y[0, 0, 0]) - math.cos(1.0)) < 1e-6 and abs(float(y[0, 0, 64]) - math.sin(1.0)) < 1e-6


# ------------------------------------------------------------- bookkeeping ----
def _mk(fbit, max_tokens, n_stored=2, lam=None, **kw):
    pol = O.Policy(fbit, max_tokens, n_slices=n_stored, **kw)
    return pol, O.LayerOracle(pol, n_stored, lam=lam)


def test_cache_structure_after_appends():
    rng = np.random.default_rng(0)
    pol, lay = _mk(4, 600, n_sink=1, window=16)
    k = _bf16(rng.standard_normal((600, 2, 128)).astype(np.float32))
    v = _bf16(rng.standard_normal((600, 2, 128)).astype(np.float32))
    lay.append(k, v)
    assert pol.n_tokens == 600 and pol.cur_bits == 4 and lay.n_reduces == 2
    assert pol.bytes_used() <= pol.budget
    bits = lay.bits[:600]
    assert bits[0] == 16 and np.all(bits[1:584] == 4) and np.all(bits[584:] == 16)
    # body tokens equal the chain applied to a fresh INT16 quantization (shift timing is irrelevant)
    c16, s16, z16 = O.quantize_asym(k[:, 0], 16)
    c4, s4 = O.chain_to(c16[1:584], s16[1:584], 4)
    assert np.array_equal(lay.ck[0, 1:584], c4) and np.array_equal(lay.sk[0, 1:584], s4)
    assert np.array_equal(lay.zk[0, :600], z16)
    assert np.array_equal(lay.ck[0, 584:600], c16[584:])
    assert lay.ck[:, 1:584].max() <= 15


@pytest.mark.parametrize("chunk", [1, 16])
def test_bulk_append_equals_token_by_token(chunk):
    rng = np.random.default_rng(1)
    lam = rng.uniform(0.5, 4.0, (2, 128)).astype(np.float32)
    k = _bf16(rng.standard_normal((700, 2, 128)).astype(np.float32) * 3)
    v = _bf16(rng.standard_normal((700, 2, 128)).astype(np.float32))
    pa, la = _mk(2, 700, lam=lam, n_sink=1, window=32, evict_chunk=chunk)
    pb, lb = _mk(2, 700, lam=lam, n_sink=1, window=32, evict_chunk=chunk)
    la.append(k, v)
    lb.append_bulk(k[:300], v[:300]); lb.append_bulk(k[300:301], v[300:301]); lb.append_bulk(k[301:], v[301:])
    assert pa.cur_bits == pb.cur_bits == 2 and pa.n_tokens == pb.n_tokens
    for name in ("ck", "cv", "sk", "zk", "sv", "zv", "bits"):
        assert np.array_equal(getattr(la, name), getattr(lb, name)), name


def test_budget_full_and_capacity_errors():
    pol, lay = _mk(8, 64, n_sink=0, window=0, count_metadata=False)
    x = np.zeros((1, 2, 128), np.float32)
    for _ in range(32):
        lay.append(x, x, auto_reduce=False)
    with pytest.raises(BufferError):
        lay.append(x, x, auto_reduce=False)
    assert pol.n_tokens == 32 and pol.cur_bits == 16
    lay.reduce()
    for _ in range(32):
        lay.append(x, x, auto_reduce=False)
    with pytest.raises(OverflowError):
        lay.append(x, x)
    with pytest.raises(RuntimeError):
        lay.reduce()


# --------------------------------------------------------------- attention ----
def _filled(n, fbit=2, G=4, seed=0, lam=None, window=8, n_stored=1):
    rng = np.random.default_rng(seed)
    pol, lay = _mk(fbit, max(n, 1), n_stored=n_stored, lam=lam, n_sink=1, window=window)
    k = _bf16(rng.standard_normal((n, n_stored, 128)).astype(np.float32) * 2)
    v = _bf16(rng.standard_normal((n, n_stored, 128)).astype(np.float32))
    lay.append(k, v)
    q = _bf16(rng.standard_normal((n_stored, G, 128)).astype(np.float32))
    return pol, lay, k, v, q


def test_attention_single_token_returns_dequantized_value():
    pol, lay, k, v, q = _filled(1)
    out = lay.decode_attention(q)
    vhat = O.dequantize(lay.cv[0, :1], lay.sv[0, :1], lay.zv[0, :1])[0]
    assert np.array_equal(out[0], np.repeat(vhat[None], 4, 0).astype(np.float32))


def test_attention_zero_query_gives_mean_of_values():
    pol, lay, k, v, q = _filled(50)
    out = lay.decode_attention(np.zeros_like(q))
    vhat = O.dequantize(lay.cv[0, :50], lay.sv[0, :50], lay.zv[0, :50])
    assert np.allclose(out[0], vhat.mean(0)[None], rtol=0, atol=1e-6)


def test_attention_brute_force_loops():
    lam = np.random.default_rng(3).uniform(0.5, 3.0, (1, 128)).astype(np.float32)
    pol, lay, k, v, q = _filled(4, lam=lam, window=1)     # sink, 2 body tokens at 2 bit, 1 window token
    assert lay.bits[:4].tolist() == [16, 2, 2, 16]
    out = lay.decode_attention(q)
    for g in range(4):
        scores = []
        for t in range(4):
            acc = 0.0
            for i in range(128):
                khat = float(lay.sk[0, t]) * int(lay.ck[0, t, i]) + float(lay.zk[0, t])
                acc += float(q[0, g, i]) * float(lam[0, i]) * khat
            scores.append(acc / math.sqrt(128.0))
        mx = max(scores)
        w = [math.exp(s - mx) for s in scores]
        for i in range(0, 128, 17):
            o = sum(w[t] * (float(lay.sv[0, t]) * int(lay.cv[0, t, i]) + float(lay.zv[0, t])) for t in range(4)) / sum(w)
            assert abs(o - float(out[0, g, i])) < 1e-6


def test_attention_matches_library_sdpa_on_dequantized_values():
    lam = np.random.default_rng(4).uniform(0.5, 3.0, (2, 128)).astype(np.float32)
    pol, lay, k, v, q = _filled(300, fbit=4, G=7, lam=lam, n_stored=2, window=16)
    out = lay.decode_attention(q)
    for s in range(2):
        kh = torch.tensor(O.dequantize(lay.ck[s, :300], lay.sk[s, :300], lay.zk[s, :300]))
        vh = torch.tensor(O.dequantize(lay.cv[s, :300], lay.sv[s, :300], lay.zv[s, :300]))
        qs = torch.tensor(q[s].astype(np.float64) * lam[s].astype(np.float64)[None])
        ref = torch.nn.functional.scaled_dot_product_attention(qs[None], kh[None], vh[None])[0]
        assert np.allclose(out[s], ref.numpy(), rtol=0, atol=2e-6)


def test_equalization_invariance_with_power_of_two_lambda():
    """(Q Lambda)(K Lambda^-1)^T = Q K^T exactly when Lambda is a power of two per channel: the
    quantizer sees the same group up to exact scaling only if all channels share the factor, so
    use one factor per slice - codes are identical and outputs match the unscaled cache."""
    lam = np.full((1, 128), 4.0, np.float32)
    _, la, k, v, q = _filled(80, lam=None, seed=7)
    _, lb, _, _, _ = _filled(80, lam=lam, seed=7)
    assert np.array_equal(la.ck, lb.ck) and np.array_equal(la.sk, lb.sk * np.float32(4.0))
    assert np.allclose(la.decode_attention(q), lb.decode_attention(q), rtol=0, atol=1e-6)


def test_int16_tier_close_to_exact_attention_on_original_values():
    """While the cache is still 16 bit, attention differs from exact attention on the unquantized
    bf16 values only through the <= S/2 per-element error of Eq. 1-2."""
    rng = np.random.default_rng(11)
    lam = rng.uniform(0.5, 3.0, (1, 128)).astype(np.float32)
    pol, lay = _mk(16, 256, n_stored=1, lam=lam)
    k = _bf16(rng.standard_normal((256, 1, 128)).astype(np.float32) * 2)
    v = _bf16(rng.standard_normal((256, 1, 128)).astype(np.float32))
    q = _bf16(rng.standard_normal((1, 5, 128)).astype(np.float32))
    lay.append(k, v)
    assert pol.cur_bits == 16 and np.all(lay.bits[:256] == 16)
    out = lay.decode_attention(q)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q[0]).double()[None], torch.tensor(k[:, 0]).double()[None], torch.tensor(v[:, 0]).double()[None])[0]
    assert np.abs(out[0] - ref.numpy()).max() < 2e-4


def test_heads_are_independent():
    pol, lay, k, v, q = _filled(64, G=6)
    full = lay.decode_attention(q)
    q2 = q.copy(); q2[0, 3] = 0
    part = lay.decode_attention(q2)
    keep = [0, 1, 2, 4, 5]
    assert np.array_equal(full[0, keep], part[0, keep])
