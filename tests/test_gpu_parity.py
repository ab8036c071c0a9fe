"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.
Codes, scales and zero-points bit-exact; attention outputs within max-abs 2e-3 and rel-L2 1e-3."""
import numpy as np
import pytest
import torch

from paper_2505_18610_b200 import synth
from tests.helpers import Mirror, make_inputs

pytestmark = pytest.mark.gpu


def _lam(layers, kv_heads, k_sample):
    return np.stack([synth.make_lambda(k_sample).numpy() for _ in range(layers)])


@pytest.mark.parametrize("fbit", [16, 8, 4, 2])
@pytest.mark.parametrize("n", [1, 2, 3, 17])
def test_tiny_token_counts(fbit, n, attention_path):
    """1-17 tokens, no window: sink + body at every width, brute-force sized."""
    k, v = make_inputs(1, 0, n, 1, 1)
    m = Mirror(1, 4, 1, 1, 64, [fbit], n_sink=1, window=0,
               budget_bytes=[2 * (264 + (n - 1) * (16 * fbit + 8))], attention_path=attention_path)     # exactly n tokens with the body at Fbit
    m.append(0, k, v, bulk=False)
    assert m.cache.layer_state(0)["cur_bits"] == (fbit if n > 1 else 16)
    m.check_state(0)
    m.check_attention(0, synth.make_q(1, 0, 0, 1, 4, n))


def test_config1_progressive_16_8_4(attention_path):
    """The small progressive case: 1 block, batch 1, 4 Q / 1 KV head, 4096 tokens fed one by one, 4 outlier channels
    x20, default budget for Fbit = 4: the block goes 16 -> 8 -> 4.  Full parity after every reduce."""
    n = 4096
    k, v = make_inputs(0, 0, n, 1, 1, n_outlier=4, factor=20.0)
    lam = _lam(1, 1, k[:512])
    m = Mirror(1, 4, 1, 1, n, [4], lam=lam, attention_path=attention_path)
    kd, vd = k.cuda(), v.cuda()
    seen = [16]
    for t in range(n):
        m.cache.append(0, kd[t:t + 1], vd[t:t + 1])
        bits = m.cache.layer_state(0)["cur_bits"]
        if bits != seen[-1] or t in (0, 128, 129, 130, 500, n - 1):
            # catch the oracle up token by token (literal process), then compare everything
            o = m.oracles[0]
            t0 = o.p.n_tokens
            o.append(k[t0:t + 1].float().numpy().reshape(-1, 1, 128), v[t0:t + 1].float().numpy().reshape(-1, 1, 128))
            if bits != seen[-1]:
                seen.append(bits)
            m.check_state(0)
            m.check_attention(0, synth.make_q(0, 0, t, 1, 4, t + 1))
    assert seen == [16, 8, 4]


@pytest.mark.parametrize("group", [1, 4, 5, 7, 8])
def test_gqa_groups(group, attention_path):
    kvh, batch, n = 2, 2, 333
    k, v = make_inputs(2, 0, n, batch, kvh)
    m = Mirror(1, group * kvh, kvh, batch, 400, [2], lam=_lam(1, kvh, k[:64]), window=32, attention_path=attention_path)
    m.append(0, k, v)
    m.check_state(0)
    m.check_attention(0, synth.make_q(2, 0, 0, batch, group * kvh, n))


@pytest.mark.parametrize("fbit,chunk,n_sink,window", [(2, 1, 1, 128), (4, 16, 1, 128), (2, 16, 0, 32), (8, 3, 4, 20),
                                                     (2, 1, 0, 0), (4, 1, 17, 5)])
def test_multi_layer_bulk_and_stepwise(fbit, chunk, n_sink, window, attention_path):
    """Several blocks / slices, ragged bulk appends followed by single-token decode steps."""
    layers, kvh, batch, group, n_max = 2, 2, 3, 7, 1500
    m = None
    ks, vs = [], []
    for l in range(layers):
        k, v = make_inputs(3, l, n_max, batch, kvh)
        ks.append(k); vs.append(v)
    lam = np.stack([synth.make_lambda(ks[l][:256]).numpy() for l in range(layers)])
    m = Mirror(layers, group * kvh, kvh, batch, n_max, [fbit, 16 if fbit == 16 else max(fbit, 4)], lam=lam,
               n_sink=n_sink, window=window, evict_chunk=chunk, attention_path=attention_path)
    cuts = [0, 1, 130, 131, 700, 1237, 1400]
    for l in range(layers):
        for a, b in zip(cuts[:-1], cuts[1:]):
            m.append(l, ks[l][a:b], vs[l][a:b])
        m.check_state(l, slices=[0, 3, 5])
        m.check_attention(l, synth.make_q(3, l, 0, batch, group * kvh, cuts[-1]))
    for t in range(cuts[-1], cuts[-1] + 40):
        for l in range(layers):
            m.append(l, ks[l][t:t + 1], vs[l][t:t + 1])
            if t % 13 == 0:
                m.check_attention(l, synth.make_q(3, l, t, batch, group * kvh, t + 1))
    for l in range(layers):
        m.check_state(l, slices=[1, 4])


def test_policy_thresholds_on_gpu(attention_path):
    """Code-bit accounting, no sink / window, Fbit = 2, 512 max tokens: reduces at 64, 128, 256 tokens."""
    n = 512
    k, v = make_inputs(4, 0, n, 1, 2)
    m = Mirror(1, 8, 2, 1, n, [2], n_sink=0, window=0, count_metadata=False, attention_path=attention_path)
    kd, vd = k.cuda(), v.cuda()
    fired, bits = [], 16
    for t in range(n):
        m.cache.append(0, kd[t:t + 1], vd[t:t + 1])
        b = m.cache.layer_state(0)["cur_bits"]
        if b != bits:
            fired.append(t); bits = b
    assert fired == [64, 128, 256]
    m.oracles[0].append(k.float().numpy().reshape(n, 2, 128), v.float().numpy().reshape(n, 2, 128))
    m.check_state(0)
    m.check_attention(0, synth.make_q(4, 0, 0, 1, 8, n))


def test_manual_reduce_and_error_codes():
    from paper_2505_18610_b200 import binding as B
    k, v = make_inputs(5, 0, 80, 1, 1)
    m = Mirror(1, 4, 1, 1, 64, [8], n_sink=0, window=0, count_metadata=False, auto_reduce=False)
    kd, vd = k.cuda(), v.cuda()
    for t in range(32):
        assert m.cache.append(0, kd[t:t + 1], vd[t:t + 1], check=False) == B.OK
    assert m.cache.append(0, kd[32:33], vd[32:33], check=False) == B.BUDGET_FULL
    assert m.cache.layer_state(0) == {"n_tokens": 32, "cur_bits": 16, "bytes_used": 32 * 512, "budget_bytes": 64 * 256}
    assert m.cache.progressive_reduce(0, check=False) == B.OK
    assert m.cache.progressive_reduce(0, check=False) == B.AT_FBIT
    for t in range(32, 64):
        assert m.cache.append(0, kd[t:t + 1], vd[t:t + 1], check=False) == B.OK
    assert m.cache.append(0, kd[64:65], vd[64:65], check=False) == B.CAPACITY
    assert m.cache.append(5, kd[:1], vd[:1], check=False) == B.INVALID_ARG
    o = m.oracles[0]
    o.append(k[:32].float().numpy().reshape(32, 1, 128), v[:32].float().numpy().reshape(32, 1, 128), auto_reduce=False)
    o.reduce()
    o.append(k[32:64].float().numpy().reshape(32, 1, 128), v[32:64].float().numpy().reshape(32, 1, 128), auto_reduce=False)
    m.check_state(0)
    m.check_attention(0, synth.make_q(5, 0, 0, 1, 4, 64))
    with pytest.raises(B.PmkvqError):
        B.Cache(1, 4, 1, 1, 64, [3])
    with pytest.raises(B.PmkvqError):
        B.Cache(1, 18, 2, 1, 64, [4])          # GQA group of 9 is outside 1..8


def test_reduce_head_batches_and_waves(attention_path):
    """Bodies of 378, 733 and 1385 tiles cross 16 -> 8 -> 4 -> 2: the in-place reduce runs its CTA-wide head
    batches (256 tiles) and one, two and three parallel waves behind them."""
    kvh, n_max = 2, 40000
    m = Mirror(1, 2 * kvh, kvh, 1, n_max, [2], attention_path=attention_path)
    done, widths = 0, []
    for upto in (6170, 6200, 11855, 11900, 22279, 22400):
        k, v = make_inputs(31, 0, upto - done, 1, kvh, pos0=done, chunk=upto)
        m.append(0, k, v)
        done = upto
        widths.append(m.cache.layer_state(0)["cur_bits"])
        if upto in (6200, 11900, 22400):
            m.check_state(0)
    assert widths == [16, 8, 8, 4, 4, 2]
    m.check_attention(0, synth.make_q(31, 0, 0, 1, 2 * kvh, done))


def test_empty_inputs_are_refused_and_empty_bodies_reduce():
    from paper_2505_18610_b200 import binding as B
    m = Mirror(2, 4, 1, 1, 64, [4, 4], n_sink=1, window=8, auto_reduce=False)
    q = synth.make_q(41, 0, 0, 1, 4, 1).cuda()
    with pytest.raises(B.PmkvqError):                       # no cached token: no softmax to take
        m.cache.decode_attention(0, q)
    k, v = make_inputs(41, 0, 3, 1, 1)
    lib = B.lib()
    assert lib.pmkvq_append(m.cache._h, 0, k.cuda().data_ptr(), v.cuda().data_ptr(), 0, None) == B.INVALID_ARG
    assert m.cache.layer_state(0)["n_tokens"] == 0
    K = torch.zeros(2, 1, 1, 128, dtype=torch.bfloat16, device="cuda")
    m.append(0, k, v)                                       # block 1 stays empty
    assert m.cache.progressive_reduce(1, check=False) == B.OK       # an empty body reduces to nothing, the width moves
    m.oracles[1].reduce()
    assert m.cache.layer_state(1)["cur_bits"] == 8 and m.cache.layer_state(0)["cur_bits"] == 16
    m.check_state(0)
    m.check_attention(0, synth.make_q(41, 0, 1, 1, 4, 3))
    # a step needs every block's token: it appends to both and attends over 4 and 1 tokens
    out = m.cache.decode_step(K, K, torch.stack([q, q]))
    torch.cuda.synchronize()
    assert m.cache.layer_state(1)["n_tokens"] == 1 and m.cache.layer_state(0)["n_tokens"] == 4
    assert torch.isfinite(out).all()


def test_split_invariance(attention_path):
    kvh, batch, n, group = 2, 2, 5000, 8
    k, v = make_inputs(6, 0, n, batch, kvh)
    m = Mirror(1, group * kvh, kvh, batch, n, [2], lam=_lam(1, kvh, k[:256]), attention_path=attention_path)
    m.append(0, k, v)
    q = synth.make_q(6, 0, 0, batch, group * kvh, n)
    outs = []
    for s in (1, 2, 3, 7, 64, 333, 1024, 0):
        m.cache.set_attention_ctas(s)
        m.check_attention(0, q)
        outs.append(m.cache.decode_attention(0, q.cuda()).cpu().numpy())
    # partitions differ by fp32 summation order and by the fp16 rounding of p * S_V (2^-12 relative per
    # token, the reference m it is taken against depends on the partition): half the output tolerance
    for o in outs[1:]:
        assert np.abs(o - outs[0]).max() < 1e-3


def test_degenerate_values(attention_path):
    """Constant V groups (S = 0), zero K, zero Q, and a huge-range token."""
    n, kvh = 200, 1
    k, v = make_inputs(7, 0, n, 1, kvh)
    v[5] = 1.5; v[150] = -2.0          # constant groups: scale 0
    k[7] = 0.0
    v[9] = v[9] * 1000.0               # one token with a huge value range
    m = Mirror(1, 4, kvh, 1, n, [2], window=16, attention_path=attention_path)
    m.append(0, k, v)
    m.check_state(0)
    q = synth.make_q(7, 0, 0, 1, 4, n)
    m.check_attention(0, q, max_abs=2e-3 * 50)    # outputs reach O(1000) with the scaled token
    q0 = torch.zeros_like(q)
    m.check_attention(0, q0, max_abs=2e-3 * 50)


@pytest.mark.parametrize("bulk", [True, False])
def test_quantizer_scale_extremes(bulk, attention_path):
    """Tokens whose scale lies outside the range of the reciprocal-based quotient (below 2^-60, above 2^60,
    exactly 0) take the plain-division path; codes, scales and zero-points stay bit-exact."""
    n, kvh = 100, 2
    k, v = make_inputs(11, 0, n, 1, kvh)
    for t, f in ((3, 1e-30), (20, 1e30), (37, 1e-36), (64, 3e25)):
        k[t] = (k[t].float() * f).to(k.dtype)
        v[t] = (v[t].float() * f).to(v.dtype)
    k[50] = 0.25; v[51] = 0.0
    m = Mirror(1, 2, kvh, 1, n, [4], window=8, attention_path=attention_path)
    m.append(0, k, v, bulk=bulk)
    m.check_state(0)


def test_decode_step_over_all_blocks(attention_path):
    """pmkvq_decode_step = append + attention for every block; compared with the oracle block by block,
    across a reduce (block 0 crosses its budget during the steps)."""
    layers, kvh, batch, group, n0, steps = 3, 2, 2, 7, 300, 24
    fbit = [2, 4, 8]
    m = Mirror(layers, group * kvh, kvh, batch, n0 + steps, fbit, window=32, attention_path=attention_path)
    for l in range(layers):
        k, v = make_inputs(8, l, n0, batch, kvh)
        m.append(l, k, v)
    for s in range(steps):
        ks, vs, qs = [], [], []
        for l in range(layers):
            k, v = make_inputs(9, l, 1, batch, kvh, pos0=n0 + s, chunk=s)
            ks.append(k[0]); vs.append(v[0])
            qs.append(synth.make_q(9, l, s, batch, group * kvh, n0 + s + 1))
        K, V, Q = torch.stack(ks).cuda(), torch.stack(vs).cuda(), torch.stack(qs).cuda()
        m.cache.set_attention_ctas((0, 1, 7, 333, 1024)[s % 5])      # the one-launch step under several splits
        out = m.cache.decode_step(K, V, Q)
        torch.cuda.synchronize()
        for l in range(layers):
            kk = K[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices]
            vv = V[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices]
            m.oracles[l].append(kk, vv)
            if s % 3 == 0 or s == steps - 1:
                qq = Q[l].float().cpu().numpy().reshape(batch * kvh, group, 128)[m.slices]
                ref = m.oracles[l].decode_attention(qq)
                got = out[l].cpu().numpy().reshape(batch * kvh, group, 128)[m.slices].astype(np.float64)
                assert np.abs(got - ref).max() <= 2e-3
                assert np.linalg.norm(got - ref) <= 1e-3 * np.linalg.norm(ref)
    for l in range(layers):
        m.check_state(l)
        assert m.cache.layer_state(l)["cur_bits"] == fbit[l]


@pytest.mark.parametrize("layers", [128, 130])
def test_decode_step_with_many_blocks(layers, attention_path):
    """128 blocks fill the argument tables of the one-launch step exactly; 130 take the block-by-block route."""
    kvh, batch, group, n0, steps = 1, 1, 2, 40, 3
    fbit = [(2, 4, 8, 16)[l % 4] for l in range(layers)]
    m = Mirror(layers, group * kvh, kvh, batch, n0 + steps, fbit, window=8, attention_path=attention_path)
    for l in range(layers):
        k, v = make_inputs(21, l, n0, batch, kvh)
        m.append(l, k, v)
    for s in range(steps):
        ks, vs, qs = [], [], []
        for l in range(layers):
            k, v = make_inputs(22, l, 1, batch, kvh, pos0=n0 + s, chunk=s)
            ks.append(k[0]); vs.append(v[0])
            qs.append(synth.make_q(22, l, s, batch, group * kvh, n0 + s + 1))
        K, V, Q = torch.stack(ks).cuda(), torch.stack(vs).cuda(), torch.stack(qs).cuda()
        out = m.cache.decode_step(K, V, Q)
        torch.cuda.synchronize()
        for l in range(layers):
            m.oracles[l].append(K[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices],
                                V[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices])
            if s == steps - 1 and l in (0, 1, 2, 3, 63, layers - 2, layers - 1):
                qq = Q[l].float().cpu().numpy().reshape(batch * kvh, group, 128)[m.slices]
                ref = m.oracles[l].decode_attention(qq)
                got = out[l].cpu().numpy().reshape(batch * kvh, group, 128)[m.slices].astype(np.float64)
                assert np.abs(got - ref).max() <= 2e-3
                assert np.linalg.norm(got - ref) <= 1e-3 * np.linalg.norm(ref)
    for l in (0, 5, 127, layers - 1):
        m.check_state(l)


@pytest.mark.parametrize("variant", [1, 2])
def test_shift_variants_direct_and_modified(variant, attention_path):
    """The two ablation strategies of Sec. 4.4.1 as cache options: bulk appends, evictions through the
    chain and progressive reduces down to 2 bit, state bit-exact and attention within tolerance."""
    layers, kvh, batch, group, n = 2, 2, 2, 4, 900
    m = Mirror(layers, group * kvh, kvh, batch, n, [2, 4], window=32, shift_variant=variant, attention_path=attention_path)
    for l in range(layers):
        k, v = make_inputs(10 + variant, l, n, batch, kvh)
        m.append(l, k[:500], v[:500])
        for t in range(500, 560):
            m.append(l, k[t:t + 1], v[t:t + 1], bulk=False)
        m.append(l, k[560:], v[560:])
        m.check_state(l)
        assert m.cache.layer_state(l)["cur_bits"] == [2, 4][l]
        m.check_attention(l, synth.make_q(10, l, 0, batch, group * kvh, n))


def test_decode_step_budget_full_leaves_every_block_untouched():
    """With auto_reduce off, a step that would push one block over its budget returns BUDGET_FULL before any
    block has received its token; after the manual reduce the same step goes through."""
    from paper_2505_18610_b200 import binding as B
    layers, kvh, batch, group = 2, 1, 1, 4
    full = 2 * (16 * 264 + 0)                       # 16 INT16 tokens per (K|V) slice, code + metadata bytes
    m = Mirror(layers, group * kvh, kvh, batch, 64, [8, 8], n_sink=0, window=0, auto_reduce=False,
               budget_bytes=[full * 4, full])      # block 1 is full at 16 tokens, block 0 is not
    k, v = make_inputs(21, 0, 17, batch, kvh)
    for l in range(layers):
        m.cache.append(l, k[:16].cuda(), v[:16].cuda())
    K = torch.stack([k[16], k[16]]).cuda().contiguous(); V = torch.stack([v[16], v[16]]).cuda().contiguous()
    Q = torch.stack([synth.make_q(21, l, 0, batch, group * kvh, 17) for l in range(layers)]).cuda().contiguous()
    with pytest.raises(B.PmkvqError) as e:
        m.cache.decode_step(K, V, Q)
    assert e.value.status == B.BUDGET_FULL
    assert [m.cache.layer_state(l)["n_tokens"] for l in range(layers)] == [16, 16]
    assert [m.cache.layer_state(l)["cur_bits"] for l in range(layers)] == [16, 16]
    m.cache.progressive_reduce(1)
    out = m.cache.decode_step(K, V, Q)
    torch.cuda.synchronize()
    assert [m.cache.layer_state(l)["n_tokens"] for l in range(layers)] == [17, 17]
    assert [m.cache.layer_state(l)["cur_bits"] for l in range(layers)] == [16, 8]
    assert torch.isfinite(out).all()


@pytest.mark.parametrize("chunk,n_sink,window", [(16, 4, 20), (3, 0, 7), (1, 17, 0)])
def test_decode_step_with_chunked_eviction(chunk, n_sink, window, attention_path):
    """The all-blocks append of pmkvq_decode_step with eviction in chunks, several sink tokens and small
    windows: blocks at different token counts are not supported by the call, different widths are."""
    layers, kvh, batch, group, n0, steps = 2, 2, 2, 5, 70, 45
    m = Mirror(layers, group * kvh, kvh, batch, n0 + steps, [2, 8], n_sink=n_sink, window=window, evict_chunk=chunk, attention_path=attention_path)
    for l in range(layers):
        k, v = make_inputs(30, l, n0, batch, kvh)
        m.append(l, k, v)
    for s in range(steps):
        ks, vs, qs = [], [], []
        for l in range(layers):
            k, v = make_inputs(31, l, 1, batch, kvh, pos0=n0 + s, chunk=s)
            ks.append(k[0]); vs.append(v[0])
            qs.append(synth.make_q(31, l, s, batch, group * kvh, n0 + s + 1))
        K, V, Q = torch.stack(ks).cuda(), torch.stack(vs).cuda(), torch.stack(qs).cuda()
        out = m.cache.decode_step(K, V, Q)
        torch.cuda.synchronize()
        for l in range(layers):
            m.oracles[l].append(K[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices],
                                V[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices])
        if s % 11 == 0 or s == steps - 1:
            for l in range(layers):
                m.check_state(l)
                qq = Q[l].float().cpu().numpy().reshape(batch * kvh, group, 128)[m.slices]
                ref = m.oracles[l].decode_attention(qq)
                got = out[l].cpu().numpy().reshape(batch * kvh, group, 128)[m.slices].astype(np.float64)
                assert np.abs(got - ref).max() <= 2e-3 and np.linalg.norm(got - ref) <= 1e-3 * np.linalg.norm(ref)
