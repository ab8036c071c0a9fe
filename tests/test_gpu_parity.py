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
    """Constant V groups (S = 0), zero K, zero Q, and a huge-range token.  With one token's values scaled by
    1000 the outputs reach O(1000) where that token has weight; the criterion for this one case is the
    stated tolerance relative to the largest output, max-abs <= 2e-3 * max(1, max |reference|), and the
    stated rel-L2."""
    n, kvh = 200, 1
    k, v = make_inputs(7, 0, n, 1, kvh)
    v[5] = 1.5; v[150] = -2.0          # constant groups: scale 0
    k[7] = 0.0
    v[9] = v[9] * 1000.0               # one token with a huge value range
    m = Mirror(1, 4, kvh, 1, n, [2], window=16, attention_path=attention_path)
    m.append(0, k, v)
    m.check_state(0)
    q = synth.make_q(7, 0, 0, 1, 4, n)
    for qq in (q, torch.zeros_like(q)):
        ref = m.oracles[0].decode_attention(qq.float().numpy().reshape(1, 4, 128))
        err, rel = m.check_attention(0, qq, max_abs=2e-3 * max(1.0, float(np.abs(ref).max())))
        print(f"degenerate values: max |ref| {np.abs(ref).max():.1f}, max-abs err {err:.2e}, rel-L2 {rel:.2e}")


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


def test_decode_step_tiny_caches_with_many_ctas(attention_path):
    """pmkvq_decode_step with the attention grid set to 1024 CTAs on caches far smaller than that: a 16-bit block
    of 8 tokens, and a 2- / 4-bit pair of 40 tokens.  Every slice must still be combined (each CTA between a
    slice's first and last owner publishes a partial) and a second step must find the tickets at zero."""
    for fbit, n0, window in (([16], 8, 4), ([2, 4], 40, 8)):
        layers, kvh, batch, group = len(fbit), 2, 1, 4
        m = Mirror(layers, group * kvh, kvh, batch, n0 + 2, fbit, window=window, attention_path=attention_path)
        for l in range(layers):
            k, v = make_inputs(51, l, n0, batch, kvh)
            m.append(l, k, v)
        m.cache.set_attention_ctas(1024)
        for s in range(2):
            ks, vs, qs = [], [], []
            for l in range(layers):
                k, v = make_inputs(52, l, 1, batch, kvh, pos0=n0 + s, chunk=s)
                ks.append(k[0]); vs.append(v[0])
                qs.append(synth.make_q(52, l, s, batch, group * kvh, n0 + s + 1))
            K, V, Q = torch.stack(ks).cuda(), torch.stack(vs).cuda(), torch.stack(qs).cuda()
            out = torch.full((layers, batch, group * kvh, 128), float("nan"), dtype=torch.float32, device="cuda")
            m.cache.decode_step(K, V, Q, out=out)
            torch.cuda.synchronize()
            for l in range(layers):
                m.oracles[l].append(K[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices],
                                    V[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices])
                ref = m.oracles[l].decode_attention(Q[l].float().cpu().numpy().reshape(batch * kvh, group, 128)[m.slices])
                got = out[l].cpu().numpy().reshape(batch * kvh, group, 128)[m.slices].astype(np.float64)
                assert np.all(np.isfinite(got)), "a slice was never combined"
                assert np.abs(got - ref).max() <= 2e-3 and np.linalg.norm(got - ref) <= 1e-3 * np.linalg.norm(ref)
        assert m.cache.device_status() == 0


def test_decode_step_capacity_leaves_every_block_untouched():
    """auto_reduce on: block 0 could take the step's token after a reduce, block 1 is at its final width and
    full.  The step fails with CAPACITY and nothing has happened: block 0 has NOT been reduced."""
    from paper_2505_18610_b200 import binding as B
    layers, kvh, batch, group = 2, 1, 1, 4
    full16 = 2 * 16 * 264                            # 16 INT16 tokens per (K|V) slice
    m = Mirror(layers, group * kvh, kvh, batch, 64, [8, 16], n_sink=0, window=0, budget_bytes=[full16, full16])
    k, v = make_inputs(53, 0, 17, batch, kvh)
    for l in range(layers):
        m.append(l, k[:16], v[:16])
    K = torch.stack([k[16], k[16]]).cuda().contiguous(); V = torch.stack([v[16], v[16]]).cuda().contiguous()
    Q = torch.stack([synth.make_q(53, l, 0, batch, group * kvh, 17) for l in range(layers)]).cuda().contiguous()
    with pytest.raises(B.PmkvqError) as e:
        m.cache.decode_step(K, V, Q)
    assert e.value.status == B.CAPACITY
    assert [m.cache.layer_state(l)["n_tokens"] for l in range(layers)] == [16, 16]
    assert [m.cache.layer_state(l)["cur_bits"] for l in range(layers)] == [16, 16]
    for l in range(layers):
        m.check_state(l)                              # bytes as well: nothing was reduced on the device either


def test_v_scales_spread_and_near_constant_token(attention_path):
    """V scales spread over 2^-12 .. 2^12 inside one slice, and a near-constant V token (range 1e-7 around 5)
    that carries most of the softmax mass, once inside the 2-bit body and once inside the INT16 window: the
    token's zero-point must reach the output although its codes weigh next to nothing."""
    n, kvh = 400, 1
    k, v = make_inputs(54, 0, n, 1, kvh)
    vf = v.float()
    for t in range(n):
        vf[t] *= 2.0 ** ((t * 7) % 25 - 12)
    q = synth.make_q(54, 0, 0, 1, 4, n)
    for t_special in (100, n - 3):
        kk, vv = k.clone(), vf.clone()
        vv[t_special] = 5.0 + 1e-7 * torch.arange(128, dtype=torch.float32).reshape(1, 1, 128) / 128.0
        kk[t_special] = (q[0, 0].float() * 6.0).to(kk.dtype)          # a Key aligned with head 0's Query: a dominant score
        m = Mirror(1, 4, kvh, 1, n, [2], window=16, attention_path=attention_path)
        m.append(0, kk, vv.to(v.dtype))
        m.check_state(0)
        ref = m.oracles[0].decode_attention(q.float().numpy().reshape(1, 4, 128))
        err, rel = m.check_attention(0, q, max_abs=2e-3 * max(1.0, float(np.abs(ref).max())))
        print(f"near-constant token at {t_special}: max |ref| {np.abs(ref).max():.1f}, err {err:.2e}, rel {rel:.2e}")


def test_sm_scale_and_lambda_extremes(attention_path):
    """A caller-chosen softmax scale and an equalization vector with entries of 1e-3 and 1e3, on Keys whose
    channels have those magnitudes (what Eq. 10 would produce for them): after K / lambda every channel is
    O(1) again, Q * lambda spans six decades, and the scale keeps the scores O(1)."""
    n, kvh, batch, group = 700, 2, 2, 5
    k, v = make_inputs(55, 0, n, batch, kvh)
    lam = np.ones((1, kvh, 128), np.float32)
    lam[0, :, ::7] = 1e-3
    lam[0, :, 3::11] = 1e3
    kf = k.float() * torch.from_numpy(lam[0]).reshape(1, 1, kvh, 128)
    k = kf.to(k.dtype)
    m = Mirror(1, group * kvh, kvh, batch, n, [2], lam=lam, window=32, sm_scale=2e-4, attention_path=attention_path)
    m.append(0, k, v)
    m.check_state(0)
    err, rel = m.check_attention(0, synth.make_q(55, 0, 0, batch, group * kvh, n))
    print(f"lambda 1e-3 .. 1e3, sm_scale 2e-4: max-abs err {err:.2e}, rel-L2 {rel:.2e}")


def test_guard_bands(attention_path):
    """No tool checks the kernels' addresses on this path, so this test does: the arena and a slack region behind
    it are filled with a pattern before the cache is created, a small cache then goes through bulk appends,
    300 decode steps with chunked eviction and all three progressive reduces, and afterwards every byte
    outside the regions the layout makes live must still hold the pattern: the slack past the arena, the part
    of every body stream beyond the most bytes the stream has ever held, and the split-K partial slots beyond
    the ones a launch can use.  All slices are compared with the oracle at the end."""
    PAT = 0xA5
    layers, kvh, batch, group, n0, steps, chunk = 2, 2, 2, 4, 200, 300, 4
    n_slices = batch * kvh
    fbit = [2, 4]
    n_max = n0 + steps                 # default budgets: the blocks cross 16 -> 8 -> 4 (-> 2) at about 100 / 170 / 290 tokens
    m = Mirror(layers, group * kvh, kvh, batch, n_max, fbit, window=32, evict_chunk=chunk,
               attention_path=attention_path, slack_bytes=1 << 20, fill_byte=PAT)
    lay = [m.cache.arena_layout(l) for l in range(layers)]
    high = np.zeros((layers, 8), np.int64)              # most bytes each stream has held so far

    def note(l):
        st = m.cache.layer_state(l)
        body = max(0, st["n_tokens"] - 1 - 32) // chunk * chunk
        tiles = (body + 15) // 16
        for s_ in range(8):
            cnt = (tiles - s_ + 7) // 8 if tiles > s_ else 0
            high[l, s_] = max(high[l, s_], cnt * (512 * st["cur_bits"] + 256))

    widths = [set() for _ in range(layers)]
    for l in range(layers):
        k, v = make_inputs(56, l, n0, batch, kvh)
        for a, b in ((0, 60), (60, 150), (150, n0)):
            m.append(l, k[a:b], v[a:b]); note(l); widths[l].add(m.cache.layer_state(l)["cur_bits"])
    for s in range(steps):
        ks, vs, qs = [], [], []
        for l in range(layers):
            k, v = make_inputs(57, l, 1, batch, kvh, pos0=n0 + s, chunk=s)
            ks.append(k[0]); vs.append(v[0])
            qs.append(synth.make_q(57, l, s, batch, group * kvh, n0 + s + 1))
        K, V, Q = torch.stack(ks).cuda(), torch.stack(vs).cuda(), torch.stack(qs).cuda()
        m.cache.decode_step(K, V, Q)
        for l in range(layers):
            m.oracles[l].append(K[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices],
                                V[l].float().cpu().numpy().reshape(1, -1, 128)[:, m.slices])
            note(l); widths[l].add(m.cache.layer_state(l)["cur_bits"])
    torch.cuda.synchronize()
    assert widths[0] == {16, 8, 4, 2} and widths[1] == {16, 8, 4}
    assert m.cache.device_status() == 0
    arena = m.cache.arena[m.cache.arena_offset:].cpu().numpy()
    used = lay[0]["arena_bytes"]
    assert (arena[used:] == PAT).all(), "bytes behind the arena were written"
    for l in range(layers):
        g = lay[l]
        for s_ in range(n_slices):
            base = g["offset"] + s_ * g["slice_stride"] + g["body_off"]
            for st_ in range(8):
                lo = base + st_ * g["stream_stride"] + int(high[l, st_])
                hi = base + (st_ + 1) * g["stream_stride"]
                assert (arena[lo:hi] == PAT).all(), f"block {l} slice {s_} stream {st_}: bytes beyond the stream's data were written"
            end = g["offset"] + s_ * g["slice_stride"] + g["body_off"] + 8 * g["stream_stride"]
            assert (arena[end:g["offset"] + (s_ + 1) * g["slice_stride"]] == PAT).all()
        # split-K workspace: a launch uses at most (CTAs + slices) partial slots; 148 CTAs at most by default
        first_unused = g["partials_off"] + (148 + n_slices) * g["partial_slot_bytes"]
        assert (arena[first_unused:g["partials_off"] + g["partials_bytes"]] == PAT).all()
    for l in range(layers):
        m.check_state(l)                                 # every slice, not a sample
        m.check_attention(l, synth.make_q(58, l, 0, batch, group * kvh, n_max))


def test_bounded_wait_gives_up_and_the_context_lives():
    """A barrier wait that nothing can satisfy runs out after its poll limit, the kernel reports it and ends;
    afterwards the same cache still computes attention, and its error word (the attention kernels' own waits)
    is clean.  Also: a checkpoint of the arena plus pmkvq_restore_layer_state brings a cache back."""
    from paper_2505_18610_b200 import binding as B
    kvh, batch, group, n = 2, 1, 4, 600
    k, v = make_inputs(61, 0, n, batch, kvh)
    m = Mirror(1, group * kvh, kvh, batch, n + 8, [2], window=16, attention_path=1)
    m.append(0, k, v)
    assert m.cache.selftest_bounded_wait() == 1
    q = synth.make_q(61, 0, 0, batch, group * kvh, n)
    m.check_attention(0, q)
    assert m.cache.device_status() == 0
    # checkpoint, move on, restore
    snap, st0 = m.cache.arena.clone(), m.cache.layer_state(0)
    before = m.cache.decode_attention(0, q.cuda()).clone()
    k2, v2 = make_inputs(62, 0, 8, batch, kvh, pos0=n)
    m.cache.append(0, k2.cuda().contiguous(), v2.cuda().contiguous())
    m.cache.arena.copy_(snap)
    m.cache.restore_layer_state(0, st0["n_tokens"], st0["cur_bits"])
    assert m.cache.layer_state(0) == st0
    assert torch.equal(m.cache.decode_attention(0, q.cuda()), before)
    with pytest.raises(B.PmkvqError):
        m.cache.restore_layer_state(0, 5, 1)        # not a width
