"""Parity at the full per-block sizes of the benchmark workloads (7B / 8B / 32B / 70B long-CoT shapes), in the launch
configuration bench.py times
(same batch, heads, context length, default attention grid, pmkvq_decode_step), on sampled (batch,
kv_head) slices the oracle can compute one by one: cache state bit-exact after the run (it crosses each
block's last progressive reduce), attention outputs within tolerance at several steps.  Two blocks per
case (one per Fbit of the schedule) keep the device footprint at a few GB,
so the per-block shapes are those of the full model (the step's one attention launch covers both blocks).  Every case runs on
both attention paths of the library."""
import numpy as np
import pytest
import torch

from oracle import pmkvq_oracle as O
from paper_2505_18610_b200 import synth
from paper_2505_18610_b200.binding import Cache
from tests.helpers import MAX_ABS_TOL, REL_L2_TOL, f32_bits

pytestmark = pytest.mark.gpu

N_SINK, WINDOW = 1, 128


def _bytes_at(n, bits, n_slices):
    nb = max(0, n - N_SINK - WINDOW)
    return 2 * n_slices * ((n - nb) * 264 + nb * (16 * bits + 8))


CASES = {
    # name: q_heads, kv_heads, batch, end tokens, Fbit of the two blocks, outlier channels, factor
    "7b_b16_32k": (28, 4, 16, 32768, [4, 2], 4, 15.0),
    "8b_b32_32k": (32, 8, 32, 32768, [4, 4], 4, 15.0),
    "32b_b8_128k": (40, 8, 8, 131072, [2, 4], 4, 15.0),
    "70b_b16_64k": (64, 8, 16, 65536, [4, 2], 4, 15.0),
}


@pytest.mark.parametrize("name", list(CASES))
def test_fullsize_sampled_slices(name, attention_path):
    q_heads, kvh, batch, n_end, fbit, n_out, factor = CASES[name]
    layers, steps, chunk = len(fbit), 6, 8192
    n_slices, group = batch * kvh, q_heads // kvh
    n0 = n_end - steps
    # block l is at 2*Fbit until its budget fills at step 2 + l: its last reduce happens inside the run
    budgets = [_bytes_at(n0 + 2 + l, min(16, 2 * fbit[l]), n_slices) for l in range(layers)]
    sample = sorted({0, n_slices // 2 + 1, n_slices - 1})
    dev = "cuda"
    lam = np.stack([synth.make_lambda(synth.make_kv(0, l, 0, 512, 1, kvh, 0, n_out, factor)[0]).numpy()
                    for l in range(layers)])
    cache = Cache(layers, q_heads, kvh, batch, n_end, fbit, budget_bytes=budgets, lam=lam, attention_path=attention_path)
    oracles = []
    for l in range(layers):
        pol = O.Policy(fbit[l], n_end, n_slices, budgets[l])
        orc = O.LayerOracle(pol, len(sample), lam=np.stack([lam[l, s % kvh] for s in sample]))
        done = 0
        while done < n0:
            n = min(chunk, n0 - done)
            k, v = synth.make_kv(0, l, done // chunk, n, batch, kvh, done, n_out, factor, device=dev)
            cache.append(l, k.contiguous(), v.contiguous())
            orc.append_bulk(k.reshape(n, n_slices, 128)[:, sample].float().cpu().numpy(),
                            v.reshape(n, n_slices, 128)[:, sample].float().cpu().numpy())
            done += n
        oracles.append(orc)
        assert cache.layer_state(l)["cur_bits"] == min(16, 2 * fbit[l])
    worst = (0.0, 0.0)
    for s in range(steps):
        ks, vs, qs = [], [], []
        for l in range(layers):
            k, v = synth.make_kv(1, l, s, 1, batch, kvh, n0 + s, n_out, factor, device=dev)
            ks.append(k[0]); vs.append(v[0])
            qs.append(synth.make_q(1, l, s, batch, q_heads, n0 + s, device=dev))
        K, V, Q = torch.stack(ks).contiguous(), torch.stack(vs).contiguous(), torch.stack(qs).contiguous()
        out = cache.decode_step(K, V, Q)
        torch.cuda.synchronize()
        for l in range(layers):
            oracles[l].append_bulk(K[l].reshape(1, n_slices, 128)[:, sample].float().cpu().numpy(),
                                   V[l].reshape(1, n_slices, 128)[:, sample].float().cpu().numpy())
            if s in (0, 2 + l, steps - 1):          # before, right after the block's reduce, at the end
                qq = Q[l].reshape(n_slices, group, 128)[sample].float().cpu().numpy()
                ref = oracles[l].decode_attention(qq)
                got = out[l].reshape(n_slices, group, 128)[sample].double().cpu().numpy()
                assert np.all(np.isfinite(got))
                err = float(np.abs(got - ref).max())
                rel = float(np.linalg.norm(got - ref) / np.linalg.norm(ref))
                worst = (max(worst[0], err), max(worst[1], rel))
                assert err <= MAX_ABS_TOL and rel <= REL_L2_TOL, (name, l, s, err, rel)
    for l in range(layers):
        st = cache.layer_state(l)
        orc = oracles[l]
        assert st["cur_bits"] == fbit[l] == orc.p.cur_bits and st["n_tokens"] == n_end == orc.p.n_tokens
        assert st["bytes_used"] == orc.p.bytes_used()
        for i, sl in enumerate(sample[:2]):
            b, h = divmod(sl, kvh)
            for is_v in (False, True):
                codes, scale, zero, bits = cache.export_slice(l, b, h, is_v)
                oc, osc, oz, ob = orc.export_slice(i, is_v)
                assert np.array_equal(bits, ob) and np.array_equal(codes, oc)
                assert np.array_equal(f32_bits(scale), f32_bits(osc)) and np.array_equal(f32_bits(zero), f32_bits(oz))
    print(f"{name}: worst max-abs {worst[0]:.2e}, worst rel-L2 {worst[1]:.2e}")
    cache.close()
