"""pmkvq_decode_attention_static: the attention call for hosts that cannot allocate device memory when
they call it (a pre-sized pool, frozen allocations, a loop that must not hit cudaMalloc's implicit
synchronisation).  Its split-K workspace is an array inside the library image, shared by every call on
the GPU, so the checks here are: same output as pmkvq_decode_attention and as the CPU oracle on two calls
in a row (the second one finds the first one's leftovers in the array), no device memory allocated or
freed across the calls, and a clean refusal beyond the array's size.
This file sorts last on purpose: a run that stops at the first failure has then run everything else."""
import numpy as np
import pytest
import torch

from oracle import pmkvq_oracle as O
from paper_2505_18610_b200 import binding as B
from paper_2505_18610_b200 import synth

pytestmark = pytest.mark.gpu

MAX_ABS_TOL, REL_L2_TOL = 2e-3, 1e-3     # the tolerances of the parity tests


def _close(a, b):
    a, b = a.double().cpu().numpy(), b.double().cpu().numpy()
    assert np.all(np.isfinite(a))
    assert np.abs(a - b).max() <= MAX_ABS_TOL
    assert np.linalg.norm(a - b) <= REL_L2_TOL * max(np.linalg.norm(b), 1e-30)


def test_static_scratch_matches_arena_scratch_twice_in_a_row():
    layers, kvh, group, batch, n = 2, 2, 7, 3, 1500
    fbit = [2, 4]
    ks, vs = zip(*[synth.make_kv(11, l, 0, n + 1, batch, kvh, 0, 4, 15.0) for l in range(layers)])
    lam = np.stack([synth.make_lambda(k[:256]).numpy() for k in ks])
    cache = B.Cache(layers, group * kvh, kvh, batch, n + 1, fbit, lam=lam)
    n_slices = batch * kvh
    oracles = []
    for l in range(layers):
        cache.append(l, ks[l][:n].cuda().contiguous(), vs[l][:n].cuda().contiguous())
        orc = O.LayerOracle(O.Policy(fbit[l], n + 1, n_slices), n_slices, lam=np.stack([lam[l, s % kvh] for s in range(n_slices)]))
        orc.append_bulk(ks[l][:n].float().numpy().reshape(n, n_slices, 128), vs[l][:n].float().numpy().reshape(n, n_slices, 128))
        oracles.append(orc)

    def oracle_out(l, q):
        ref = oracles[l].decode_attention(q.float().cpu().numpy().reshape(n_slices, group, 128))
        return torch.from_numpy(ref.reshape(batch, group * kvh, 128))

    out_static = torch.full((batch, group * kvh, 128), float("nan"), dtype=torch.float32, device="cuda")
    # first call: block 0 (2 bit)
    q0 = synth.make_q(11, 0, 0, batch, group * kvh, n).cuda()
    want = cache.decode_attention(0, q0)
    cache.decode_attention_static(0, q0, out_static)          # the first call on this GPU looks the array up
    torch.cuda.synchronize()
    _close(out_static, want)
    _close(out_static, oracle_out(0, q0))
    # no allocation: neither torch's allocator nor the device's free memory moves across a call
    out_static.fill_(float("nan"))
    torch.cuda.synchronize()
    stats0 = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    cache.decode_attention_static(0, q0, out_static)
    torch.cuda.synchronize()
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0]) == stats0
    _close(out_static, want)
    # second call right behind it, another block (4 bit), another grid shape, one more token: the array
    # still holds the first call's partials and tickets
    cache.append(1, ks[1][n:n + 1].cuda().contiguous(), vs[1][n:n + 1].cuda().contiguous())
    oracles[1].append_bulk(ks[1][n:n + 1].float().numpy().reshape(1, n_slices, 128), vs[1][n:n + 1].float().numpy().reshape(1, n_slices, 128))
    cache.set_attention_ctas(37)
    q1 = synth.make_q(11, 1, 1, batch, group * kvh, n + 1).cuda()
    out_static.fill_(float("nan"))
    cache.decode_attention_static(1, q1, out_static)
    want = cache.decode_attention(1, q1)
    torch.cuda.synchronize()
    _close(out_static, want)
    _close(out_static, oracle_out(1, q1))
    cache.close()


def test_static_scratch_refuses_what_it_cannot_hold():
    # 1200 slices need more partial slots than the 4 MiB array has; the arena-backed call still works
    batch = 1200
    cache = B.Cache(1, 1, 1, batch, 8, [16], window=0)
    k, v = synth.make_kv(12, 0, 0, 4, batch, 1, 0, 0, 1.0)
    cache.append(0, k.cuda().contiguous(), v.cuda().contiguous())
    q = synth.make_q(12, 0, 0, batch, 1, 4).cuda()
    out = torch.zeros(batch, 1, 128, dtype=torch.float32, device="cuda")
    assert cache.decode_attention_static(0, q, out, check=False) == B.SCRATCH_LIMIT
    assert float(out.abs().max()) == 0.0                      # nothing was launched
    assert torch.isfinite(cache.decode_attention(0, q)).all()
    cache.close()
