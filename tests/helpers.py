"""Shared helpers of the GPU parity tests: drive the CUDA cache and the CPU oracle with the same
seeded inputs and compare what each holds / returns."""
from __future__ import annotations

import numpy as np
import torch

from oracle import pmkvq_oracle as O
from paper_2505_18610_b200 import synth

MAX_ABS_TOL = 2e-3     # the stated tolerance on attention outputs
REL_L2_TOL = 1e-3


def f32_bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


class Mirror:
    """One CUDA cache plus, per layer, an oracle holding a chosen subset of (batch, kv_head) slices."""

    def __init__(self, layers, q_heads, kv_heads, batch, max_tokens, fbit, slices=None, lam=None,
                 budget_bytes=None, **kw):
        from paper_2505_18610_b200.binding import Cache
        self.layers, self.q_heads, self.kv_heads, self.batch = layers, q_heads, kv_heads, batch
        self.group = q_heads // kv_heads
        n_slices = batch * kv_heads
        self.slices = list(range(n_slices)) if slices is None else list(slices)
        self.lam = None if lam is None else np.asarray(lam, np.float32).reshape(layers, kv_heads, 128)
        self.cache = Cache(layers, q_heads, kv_heads, batch, max_tokens, fbit, budget_bytes=budget_bytes,
                           lam=self.lam, **kw)
        okw = {k: kw[k] for k in ("n_sink", "window", "evict_chunk", "count_metadata") if k in kw}
        variant = kw.get("shift_variant", 0)
        self.oracles = []
        for l in range(layers):
            pol = O.Policy(fbit[l], max_tokens, n_slices, None if budget_bytes is None else budget_bytes[l], **okw)
            lam_s = None if self.lam is None else np.stack([self.lam[l, s % kv_heads] for s in self.slices])
            self.oracles.append(O.LayerOracle(pol, len(self.slices), lam=lam_s, shift_variant=variant))
        self.sm_scale = kw.get("sm_scale") or None

    def append(self, layer, k, v, bulk=True):
        """k, v: CPU or CUDA bf16 [n, batch, kv_heads, 128]."""
        kd, vd = k.cuda().contiguous(), v.cuda().contiguous()
        self.cache.append(layer, kd, vd)
        n = k.shape[0]
        kk = k.float().cpu().numpy().reshape(n, -1, 128)[:, self.slices]
        vv = v.float().cpu().numpy().reshape(n, -1, 128)[:, self.slices]
        if bulk:
            self.oracles[layer].append_bulk(kk, vv)
        else:
            self.oracles[layer].append(kk, vv)

    def check_state(self, layer, slices=None):
        orc = self.oracles[layer]
        st = self.cache.layer_state(layer)
        assert st["n_tokens"] == orc.p.n_tokens and st["cur_bits"] == orc.p.cur_bits
        assert st["bytes_used"] == orc.p.bytes_used() and st["budget_bytes"] == orc.p.budget
        for si in (range(len(self.slices)) if slices is None else slices):
            s = self.slices[si]
            b, h = divmod(s, self.kv_heads)
            for is_v in (False, True):
                codes, scale, zero, bits, packed = self.cache.export_slice(layer, b, h, is_v, packed=True)
                oc, osc, oz, ob = orc.export_slice(si, is_v)
                assert np.array_equal(bits, ob), "token widths differ"
                assert np.array_equal(codes, oc), f"codes differ (layer {layer} slice {s} V={is_v})"
                assert np.array_equal(f32_bits(scale), f32_bits(osc)), "scales differ"
                assert np.array_equal(f32_bits(zero), f32_bits(oz)), "zero-points differ"
                want = np.concatenate([O.pack_canonical(oc[t], int(ob[t])) for t in range(len(ob))]) if len(ob) else np.zeros(0, np.uint8)
                assert np.array_equal(packed, want), "canonical packed bytes differ"

    def check_attention(self, layer, q, max_abs=MAX_ABS_TOL, rel_l2=REL_L2_TOL):
        """q: bf16 [batch, q_heads, 128] (CPU or CUDA).  Returns (max_abs_err, rel_l2_err)."""
        out = self.cache.decode_attention(layer, q.cuda().contiguous())
        torch.cuda.synchronize()
        got = out.cpu().numpy().reshape(self.batch * self.kv_heads, self.group, 128)[self.slices]
        qq = q.float().cpu().numpy().reshape(self.batch * self.kv_heads, self.group, 128)[self.slices]
        ref = self.oracles[layer].decode_attention(qq, sm_scale=self.sm_scale)
        assert np.all(np.isfinite(got)), "non-finite attention output"
        err = float(np.abs(got.astype(np.float64) - ref).max())
        rel = float(np.linalg.norm(got.astype(np.float64) - ref) / max(np.linalg.norm(ref), 1e-30))
        assert err <= max_abs, f"max abs err {err:.3e} > {max_abs}"
        assert rel <= rel_l2, f"rel L2 err {rel:.3e} > {rel_l2}"
        return err, rel


def make_inputs(seed, layer, n, batch, kv_heads, pos0=0, n_outlier=4, factor=15.0, chunk=0):
    return synth.make_kv(seed, layer, chunk, n, batch, kv_heads, pos0, n_outlier, factor)
