#!/usr/bin/env python
"""Benchmark of the PM-KVQ decode hot path on B200.

A "step" is one decode step of the whole model's attention path: for every transformer block,
quantize-on-append of one new token per sequence (with window eviction and, when the block's
budget fills, the progressive reduce) followed by fused dequantize + GQA decode attention over the
whole mixed-precision cache.  There are no weights / MLP in this path.

Default workload: 7B long-CoT shape, 28 blocks, 28 Q / 4 KV heads, head_dim
128, batch 16, 32K cached tokens at the end of the run, Fbit 4 in the first/last 4 blocks and 2
elsewhere; budgets are set so every block's last reduce (2*Fbit -> Fbit) falls inside the run.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload 7b|8b|tiny]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_18610_b200 import synth  # noqa: E402

WORKLOADS = {
    # name: layers, q_heads, kv_heads, batch, end tokens, (edge Fbit, inner Fbit, n_edge), outliers, factor
    "7b": dict(name="7b_longcot_b16_32k", layers=28, q_heads=28, kv_heads=4, batch=16,
               end_tokens=32768, edge_bits=4, inner_bits=2, n_edge=4, n_outlier=4, factor=15.0),
    "8b": dict(name="8b_b32_32k_uniform4", layers=32, q_heads=32, kv_heads=8, batch=32,
               end_tokens=32768, edge_bits=4, inner_bits=4, n_edge=4, n_outlier=4, factor=15.0),
    "32b": dict(name="32b_b8_128k_mixed_2_4", layers=64, q_heads=40, kv_heads=8, batch=8,
                end_tokens=131072, edge_bits=4, inner_bits=2, n_edge=16, n_outlier=4, factor=15.0),
    "70b": dict(name="70b_b16_64k_120GB", layers=80, q_heads=64, kv_heads=8, batch=16,
                end_tokens=65536, schedule="70b", n_outlier=4, factor=15.0),
    "7b-4l": dict(name="7b_longcot_b16_32k, 4 of 28 blocks (profiling case)", layers=4, q_heads=28, kv_heads=4, batch=16,
                  end_tokens=32768, edge_bits=4, inner_bits=2, n_edge=1, n_outlier=4, factor=15.0),
    "tiny": dict(name="tiny_smoke", layers=2, q_heads=8, kv_heads=2, batch=2, end_tokens=2048, edge_bits=4,
                 inner_bits=2, n_edge=1, n_outlier=4, factor=15.0),
}
N_SINK, WINDOW = 1, 128


def tokbytes(bits):
    return 16 * bits + 8


def bytes_at(n, bits, n_slices):
    nb = max(0, n - N_SINK - WINDOW)
    return 2 * n_slices * ((n - nb) * tokbytes(16) + nb * tokbytes(bits))


def plan(wl, steps, warmup):
    """Prefill length, per-block Fbit and budgets such that block l's last reduce fires inside the
    timed steps (staggered over the blocks)."""
    L, n_slices = wl["layers"], wl["batch"] * wl["kv_heads"]
    n0 = wl["end_tokens"] - steps - warmup
    assert n0 > N_SINK + WINDOW + 16, "too many steps for this workload"
    budgets = []
    if wl.get("schedule") == "70b":
        # a ~120 GB cache whose blocks sit at different points of the 16 -> 8 -> 4 -> 2 chain: 8 blocks
        # cross 16 -> 8 during the run, 16 cross 8 -> 4, 30 cross 4 -> 2, the other 26 are already at 2 bit
        fbit, crossing = [], []
        for l in range(L):
            fbit.append(8 if l >= L - 8 else 4 if l >= L - 24 else 2)
            crossing.append(l >= L - 54)
        k = 0
        for l in range(L):
            if crossing[l]:
                fire_step = warmup + (k * steps) // 54
                budgets.append(bytes_at(n0 + fire_step, 2 * fbit[l], n_slices)); k += 1
            else:
                budgets.append(bytes_at(wl["end_tokens"], fbit[l], n_slices))
        return fbit, budgets, n0
    fbit = synth.bit_schedule(L, wl["edge_bits"], wl["inner_bits"], wl["n_edge"])
    for l in range(L):
        fire_step = warmup + (l * steps) // L          # timed-region step at which block l reduces
        n_star = n0 + fire_step                        # cache holds n_star tokens at 2*Fbit; the next append reduces
        budgets.append(bytes_at(n_star, 2 * fbit[l], n_slices))
    return fbit, budgets, n0


def make_lambda(wl, seed, device):
    lam = []
    for l in range(wl["layers"]):
        k, _ = synth.make_kv(seed, l, 0, 512, 1, wl["kv_heads"], 0, wl["n_outlier"], wl["factor"], device=device)
        lam.append(synth.make_lambda(k).numpy())
    return np.stack(lam)


def build_cache(wl, fbit, budgets, lam, n0, device, chunk=8192, seed=0, shared_chunks=False, attention_path=0,
                max_tokens=None):
    """Prefill a cache of the workload's shape with n0 tokens per block.  With shared_chunks every block
    receives the same seeded chunk (the per-width and compact records: timing does not depend on the values)."""
    from paper_2505_18610_b200.binding import Cache
    cache = Cache(wl["layers"], wl["q_heads"], wl["kv_heads"], wl["batch"], max_tokens or wl["end_tokens"], fbit,
                  budget_bytes=budgets, lam=lam, n_sink=N_SINK, window=WINDOW, device=device,
                  attention_path=attention_path)
    if shared_chunks:
        done = 0
        while done < n0:
            n = min(chunk, n0 - done)
            k, v = synth.make_kv(seed, 0, done // chunk, n, wl["batch"], wl["kv_heads"], done, wl["n_outlier"],
                                 wl["factor"], device=device)
            k, v = k.contiguous(), v.contiguous()
            for l in range(wl["layers"]):
                cache.append(l, k, v)
            done += n
    else:
        for l in range(wl["layers"]):
            done = 0
            while done < n0:
                n = min(chunk, n0 - done)
                k, v = synth.make_kv(seed, l, done // chunk, n, wl["batch"], wl["kv_heads"], done, wl["n_outlier"],
                                     wl["factor"], device=device)
                cache.append(l, k.contiguous(), v.contiguous())
                done += n
    torch.cuda.synchronize()
    return cache


def step_inputs(wl, n_pool, seed, device, pos):
    """A pool of per-step inputs: K, V [pool, L, 1, B, Hkv, 128] and Q [pool, L, B, Hq, 128], bf16."""
    ks, vs, qs = [], [], []
    for i in range(n_pool):
        kl, vl, ql = [], [], []
        for l in range(wl["layers"]):
            k, v = synth.make_kv(seed + 1, l, i, 1, wl["batch"], wl["kv_heads"], pos + i, wl["n_outlier"], wl["factor"],
                                 device=device)
            kl.append(k); vl.append(v)
            ql.append(synth.make_q(seed + 1, l, i, wl["batch"], wl["q_heads"], pos + i, device=device))
        ks.append(torch.stack(kl)); vs.append(torch.stack(vl)); qs.append(torch.stack(ql))
    return torch.stack(ks).contiguous(), torch.stack(vs).contiguous(), torch.stack(qs).contiguous()


def step_bytes(cache, wl, bits_before):
    """Algorithmic bytes of the step that just ran (state after the step), per block summed:
    attention (codes + scale + zero of every token, Q, out, lambda) + append + eviction + reduce."""
    n_slices = wl["batch"] * wl["kv_heads"]
    total = 0
    for l in range(wl["layers"]):
        st = cache.layer_state(l)
        total += cache.attention_bytes(l)
        total += 2 * n_slices * (256 + tokbytes(16))                           # bf16 in, INT16 token out
        total += 2 * n_slices * (tokbytes(16) + tokbytes(st["cur_bits"]))      # one token leaves the window
        if st["cur_bits"] != bits_before[l]:                                   # a reduce fired in this step
            b = st["cur_bits"]
            nb = max(0, st["n_tokens"] - 1 - N_SINK - WINDOW)
            total += 2 * n_slices * nb * (16 * 2 * b + 16 * b + 8)
        bits_before[l] = st["cur_bits"]
    return total


def max_over_ranks(times, dist, device):
    """Every rank's device-side times -> the slowest rank's, on every rank (all-reduce MAX).  The data
    path has no collective: ranks hold disjoint batch shards and only their timings meet here."""
    if dist is None:
        return [float(t) for t in times]
    t = torch.tensor([float(x) for x in times], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(units_per_rank, world, ms):
    """Weak scaling: every rank processes `units_per_rank`; the job's rate is all of them over the
    slowest rank's time."""
    return world * units_per_rank / (ms * 1e-3)


def kernel_source_digest():
    """sha256 over the sources the attention kernel is compiled from (its own file and the two it includes):
    the ncu traffic figure below is only quoted for the kernel it was measured on."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2505_18610_b200", "csrc")
    for f in ("kernels_attn.cuh", "kernels_attn_tc.cuh", "tc05.cuh", "kernels_cache.cuh", "layout.cuh"):
        with open(os.path.join(d, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


# DRAM read + write bytes of one captured launch of the all-blocks attention kernel (ncu, 4 blocks of the 7B shape
# at their final widths: a launch of the 28-block workload moves 7x the bytes, block by block the same way), its
# algorithmic bytes, and the digest of the sources it was taken on.
NCU_TRAFFIC = {"digest": "56db185c15984adb", "traffic_bytes": 977_199_872, "algorithmic_bytes": 954_646_528}


def time_attention_all(cache, q, out, launches, warm=3):
    """CUDA-event time of `launches` calls of pmkvq_decode_attention_all (one attention launch over all blocks,
    nothing appended) on the current stream.  Returns the list of per-launch milliseconds."""
    for _ in range(warm):
        cache.decode_attention_all(q, out)
    torch.cuda.synchronize()
    evs = []
    for _ in range(launches):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); cache.decode_attention_all(q, out); e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


def width_leg(wl, device, peak, blocks=None, launches=12):
    """Steady-state attention at one width: caches of the workload's shape (all its blocks) whose whole body
    sits at 2 / 4 / 8 / 16 bit, timed with one all-blocks attention launch per event pair."""
    out = {}
    blocks = blocks or wl["layers"]
    sub = dict(wl, layers=blocks)
    for path, pname in ((0, "warp_mma"), (1, "tensor_memory")):
        for bits in (2, 4, 8, 16):
            if path == 1 and bits > 4:
                continue                      # the two paths only differ at 4 and 2 bit
            cache = build_cache(sub, [bits] * blocks, None, None, wl["end_tokens"], device, shared_chunks=True,
                                attention_path=path)
            assert all(cache.layer_state(l)["cur_bits"] == bits for l in range(blocks))
            q = torch.stack([synth.make_q(2, l, 0, wl["batch"], wl["q_heads"], wl["end_tokens"], device=device)
                             for l in range(blocks)]).contiguous()
            o = torch.empty(blocks, wl["batch"], wl["q_heads"], 128, dtype=torch.float32, device=device)
            ts = time_attention_all(cache, q, o, launches)
            by = sum(cache.attention_bytes(l) for l in range(blocks))
            ms = float(np.median(ts))
            rec = {"blocks_per_launch": blocks, "bytes_per_launch": by, "us_per_launch": ms * 1e3,
                   "us_per_block": ms * 1e3 / blocks, "GBps": by / (ms * 1e-3) / 1e9, "frac": by / (ms * 1e-3) / 1e9 / peak}
            cache.device_status()
            cache.close(); del cache
            torch.cuda.empty_cache()
            out.setdefault(pname, {})[f"{bits}bit"] = rec
    return out


def busy_wait_warm(device, ms=30.0):
    """Keep the GPU busy for about `ms` with plain copies (1 GiB each, larger than L2) and return with the queue
    still holding the last of them, so that what is timed next starts on a GPU at its working clocks."""
    global _WARM
    if _WARM is None or _WARM[0].device != torch.device(device):
        _WARM = (torch.empty(1 << 28, dtype=torch.float32, device=device), torch.empty(1 << 28, dtype=torch.float32, device=device))
    for _ in range(max(1, int(ms / 0.35))):
        _WARM[1].copy_(_WARM[0])


_WARM = None


def reduce_leg(wl, device, peak, repeats=3):
    """One progressive-reduce event of each width at the workload's per-block shape, timed alone: a one-block
    cache is filled at 16 bit to the full context and reduced 16 -> 8 -> 4 -> 2 by hand.  Bytes per event are
    body groups x (16 * 2b + 16 * b + 8): codes read, codes written, scale read and written."""
    from paper_2505_18610_b200.binding import Cache
    n_slices = wl["batch"] * wl["kv_heads"]
    n = wl["end_tokens"]
    best = {}
    launches = {}
    for _ in range(repeats):
        cache = Cache(1, wl["q_heads"], wl["kv_heads"], wl["batch"], n, [2], budget_bytes=[bytes_at(n, 16, n_slices)],
                      n_sink=N_SINK, window=WINDOW, auto_reduce=False, device=device)
        done = 0
        while done < n:
            m = min(8192, n - done)
            k, v = synth.make_kv(4, 0, done // 8192, m, wl["batch"], wl["kv_heads"], done, wl["n_outlier"], wl["factor"],
                                 device=device)
            cache.append(0, k.contiguous(), v.contiguous())
            done += m
        nb = n - N_SINK - WINDOW
        for b in (8, 4, 2):
            l0 = cache.launch_count()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            busy_wait_warm(device)           # an event fires between decode steps, on a GPU that is busy
            e0.record(); cache.progressive_reduce(0); e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            key = f"{2 * b}to{b}"
            best[key] = min(best.get(key, 1e9), ms)
            launches[key] = cache.launch_count() - l0
        cache.close(); del cache
        torch.cuda.empty_cache()
    out = {}
    nb = n - N_SINK - WINDOW
    for b in (8, 4, 2):
        key = f"{2 * b}to{b}"
        by = 2 * n_slices * nb * (16 * 2 * b + 16 * b + 8)
        out[key] = {"us": best[key] * 1e3, "bytes": by, "GBps": by / (best[key] * 1e-3) / 1e9,
                    "frac": by / (best[key] * 1e-3) / 1e9 / peak, "launches": launches[key]}
    return out


def aux_leg(wl, device, peak):
    """The kernels beside the decode step, timed alone with CUDA events: the bulk prefill append of 8192 tokens
    into one block of the workload's shape (best of 5 calls after a warm-up), one progressive-reduce event per
    width, and the alpha grid search of the calibration (2048 tokens x 8 sequences, 20 alphas, 2 bit)."""
    from paper_2505_18610_b200 import binding as B
    n = 8192
    k, v = synth.make_kv(3, 0, 0, n, wl["batch"], wl["kv_heads"], 0, wl["n_outlier"], wl["factor"], device=device)
    k, v = k.contiguous(), v.contiguous()
    n_slices = wl["batch"] * wl["kv_heads"]
    ts = []
    for _ in range(6):
        cache = B.Cache(1, wl["q_heads"], wl["kv_heads"], wl["batch"], 32768, [16], n_sink=N_SINK, window=WINDOW, device=device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        busy_wait_warm(device)
        e0.record(); cache.append(0, k, v); e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
        cache.close(); del cache
    append_bytes = 2 * n * n_slices * (256 + tokbytes(16))
    out = {"bulk_append": {"tokens": n, "ms": min(ts[1:]), "GBps": append_bytes / (min(ts[1:]) * 1e-3) / 1e9,
                           "frac": append_bytes / (min(ts[1:]) * 1e-3) / 1e9 / peak,
                           "bytes": append_bytes, "what": "bf16 K, V in, INT16 tiles out, one block"}}
    out["reduce"] = reduce_leg(wl, device, peak)
    g = torch.Generator().manual_seed(5)
    nt, ns, kvh, grp = 2048, 8, wl["kv_heads"], wl["q_heads"] // wl["kv_heads"]    # a 2,048-token calibration text
    kk = torch.randn(nt, ns, kvh, 128, generator=g); kk[..., 9] *= 25.0; kk[..., 73] *= 25.0
    qq = torch.randn(nt, ns, kvh * grp, 128, generator=g)
    vv = torch.randn(nt, ns, kvh, 128, generator=g)
    kk, qq, vv = (t.to(torch.bfloat16).to(device).contiguous() for t in (kk, qq, vv))
    ts = []
    for _ in range(3):
        torch.cuda.synchronize(); t0 = time.perf_counter()
        best, losses = B.alpha_grid_search(kk, qq, vv, 2, pos_scale=4.0)
        ts.append((time.perf_counter() - t0) * 1e3)
    flop = 21 * ns * kvh * grp * (nt * (nt + 1) / 2) * 128 * 4
    out["alpha_grid_search"] = {"tokens": nt, "sequences": ns, "alphas": 20, "bits": 2, "ms": min(ts[1:]), "best_alpha": best,
                                "useful_TFLOPs": flop / (min(ts[1:]) * 1e-3) / 1e12,   # each product is three fp16 MMAs
                                "what": "host-timed call (it ends with a synchronize); 21 causal attention passes"}
    return out


def steady_state_record(name, device, peak, launches=5, steps=4):
    """A compact steady-state record of another workload: the cache is built once with every block at its
    final width (default budgets), then timed twice: the all-blocks attention launch alone, and whole decode
    steps (append + eviction + attention) through pmkvq_decode_step."""
    wl = WORKLOADS[name]
    if wl.get("schedule") == "70b":
        fbit = plan(wl, 8, 3)[0]
    else:
        fbit = synth.bit_schedule(wl["layers"], wl["edge_bits"], wl["inner_bits"], wl["n_edge"])
    n0 = wl["end_tokens"] - steps - 3
    cache = build_cache(wl, fbit, None, None, n0, device, shared_chunks=True)
    assert all(cache.layer_state(l)["cur_bits"] == fbit[l] for l in range(wl["layers"]))
    L = wl["layers"]
    q = torch.stack([synth.make_q(2, l % 4, 0, wl["batch"], wl["q_heads"], n0, device=device) for l in range(L)]).contiguous()
    o = torch.empty(L, wl["batch"], wl["q_heads"], 128, dtype=torch.float32, device=device)
    # warm-up long enough (>= 10 launches of several ms) that both timings below see the GPU under sustained
    # load: on a 1 kW part the SM clock settles lower under the power cap after ~0.1 s, and this kernel follows it
    ts = time_attention_all(cache, q, o, launches, warm=10)
    by = sum(cache.attention_bytes(l) for l in range(L))
    ms = float(np.median(ts))
    k1, v1 = synth.make_kv(5, 0, 0, 1, wl["batch"], wl["kv_heads"], n0, wl["n_outlier"], wl["factor"], device=device)
    K = k1[0].unsqueeze(0).expand(L, -1, -1, -1).contiguous(); V = v1[0].unsqueeze(0).expand(L, -1, -1, -1).contiguous()
    for _ in range(3):
        cache.decode_step(K, V, q, out=o)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        cache.decode_step(K, V, q, out=o)
    e1.record()
    torch.cuda.synchronize()
    step_ms = e0.elapsed_time(e1) / steps
    by_step = sum(cache.attention_bytes(l) for l in range(L))
    cache.device_status()
    rec = {"workload": wl["name"], "fbit_counts": {str(b): fbit.count(b) for b in sorted(set(fbit))},
           "cache_GB": by / 1e9, "attention_ms_per_launch": ms, "attention_GBps": by / (ms * 1e-3) / 1e9,
           "attention_frac": by / (ms * 1e-3) / 1e9 / peak, "step_ms": step_ms,
           "step_GBps": by_step / (step_ms * 1e-3) / 1e9, "tokens_per_s": wl["batch"] / (step_ms * 1e-3),
           "what": "every block at its final width; after 10 warm-up launches, attention launch alone (median of %d) and whole decode steps (%d)" % (launches, steps)}
    cache.close(); del cache
    torch.cuda.empty_cache()
    return rec


class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.QUERY,
                                       "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def wait_first(self, timeout=5.0):
        """Block until the sampler has written its first line (nvidia-smi takes a moment to start)."""
        t0 = time.time()
        while self.p is not None and time.time() - t0 < timeout and os.path.getsize(self.f.name) == 0:
            time.sleep(0.01)

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush(); self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def run_steps(cache, wl, pool, steps, first_step, out, host_io=None):
    """Run `steps` decode steps.  With host_io the step's inputs come from pinned host memory and the
    outputs go back to pinned host memory (end-to-end leg)."""
    K, V, Q = pool
    n_pool = K.shape[0]
    for s in range(steps):
        i = (first_step + s) % n_pool
        if host_io is not None:
            hk, hv, hq, ho, dk, dv, dq, do = host_io
            dk.copy_(hk[i], non_blocking=True); dv.copy_(hv[i], non_blocking=True); dq.copy_(hq[i], non_blocking=True)
            cache.decode_step(dk, dv, dq, out=do)
            ho.copy_(do, non_blocking=True)
        else:
            cache.decode_step(K[i], V[i], Q[i], out=out)


def cpu_oracle_leg(wl, seconds_target=12.0, steps=None, warmup=1, n_sample_slices=4):
    """Time the CPU oracle as it stands on a bounded sample: `n_sample_slices` (batch, kv_head) slices of
    one 2-bit-Fbit block and one 4-bit-Fbit block at the full context length; each oracle step = append
    one token + decode attention on those slices.  Returns (GB/s, seconds per step, description, cores)."""
    from oracle import pmkvq_oracle as O
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    G = wl["q_heads"] // wl["kv_heads"]
    n_end = wl["end_tokens"]
    n_slices = wl["batch"] * wl["kv_heads"]
    layers = sorted({0, wl["layers"] // 2})
    fbit = plan(wl, 8, 3)[0]
    kvh = wl["kv_heads"]
    bsz = max(1, n_sample_slices // kvh)
    S = bsz * kvh
    orcs, bytes_per_step = [], 0
    n_prefill = n_end - 64
    for l in layers:
        pol = O.Policy(fbit[l], n_end, n_slices)
        k, v = synth.make_kv(0, l, 0, n_prefill, bsz, kvh, 0, wl["n_outlier"], wl["factor"])
        lam = synth.make_lambda(k[:512]).numpy()
        orc = O.LayerOracle(pol, S, lam=np.tile(lam, (bsz, 1)))
        orc.append_bulk(k.float().numpy().reshape(n_prefill, S, 128), v.float().numpy().reshape(n_prefill, S, 128))
        orcs.append((l, orc))
        nb = n_end - N_SINK - WINDOW
        bytes_per_step += 2 * S * ((N_SINK + WINDOW) * tokbytes(16) + nb * tokbytes(fbit[l])) + S * G * 128 * 6
    rng = np.random.default_rng(0)

    def one_step(i):
        for l, orc in orcs:
            kt = torch.tensor(rng.standard_normal((1, S, 128)).astype(np.float32)).to(torch.bfloat16).float().numpy()
            orc.append_bulk(kt, kt)
            q = torch.tensor(rng.standard_normal((S, G, 128)).astype(np.float32)).to(torch.bfloat16).float().numpy()
            orc.decode_attention(q)

    for i in range(warmup):
        one_step(i)
    t0 = time.perf_counter(); one_step(0); t1 = time.perf_counter() - t0
    if steps is None:
        steps = int(max(1, min(60, seconds_target / max(t1, 1e-3))))
    t0 = time.perf_counter()
    for i in range(steps):
        one_step(i)
    dt = (time.perf_counter() - t0) / steps
    desc = (f"{S} of {n_slices} (batch, kv_head) slices of blocks {layers} (Fbit {[fbit[l] for l in layers]}) at "
            f"{n_end} cached tokens; per step: append 1 token + decode attention; {steps} steps timed")
    return bytes_per_step / dt / 1e9, dt, desc, cores, steps, S * len(layers)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="pmkvq", choices=["pmkvq", "reference"])
    ap.add_argument("--workload", default="7b", choices=sorted(WORKLOADS))
    ap.add_argument("--ctas", type=int, default=0, help="attention grid override (0 = library default: one wave)")
    ap.add_argument("--attention-path", type=int, default=0, choices=[0, 1],
                    help="0 warp-level MMAs (default), 1 tensor memory at 4 and 2 bit")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-aux", action="store_true", help="skip the prefill-append, reduce and calibration timings")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-widths", action="store_true", help="skip the per-width steady-state records")
    ap.add_argument("--no-others", action="store_true", help="skip the compact 8B / 32B / 70B records")
    ap.add_argument("--only", default="", choices=["", "reduce", "append", "agrid"],
                    help="profiling runs: only the progressive-reduce events, only the bulk append, or only a (small) alpha "
                         "grid search of the aux leg")
    ap.add_argument("--attention-only", type=int, default=0,
                    help="profiling runs: build the cache at its final widths and launch the attention this many times")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    steps, warmup = args.steps, max(3, args.warmup)

    if args.impl == "reference":
        if rank != 0:
            return
        gbs, dt, desc, cores, nst, n_units = cpu_oracle_leg(wl, steps=steps, warmup=min(warmup, 2))
        line = {"impl": "reference", "metric": "decode_attention_GBps", "value": gbs, "unit": "GB/s",
                "n_gpus": args.gpus, "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": {"workload": wl["name"], "sample": desc},
                "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": desc},
                "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the product path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        with open(peaks_path) as f:
            peak, peak_src = float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak, peak_src = 6650.0, "fallback"

    fbit, budgets, n0 = plan(wl, steps, warmup)
    lam = make_lambda(wl, 0, device)
    L = wl["layers"]
    out_dev = torch.empty(L, wl["batch"], wl["q_heads"], 128, dtype=torch.float32, device=device)

    if args.only == "reduce":
        print(json.dumps({"only": "reduce", "workload": wl["name"], "reduce": reduce_leg(wl, device, peak, repeats=1)}))
        return
    if args.only == "append":
        from paper_2505_18610_b200 import binding as B
        k, v = synth.make_kv(3, 0, 0, 8192, wl["batch"], wl["kv_heads"], 0, wl["n_outlier"], wl["factor"], device=device)
        k, v = k.contiguous(), v.contiguous()
        for _ in range(3):
            c = B.Cache(1, wl["q_heads"], wl["kv_heads"], wl["batch"], 32768, [16], n_sink=N_SINK, window=WINDOW, device=device)
            c.append(0, k, v); torch.cuda.synchronize(); c.close()
        print(json.dumps({"only": "append", "workload": wl["name"], "tokens": 8192}))
        return
    if args.only == "agrid":     # 3 alphas on 2048 tokens x 2 sequences: 4 attention passes, small enough to capture
        from paper_2505_18610_b200 import binding as B
        g = torch.Generator().manual_seed(5)
        nt, ns, kvh, grp = 2048, 2, wl["kv_heads"], wl["q_heads"] // wl["kv_heads"]
        kk = torch.randn(nt, ns, kvh, 128, generator=g); kk[..., 9] *= 25.0; kk[..., 73] *= 25.0
        qq = torch.randn(nt, ns, kvh * grp, 128, generator=g)
        vv = torch.randn(nt, ns, kvh, 128, generator=g)
        kk, qq, vv = (t.to(torch.bfloat16).to(device).contiguous() for t in (kk, qq, vv))
        best, losses = B.alpha_grid_search(kk, qq, vv, 2, alphas=np.array([0.0, 0.5, 0.8], dtype=np.float32), pos_scale=4.0)
        print(json.dumps({"only": "agrid", "tokens": nt, "sequences": ns, "best_alpha": best, "losses": [float(x) for x in losses]}))
        return
    if args.attention_only:      # profiling runs: the steady-state attention launch and nothing else
        cache = build_cache(wl, fbit, None, lam, wl["end_tokens"], device, shared_chunks=True, attention_path=args.attention_path)
        q = torch.stack([synth.make_q(2, l, 0, wl["batch"], wl["q_heads"], wl["end_tokens"], device=device) for l in range(L)]).contiguous()
        ts = time_attention_all(cache, q, out_dev, args.attention_only, warm=2)
        by = sum(cache.attention_bytes(l) for l in range(L))
        print(json.dumps({"attention_only": True, "workload": wl["name"], "launches": args.attention_only,
                          "ms_per_launch": float(np.median(ts)), "GBps": by / (float(np.median(ts)) * 1e-3) / 1e9, "bytes": by}))
        return

    n_pool = 8
    pool = step_inputs(wl, n_pool, 0, device, n0)

    # ---------------- the cache is built once; its freshly prefilled state is kept for the end-to-end leg ----------------
    cache = build_cache(wl, fbit, budgets, lam, n0, device, attention_path=args.attention_path)
    if args.ctas:
        cache.set_attention_ctas(args.ctas)
    states0 = [cache.layer_state(l) for l in range(L)]
    snapshot = None
    if not args.no_e2e and cache.arena.numel() < 70e9:
        snapshot = cache.arena.clone()

    # ---------------- device-resident leg: `value` (the trajectory: appends, evictions, every block's last reduce) ----------------
    # the clock sampler runs from the warm-up steps to the end of the end-to-end leg (the GPU is under this
    # workload's load the whole time); the timed region starts once it has delivered its first sample
    sampler = ClockSampler(local_rank) if rank == 0 else None
    run_steps(cache, wl, pool, warmup, 0, out_dev)
    bits_before = [cache.layer_state(l)["cur_bits"] for l in range(L)]
    if sampler:
        sampler.wait_first()
    barrier()
    launches0 = cache.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total_bytes = 0
    ev0.record()
    for s in range(steps):
        run_steps(cache, wl, pool, 1, warmup + s, out_dev)
        total_bytes += step_bytes(cache, wl, bits_before)       # host-side bookkeeping only
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    launches = cache.launch_count() - launches0
    n_reduced = sum(1 for l in range(L) if cache.layer_state(l)["cur_bits"] == fbit[l])
    final_tokens = cache.layer_state(0)["n_tokens"]

    # ---------------- roofline leg: the attention launch alone, on the cache as the run left it ----------------
    # (every block that can be is at its final width now: no reduce, no append, only decode_attn_fused_kernel)
    n_attn = max(10, min(steps, 40))
    ts = time_attention_all(cache, pool[2][0], out_dev, n_attn)
    attn_ms = float(np.sum(ts))
    attn_bytes = sum(cache.attention_bytes(l) for l in range(L))
    widths_now = {str(b): sum(1 for l in range(L) if cache.layer_state(l)["cur_bits"] == b) for b in (2, 4, 8, 16)}
    cache.device_status()

    # ---------------- end-to-end leg: the same trajectory with host buffers in, host buffers out ----------------
    e2e_ms, h2d, d2h = float("nan"), 0, 0
    if not args.no_e2e:
        if snapshot is not None:
            cache.arena.copy_(snapshot)
            for l in range(L):
                cache.restore_layer_state(l, states0[l]["n_tokens"], states0[l]["cur_bits"])
            del snapshot
        else:
            cache.close(); del cache
            torch.cuda.empty_cache()
            cache = build_cache(wl, fbit, budgets, lam, n0, device, attention_path=args.attention_path)
            if args.ctas:
                cache.set_attention_ctas(args.ctas)
        K, V, Q = pool
        hk, hv, hq = K.cpu().pin_memory(), V.cpu().pin_memory(), Q.cpu().pin_memory()
        dk, dv, dq = torch.empty_like(K[0]), torch.empty_like(V[0]), torch.empty_like(Q[0])
        do = torch.empty(L, wl["batch"], wl["q_heads"], 128, dtype=torch.float32, device=device)
        ho = torch.empty(do.shape, dtype=torch.float32).pin_memory()
        host_io = (hk, hv, hq, ho, dk, dv, dq, do)
        run_steps(cache, wl, pool, warmup, 0, out_dev, host_io=host_io)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run_steps(cache, wl, pool, steps, warmup, out_dev, host_io=host_io)
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        h2d = (dk.numel() + dv.numel() + dq.numel()) * 2
        d2h = do.numel() * 4
    clocks = sampler.stop() if sampler else None
    cache.close(); del cache
    torch.cuda.empty_cache()

    # ---------------- max over ranks ----------------
    ms, e2e_ms, attn_ms = max_over_ranks([ms, e2e_ms, attn_ms], dist, device)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    value = whole_job_rate(total_bytes, world, ms) / 1e9
    traffic = None
    if wl is WORKLOADS["7b"] and kernel_source_digest() == NCU_TRAFFIC["digest"]:
        # measured traffic / algorithmic bytes of the captured launch, applied to this run's launch
        traffic = NCU_TRAFFIC["traffic_bytes"] / NCU_TRAFFIC["algorithmic_bytes"] * attn_bytes
    achieved = attn_bytes * n_attn / (attn_ms * 1e-3) / 1e9
    line = {
        "metric": "decode_attention_GBps", "value": value, "unit": "GB/s", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int2/int4/int8/int16 codes as f16 MMA operands, f32 accumulate", "data": "synthetic",
        "config": {"workload": wl["name"],
                   "shape": f"{L} blocks x ({wl['q_heads']} Q / {wl['kv_heads']} KV heads, head_dim 128) x batch "
                            f"{wl['batch']} per GPU x {final_tokens} cached tokens at the end",
                   "fbit_per_block": fbit,
                   "blocks_reduced_to_fbit_in_run": n_reduced, "n_sink": N_SINK, "window": WINDOW,
                   "attention_path": "tensor memory (tcgen05.mma)" if args.attention_path else "warp-level MMAs (mma.sync)",
                   "l2": "per-step working set (the whole cache) is far larger than L2; no flush needed",
                   "path": "attention path only (no weights / MLP)", "sharding": "batch, no collective"},
        "tokens_per_s": whole_job_rate(wl["batch"] * steps, world, ms),
        "frac_of_8TBps_nominal": value / world / 8000.0,
        "roofline": {"bound": "hbm", "kernel": "decode_attn_fused_kernel: the attention of all blocks, one launch",
                     "achieved": achieved, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic,
                     "traffic_source": "ncu dram read+write / algorithmic bytes of a captured 4-block launch of the same kernel, times this "
                                       "run's launch; null if the kernel sources changed since the capture",
                     "avg_launch_ms": attn_ms / n_attn, "launches_timed": n_attn,
                     "algorithmic_bytes_per_launch": attn_bytes, "blocks_at_width": widths_now,
                     "how": "after the timed steps (every block's last reduce is behind it) the attention launch alone is "
                            "repeated on the same cache through pmkvq_decode_attention_all, one CUDA event pair per launch; "
                            "nothing is appended or reduced in between"},
        "e2e": {"value": world * total_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms / steps,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "clocks": clocks,
    }
    if world == 1:
        if not args.no_widths:
            line["roofline_by_width"] = width_leg(wl, device, peak)
        if not args.no_aux:
            line["aux"] = aux_leg(wl, device, peak)
        if not args.no_others:
            line["other_workloads"] = {n: steady_state_record(n, device, peak) for n in ("8b", "32b", "70b") if WORKLOADS[n] is not wl}
        if not args.no_cpu_baseline:
            gbs, dt, desc, cores, nst, _ = cpu_oracle_leg(wl)
            line["cpu_baseline"] = {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": desc,
                                    "s_per_oracle_step": dt}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
