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
        # a ~100 GB cache whose blocks sit at different points of the 16 -> 8 -> 4 -> 2 chain: 4 blocks
        # cross 16 -> 8 during the run, 8 cross 8 -> 4, 30 cross 4 -> 2, the other 38 are already at 2 bit
        fbit, crossing = [], []
        for l in range(L):
            fbit.append(8 if l >= L - 4 else 4 if l >= L - 12 else 2)
            crossing.append(l >= L - 42)
        k = 0
        for l in range(L):
            if crossing[l]:
                fire_step = warmup + (k * steps) // 42
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


def build_cache(wl, fbit, budgets, lam, n0, device, chunk=8192, seed=0):
    from paper_2505_18610_b200.binding import Cache
    cache = Cache(wl["layers"], wl["q_heads"], wl["kv_heads"], wl["batch"], wl["end_tokens"], fbit,
                  budget_bytes=budgets, lam=lam, n_sink=N_SINK, window=WINDOW, device=device)
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
    for f in ("kernels_attn.cuh", "kernels_cache.cuh", "layout.cuh"):
        with open(os.path.join(d, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


# DRAM read + write bytes of one launch of the all-blocks attention kernel from the ncu capture summarised in
# profiles/decode_attn_fused_7b_shape.md (4 blocks of the 7B shape: a launch of the 28-block workload moves
# 7x the bytes, block by block the same way), its algorithmic bytes, and the digest of the sources it was
# taken on.
NCU_TRAFFIC = {"digest": "302fac57a5376af8", "traffic_bytes": 976_058_112, "algorithmic_bytes": 954_646_528}


def aux_leg(wl, device):
    """The two kernels beside the decode step, timed alone with CUDA events (best of 5 calls after a warm-up):
    the bulk prefill append of 8192 tokens into one block of the workload's shape, and the alpha grid search
    of the calibration (2048 tokens x 8 sequences of the workload's head counts, 20 alphas, 2 bit)."""
    from paper_2505_18610_b200 import binding as B
    n = 8192
    k, v = synth.make_kv(3, 0, 0, n, wl["batch"], wl["kv_heads"], 0, wl["n_outlier"], wl["factor"], device=device)
    k, v = k.contiguous(), v.contiguous()
    n_slices = wl["batch"] * wl["kv_heads"]
    ts = []
    for _ in range(6):
        cache = B.Cache(1, wl["q_heads"], wl["kv_heads"], wl["batch"], 32768, [16], n_sink=N_SINK, window=WINDOW, device=device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(); cache.append(0, k, v); e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
        cache.close(); del cache
    append_bytes = 2 * n * n_slices * (256 + tokbytes(16))
    out = {"bulk_append": {"tokens": n, "ms": min(ts[1:]), "GBps": append_bytes / (min(ts[1:]) * 1e-3) / 1e9,
                           "bytes": append_bytes, "what": "bf16 K, V in, INT16 tiles out, one block"}}
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
                                "fp32_TFLOPs": flop / (min(ts[1:]) * 1e-3) / 1e12,
                                "what": "host-timed call (it ends with a synchronize); 21 causal attention passes"}
    return out


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


def run_steps(cache, wl, pool, steps, first_step, out, host_io=None, attn_events=None):
    """Run `steps` decode steps.  With host_io the step's inputs come from pinned host memory and the
    outputs go back to pinned host memory (end-to-end leg)."""
    K, V, Q = pool
    n_pool = K.shape[0]
    L = wl["layers"]
    for s in range(steps):
        i = (first_step + s) % n_pool
        if host_io is not None:
            hk, hv, hq, ho, dk, dv, dq, do = host_io
            dk.copy_(hk[i], non_blocking=True); dv.copy_(hv[i], non_blocking=True); dq.copy_(hq[i], non_blocking=True)
            cache.decode_step(dk, dv, dq, out=do)
            ho.copy_(do, non_blocking=True)
        elif attn_events is None:
            cache.decode_step(K[i], V[i], Q[i], out=out)
        else:
            # an event pair around the step's launches: the all-blocks attention kernel and the all-blocks
            # append kernel before it (and, in the few steps where a block's budget fills, its reduce)
            bits0 = [cache.layer_state(l)["cur_bits"] for l in range(L)]
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            cache.decode_step(K[i], V[i], Q[i], out=out)
            e1.record()
            reduced = any(cache.layer_state(l)["cur_bits"] != bits0[l] for l in range(L))
            attn_events.append((e0, e1, sum(cache.attention_bytes(l) for l in range(L)), reduced))


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
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-aux", action="store_true", help="skip the prefill-append and calibration timings")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-kernel-timing", action="store_true", help="skip the per-launch event leg (profiling runs)")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    steps, warmup = args.steps, max(3, args.warmup)
    G = wl["q_heads"] // wl["kv_heads"]

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

    fbit, budgets, n0 = plan(wl, steps, warmup)
    lam = make_lambda(wl, 0, device)
    n_pool = 8
    pool = step_inputs(wl, n_pool, 0, device, n0)
    n_slices = wl["batch"] * wl["kv_heads"]

    out_dev = torch.empty(wl["layers"], wl["batch"], wl["q_heads"], 128, dtype=torch.float32, device=device)

    # ---------------- device-resident leg: `value` ----------------
    cache = build_cache(wl, fbit, budgets, lam, n0, device)
    if args.ctas:
        cache.set_attention_ctas(args.ctas)
    run_steps(cache, wl, pool, warmup, 0, out_dev)
    bits_before = [cache.layer_state(l)["cur_bits"] for l in range(wl["layers"])]
    barrier()
    launches0 = cache.launch_count()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total_bytes = 0
    ev0.record()
    for s in range(steps):
        run_steps(cache, wl, pool, 1, warmup + s, out_dev)
        total_bytes += step_bytes(cache, wl, bits_before)       # host-side bookkeeping only
    ev1.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    ms = ev0.elapsed_time(ev1)
    launches = cache.launch_count() - launches0
    n_reduced = sum(1 for l in range(wl["layers"]) if cache.layer_state(l)["cur_bits"] == fbit[l])
    final_tokens = cache.layer_state(0)["n_tokens"]
    cache.close(); del cache
    torch.cuda.empty_cache()

    # ---------------- the same timed region again, with an event pair around every step ----------------
    attn_ms, attn_bytes, n_attn, instr_ms = float("nan"), 0, 0, float("nan")
    if not args.no_kernel_timing:
        cache = build_cache(wl, fbit, budgets, lam, n0, device)
        if args.ctas:
            cache.set_attention_ctas(args.ctas)
        run_steps(cache, wl, pool, warmup, 0, out_dev)
        barrier()
        attn_events = []
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        k0.record()
        run_steps(cache, wl, pool, steps, warmup, out_dev, attn_events=attn_events)
        k1.record()
        barrier()
        instr_ms = k0.elapsed_time(k1)
        plain = [(a, b, c) for a, b, c, reduced in attn_events if not reduced] or [(a, b, c) for a, b, c, _ in attn_events]
        attn_ms = sum(a.elapsed_time(b) for a, b, _ in plain)
        attn_bytes = sum(c for _, _, c in plain)
        n_attn = len(plain)
        cache.close(); del cache
        torch.cuda.empty_cache()

    # ---------------- end-to-end leg: host buffers in, host buffers out ----------------
    e2e_ms, h2d, d2h = float("nan"), 0, 0
    if not args.no_e2e:
        cache = build_cache(wl, fbit, budgets, lam, n0, device)
        if args.ctas:
            cache.set_attention_ctas(args.ctas)
        K, V, Q = pool
        hk, hv, hq = K.cpu().pin_memory(), V.cpu().pin_memory(), Q.cpu().pin_memory()
        dk, dv, dq = torch.empty_like(K[0]), torch.empty_like(V[0]), torch.empty_like(Q[0])
        do = torch.empty(wl["layers"], wl["batch"], wl["q_heads"], 128, dtype=torch.float32, device=device)
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
        cache.close(); del cache

    # ---------------- max over ranks ----------------
    ms, e2e_ms, attn_ms = max_over_ranks([ms, e2e_ms, attn_ms], dist, device)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        with open(peaks_path) as f:
            peak, peak_src = float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak, peak_src = 6650.0, "fallback"
    value = whole_job_rate(total_bytes, world, ms) / 1e9
    traffic = None
    if wl is WORKLOADS["7b"] and kernel_source_digest() == NCU_TRAFFIC["digest"] and n_attn:
        # measured traffic / algorithmic bytes of the captured launches, applied to this run's average launch
        ratio = NCU_TRAFFIC["traffic_bytes"] / NCU_TRAFFIC["algorithmic_bytes"]
        traffic = ratio * attn_bytes / n_attn
    achieved = attn_bytes / (attn_ms * 1e-3) / 1e9 if n_attn else float("nan")
    line = {
        "metric": "decode_attention_GBps", "value": value, "unit": "GB/s", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int2/int4/int16 codes, f16 mma.sync, f32 accumulate", "data": "synthetic",
        "config": {"workload": wl["name"],
                   "shape": f"{wl['layers']} blocks x ({wl['q_heads']} Q / {wl['kv_heads']} KV heads, head_dim 128) x batch "
                            f"{wl['batch']} per GPU x {final_tokens} cached tokens at the end",
                   "fbit_per_block": fbit,
                   "blocks_reduced_to_fbit_in_run": n_reduced, "n_sink": N_SINK, "window": WINDOW,
                   "l2": "per-step working set (the whole cache) is far larger than L2; no flush needed",
                   "path": "attention path only (no weights / MLP)", "sharding": "batch, no collective"},
        "tokens_per_s": whole_job_rate(wl["batch"] * steps, world, ms),
        "frac_of_8TBps_nominal": value / world / 8000.0,
        "roofline": {"bound": "hbm", "kernel": "decode_attn_fused_kernel: the attention of all blocks of a step, one launch",
                     "achieved": achieved, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic,
                     "traffic_source": "ncu dram read+write / algorithmic bytes of a captured 4-block launch of the same kernel, times this "
                                       "run's average launch; null if the kernel sources changed since the capture",
                     "avg_launch_ms": attn_ms / max(1, n_attn), "launches_timed": n_attn,
                     "algorithmic_bytes_per_launch": attn_bytes / max(1, n_attn),
                     "how": "the timed steps replayed on an identical cache with a CUDA event pair around every step; "
                            "the pair also spans the step's append kernel (one launch, under 1 % of the step); steps in "
                            "which a block was reduced are left out of the average",
                     "ms_per_step_with_events": instr_ms / steps},
        "e2e": {"value": world * total_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms / steps,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        gbs, dt, desc, cores, nst, _ = cpu_oracle_leg(wl)
        line["cpu_baseline"] = {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": desc,
                                "s_per_oracle_step": dt}
    if not args.no_aux and world == 1:
        line["aux"] = aux_leg(wl, device)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
