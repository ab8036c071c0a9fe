"""Plain, slow, obviously-correct CPU oracle of the PM-KVQ decode hot path.

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg; never by the product package.  numpy only.
It is independent of the CUDA path: no shared code, tables or helpers.

What it computes, and the passage of the paper each part follows:

* ``quantize_asym``           - asymmetric uniform quantizer, Eq. 1-2 (Sec. 2.2),
                                one group = one token x one KV head x 128
                                channels (group size 128, Sec. 4.1.3).
* ``shift_reduce``            - "Equivalent Right Shift" 2b -> b, Eq. 3 (Sec. 3.1),
                                with ``S_b = (2^b+1) S_2b`` and ``Z_b = Z_2b``.
* ``direct_right_shift`` /
  ``modified_right_shift``    - the two ablation variants of Sec. 4.4.1; ``halve`` /
                                ``chain_variant`` apply the chosen one, and
                                ``LayerOracle(shift_variant=...)`` runs the cache with it.
* ``Policy``                  - progressive policy of Sec. 3.1: 16-bit first,
                                halve the width of the existing cache when the
                                block's budget is full, stop at Fbit; first token
                                and most recent 128 tokens stay INT16 (Sec. 4.1.2).
* ``LayerOracle``             - one transformer block's cache for a set of
                                (batch, kv-head) slices: append, window eviction,
                                progressive reduce, decode attention with the
                                channel-wise Key equalization of Eq. 9 (Sec. 3.3).

Arithmetic: the quantizer works in IEEE fp32 exactly as written (sub, true
division, round-half-to-even) so that codes / scales / zero-points have one
correct bit pattern; the shift is integer arithmetic; attention is the plain
definition softmax(s * Q K^T) V on the dequantized values in float64.

Parity status of each function (what pins it, see tests/test_oracle_*.py):
  quantize_asym        pinned  (closed form on hand cases, error bound <= S/2,
                                end points, exact-rational cross-check)
  shift_reduce         pinned  (exhaustive vs nearest-integer division, identity
                                (2^2b-2^b+1)(2^b+1) = 2^3b+1, theorem of App. D
                                in exact rational arithmetic)
  reduce_scale         pinned  (S chain equals (max-Z)/(2^b-1) within 3 roundings)
  Policy               pinned  (halving thresholds 4096/8192/16384 for Fbit=2 and
                                32K maximum length, App. C.7 / Fig. 2a)
  decode_attention     pinned  (N=1, equal scores, brute force loops, library
                                softmax-attention on the dequantized values,
                                equalization invariance with power-of-two lambda)
  direct / modified right shift
                       pinned  (floor division by 2^b; dequantized value = centre of the
                                merged bin for the modified variant; half-step error bound
                                for Equivalent and Modified, 3/4 of a step for Direct)
  rope_interpolated / calibrate_lambda
                       pinned  (norm of every rotated pair is kept; one constant pair sweeps the
                                closed form r*|cos(m s theta_i + phi)|; s = 4 on n tokens equals
                                s = 1 at positions 0, 4, 8, ...; with the lowest-frequency pair's
                                2 pi / theta_i = 54,410-token period (Sec. 3.3) a 2,048-token text
                                reaches the pair's full amplitude only with interpolation)
  causal_self_attention / attention_reconstruction_losses / grid_search_alpha
                       pinned  (brute-force loops on a tiny case incl. the head-to-KV-head map;
                                loss vanishes at 16 bit for every alpha, so Lambda and Lambda^-1 pair
                                up; one token: loss = the Value quantization error alone, whatever
                                alpha; the last query row equals decode_attention of a LayerOracle
                                holding the same tokens; at alpha = 1 the loss is unchanged by
                                power-of-two rescaling of a channel pair of K against Q; an outlier
                                channel pair moves the best alpha away from 0)
  allocate_bits_brute_force
                       pinned  (it IS the definition of Eq. 6-8 written out; limits: budget at
                                the floor / unbounded; hand case)
  pack_canonical       pinned  (hand-written byte examples, round trip)
  accuracy on real models      parity unpinned (needs weights / benchmark items)
"""
from __future__ import annotations

import numpy as np

HEAD_DIM = 128
WIDTHS = (16, 8, 4, 2)


# --------------------------------------------------------------------------
# Eq. 1-2: asymmetric uniform quantizer, one group = last axis
# --------------------------------------------------------------------------
def quantize_asym(x, bits: int):
    """Quantize fp32 groups (last axis) to ``bits``-bit unsigned codes.

    Eq. 1-2: Z = min(x), S = (max(x) - Z) / (2^bits - 1), code = round((x - Z) / S).
    All steps are single fp32 operations; rounding is round-half-to-even.
    A constant group (max == Z) gets S = 0 and all codes 0 (dequantizes to Z).
    Returns (codes uint16, S float32, Z float32); S and Z have x.shape[:-1].
    """
    x = np.asarray(x, dtype=np.float32)
    qmax = np.float32((1 << bits) - 1)
    z = x.min(axis=-1).astype(np.float32)
    m = x.max(axis=-1).astype(np.float32)
    s = ((m - z).astype(np.float32) / qmax).astype(np.float32)
    d = (x - z[..., None]).astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = (d / s[..., None]).astype(np.float32)
    c = np.rint(t)                      # numpy rint = round-half-to-even
    c = np.where(s[..., None] == 0, np.float32(0), c)
    c = np.clip(c, 0, float(qmax))
    return c.astype(np.uint16), s, z


def dequantize(codes, s, z):
    """x_hat = S * code + Z in float64 (inverse of Eq. 1)."""
    return (np.asarray(s, dtype=np.float64)[..., None] * np.asarray(codes, dtype=np.float64)
            + np.asarray(z, dtype=np.float64)[..., None])


# --------------------------------------------------------------------------
# Eq. 3: Equivalent Right Shift, and the two ablation variants (Sec. 4.4.1)
# --------------------------------------------------------------------------
def shift_multiplier(b: int) -> int:
    """The constant 2^(2b) - 2^b + 1 of Eq. 3."""
    return (1 << (2 * b)) - (1 << b) + 1


def shift_reduce(codes_2b, b: int):
    """Eq. 3: X_b = ((2^2b - 2^b + 1) * (X_2b + 2^(b-1))) >> 3b, for b in {8, 4, 2}."""
    c = np.asarray(codes_2b).astype(np.uint64)
    out = (np.uint64(shift_multiplier(b)) * (c + np.uint64(1 << (b - 1)))) >> np.uint64(3 * b)
    return out.astype(np.uint16)


def reduce_scale(s_2b, b: int):
    """S_b = (2^b + 1) * S_2b as one fp32 multiply (Sec. 3.1); Z is unchanged."""
    return (np.asarray(s_2b, dtype=np.float32) * np.float32((1 << b) + 1)).astype(np.float32)


def chain_to(codes16, s16, bits: int):
    """Apply Eq. 3 repeatedly 16 -> 8 -> ... -> ``bits`` to INT16 codes and their scale."""
    c, s, w = np.asarray(codes16, dtype=np.uint16), np.asarray(s16, dtype=np.float32), 16
    while w > bits:
        w //= 2
        c, s = shift_reduce(c, w), reduce_scale(s, w)
    return c, s


SHIFT_EQUIVALENT, SHIFT_DIRECT, SHIFT_MODIFIED = 0, 1, 2


def halve(codes_2b, s_2b, z_2b, b: int, variant: int = SHIFT_EQUIVALENT):
    """One halving 2b -> b of codes, scale and zero-point with the chosen shrinking strategy
    (Sec. 3.1 for the Equivalent Right Shift, Sec. 4.4.1 for the two ablation variants)."""
    if variant == SHIFT_DIRECT:
        return direct_right_shift(codes_2b, s_2b, z_2b, b)
    if variant == SHIFT_MODIFIED:
        return modified_right_shift(codes_2b, s_2b, z_2b, b)
    return shift_reduce(codes_2b, b), reduce_scale(s_2b, b), np.asarray(z_2b, dtype=np.float32)


def chain_variant(codes16, s16, z16, bits: int, variant: int = SHIFT_EQUIVALENT):
    """16 -> 8 -> ... -> ``bits`` with the chosen strategy, one halving after the other."""
    c, s, z, w = np.asarray(codes16, np.uint16), np.asarray(s16, np.float32), np.asarray(z16, np.float32), 16
    while w > bits:
        w //= 2
        c, s, z = halve(c, s, z, w, variant)
    return c, s, z


def direct_right_shift(codes_2b, s_2b, z_2b, b: int):
    """Ablation (1) of Sec. 4.4.1: X_b = X_2b >> b, Z unchanged, S_b = (2^b+1) S_2b."""
    c = (np.asarray(codes_2b).astype(np.uint32) >> np.uint32(b)).astype(np.uint16)
    return c, reduce_scale(s_2b, b), np.asarray(z_2b, dtype=np.float32)


def modified_right_shift(codes_2b, s_2b, z_2b, b: int):
    """Ablation (2) of Sec. 4.4.1: X_b = X_2b >> b, S_b = 2^b S_2b, Z_b = Z_2b + (S_b - S_2b)/2."""
    s2 = np.asarray(s_2b, dtype=np.float32)
    c = (np.asarray(codes_2b).astype(np.uint32) >> np.uint32(b)).astype(np.uint16)
    sb = (s2 * np.float32(1 << b)).astype(np.float32)
    zb = (np.asarray(z_2b, dtype=np.float32)
          + ((sb - s2).astype(np.float32) * np.float32(0.5)).astype(np.float32)).astype(np.float32)
    return c, sb, zb


# --------------------------------------------------------------------------
# Canonical packed layout used to compare codes bit-for-bit
# --------------------------------------------------------------------------
def pack_canonical(codes, bits: int):
    """Pack one token's 128 codes: element i sits in byte floor(i*bits/8) at bit offset
    (i*bits) mod 8, least-significant bits first; 16-bit codes are little-endian."""
    c = np.asarray(codes, dtype=np.uint16)
    n = c.shape[-1]
    if bits == 16:
        out = np.empty(c.shape[:-1] + (2 * n,), dtype=np.uint8)
        out[..., 0::2] = (c & 0xFF).astype(np.uint8)
        out[..., 1::2] = (c >> 8).astype(np.uint8)
        return out
    per = 8 // bits
    c = c.reshape(c.shape[:-1] + (n // per, per)).astype(np.uint32)
    out = np.zeros(c.shape[:-1], dtype=np.uint32)
    for j in range(per):
        out |= c[..., j] << np.uint32(j * bits)
    return out.astype(np.uint8)


def unpack_canonical(packed, bits: int, n: int = HEAD_DIM):
    p = np.asarray(packed, dtype=np.uint8)
    if bits == 16:
        return (p[..., 0::2].astype(np.uint16) | (p[..., 1::2].astype(np.uint16) << 8))[..., :n]
    per = 8 // bits
    out = np.empty(p.shape[:-1] + (p.shape[-1] * per,), dtype=np.uint16)
    for j in range(per):
        out[..., j::per] = (p >> (j * bits)) & ((1 << bits) - 1)
    return out[..., :n]


# --------------------------------------------------------------------------
# Policy of Sec. 3.1 (host arithmetic)
# --------------------------------------------------------------------------
def tokbytes(bits: int, count_metadata: bool = True) -> int:
    """Bytes of ONE of K or V for one token of one KV head: 128 codes, plus an fp32
    scale and an fp32 zero-point when metadata is counted."""
    return HEAD_DIM * bits // 8 + (8 if count_metadata else 0)


class Policy:
    """Token bookkeeping of one transformer block (all slices of the batch share it).

    Tokens 0..n_sink-1 and the most recent ``window`` (up to window+evict_chunk-1)
    tokens are INT16 (Sec. 4.1.2); everything in between is the "body" at ``cur_bits``.
    ``cur_bits`` starts at 16 and is halved (whole body at once, Sec. 3.1) when an
    append would push the block over ``budget_bytes``; it never goes below ``fbit``.
    """

    def __init__(self, fbit, max_tokens, n_slices, budget_bytes=None, n_sink=1, window=128,
                 evict_chunk=1, count_metadata=True):
        assert fbit in WIDTHS and evict_chunk >= 1 and n_sink >= 0 and window >= 0
        self.fbit, self.max_tokens, self.n_slices = fbit, max_tokens, n_slices
        self.n_sink, self.window, self.evict_chunk = n_sink, window, evict_chunk
        self.count_metadata = count_metadata
        self.budget = self.default_budget() if budget_bytes is None else int(budget_bytes)
        self.n_tokens = 0
        self.cur_bits = 16

    # structure as a function of the token count
    def n_sink_at(self, n):
        return min(n, self.n_sink)

    def n_body_at(self, n):
        excess = n - self.n_sink - self.window
        return 0 if excess <= 0 else (excess // self.evict_chunk) * self.evict_chunk

    def bytes_at(self, n, bits):
        nb = self.n_body_at(n)
        n16 = n - nb
        per_slice = 2 * (n16 * tokbytes(16, self.count_metadata) + nb * tokbytes(bits, self.count_metadata))
        return per_slice * self.n_slices

    def default_budget(self):
        """Budget from Fbit and the maximum context length (Sec. 3.1): the bytes of a cache whose
        body is at Fbit, at its largest over the last ``evict_chunk`` token counts up to max_tokens
        (with chunked eviction the INT16 window is fullest just before a chunk leaves it)."""
        lo = max(0, self.max_tokens - self.evict_chunk + 1)
        return max(self.bytes_at(n, self.fbit) for n in range(lo, self.max_tokens + 1))

    def bytes_used(self):
        return self.bytes_at(self.n_tokens, self.cur_bits)

    def reduces_needed_for(self, n_after):
        """How many halvings must happen before the cache may hold n_after tokens.
        Returns (count, ok); ok is False when it does not fit even at Fbit or exceeds
        max_tokens."""
        if n_after > self.max_tokens:
            return 0, False
        bits, k = self.cur_bits, 0
        while self.bytes_at(n_after, bits) > self.budget:
            if bits <= self.fbit:
                return k, False
            bits //= 2
            k += 1
        return k, True


# --------------------------------------------------------------------------
# One transformer block's cache for a chosen set of (batch, kv_head) slices
# --------------------------------------------------------------------------
class LayerOracle:
    """Cache of one transformer block, holding ``n_stored`` slices of the block's
    ``policy.n_slices`` (batch x kv_head) slices.  Per slice and per token it keeps the
    codes of K and V (uint16, value < 2^bits), their fp32 scale and zero-point, and the
    token's width.  ``lam`` is the per-channel equalization vector of Eq. 9 for each
    stored slice, shape [n_stored, 128] (all ones when None).
    """

    def __init__(self, policy: Policy, n_stored: int, lam=None, shift_variant: int = SHIFT_EQUIVALENT):
        self.p = policy
        self.variant = shift_variant
        cap = policy.max_tokens
        self.S = n_stored
        self.lam = (np.ones((n_stored, HEAD_DIM), np.float32) if lam is None
                    else np.asarray(lam, dtype=np.float32).reshape(n_stored, HEAD_DIM))
        self.inv_lam = (np.float32(1.0) / self.lam).astype(np.float32)
        self.ck = np.zeros((n_stored, cap, HEAD_DIM), np.uint16)
        self.cv = np.zeros((n_stored, cap, HEAD_DIM), np.uint16)
        self.sk = np.zeros((n_stored, cap), np.float32)
        self.zk = np.zeros((n_stored, cap), np.float32)
        self.sv = np.zeros((n_stored, cap), np.float32)
        self.zv = np.zeros((n_stored, cap), np.float32)
        self.bits = np.zeros((cap,), np.uint8)
        self.n_reduces = 0

    # -- Sec. 3.1: shrink the whole body 2b -> b --------------------------------
    def reduce(self):
        p = self.p
        if p.cur_bits <= p.fbit:
            raise RuntimeError("already at Fbit")
        b = p.cur_bits // 2
        lo, hi = p.n_sink_at(p.n_tokens), p.n_sink_at(p.n_tokens) + p.n_body_at(p.n_tokens)
        if hi > lo:
            self.ck[:, lo:hi], self.sk[:, lo:hi], self.zk[:, lo:hi] = halve(
                self.ck[:, lo:hi], self.sk[:, lo:hi], self.zk[:, lo:hi], b, self.variant)
            self.cv[:, lo:hi], self.sv[:, lo:hi], self.zv[:, lo:hi] = halve(
                self.cv[:, lo:hi], self.sv[:, lo:hi], self.zv[:, lo:hi], b, self.variant)
            self.bits[lo:hi] = b
        p.cur_bits = b
        self.n_reduces += 1

    # -- one decode-step append, in the order: budget test, quantize, evict -------
    def append_token(self, k_t, v_t, auto_reduce=True):
        """k_t, v_t: [n_stored, 128] fp32 values that are exactly representable in bf16."""
        p = self.p
        n_after = p.n_tokens + 1
        k, ok = p.reduces_needed_for(n_after)
        if not ok:
            raise OverflowError("capacity: cache does not fit at Fbit or exceeds max_tokens")
        if k and not auto_reduce:
            raise BufferError("budget full")
        for _ in range(k):
            self.reduce()
        t = p.n_tokens
        xk = (np.asarray(k_t, dtype=np.float32) * self.inv_lam).astype(np.float32)   # K * Lambda^-1 (Eq. 9)
        xv = np.asarray(v_t, dtype=np.float32)
        self.ck[:, t], self.sk[:, t], self.zk[:, t] = quantize_asym(xk, 16)
        self.cv[:, t], self.sv[:, t], self.zv[:, t] = quantize_asym(xv, 16)
        self.bits[t] = 16
        old_body_end = p.n_sink_at(p.n_tokens) + p.n_body_at(p.n_tokens)
        p.n_tokens = n_after
        new_body_end = p.n_sink_at(n_after) + p.n_body_at(n_after)
        for e in range(old_body_end, new_body_end):      # tokens leaving the INT16 window
            if e < p.n_sink:
                continue
            self.ck[:, e], self.sk[:, e], self.zk[:, e] = chain_variant(
                self.ck[:, e], self.sk[:, e], self.zk[:, e], p.cur_bits, self.variant)
            self.cv[:, e], self.sv[:, e], self.zv[:, e] = chain_variant(
                self.cv[:, e], self.sv[:, e], self.zv[:, e], p.cur_bits, self.variant)
            self.bits[e] = p.cur_bits

    def append(self, k, v, auto_reduce=True):
        """k, v: [n_new, n_stored, 128]; the literal one-token-at-a-time process."""
        for i in range(len(k)):
            self.append_token(k[i], v[i], auto_reduce)

    def append_bulk(self, k, v):
        """Vectorized equivalent of ``append`` with auto_reduce (pinned equal to it in the
        tests): by Eq. 3's chain structure the final codes do not depend on when a token
        was shifted, only on the final width."""
        p = self.p
        k = np.asarray(k, dtype=np.float32)
        v = np.asarray(v, dtype=np.float32)
        n_new = len(k)
        n_after = p.n_tokens + n_new
        r, ok = p.reduces_needed_for(n_after)
        if not ok:
            raise OverflowError("capacity")
        for _ in range(r):
            self.reduce()
        t0 = p.n_tokens
        xk = (k * self.inv_lam[None]).astype(np.float32)
        ck, sk, zk = quantize_asym(xk, 16)
        cv, sv, zv = quantize_asym(v, 16)
        self.ck[:, t0:n_after], self.sk[:, t0:n_after], self.zk[:, t0:n_after] = (
            ck.transpose(1, 0, 2), sk.T, zk.T)
        self.cv[:, t0:n_after], self.sv[:, t0:n_after], self.zv[:, t0:n_after] = (
            cv.transpose(1, 0, 2), sv.T, zv.T)
        self.bits[t0:n_after] = 16
        old_body_end = p.n_sink_at(t0) + p.n_body_at(t0)
        p.n_tokens = n_after
        new_body_end = p.n_sink_at(n_after) + p.n_body_at(n_after)
        lo, hi = max(old_body_end, p.n_sink), new_body_end
        if hi > lo:
            self.ck[:, lo:hi], self.sk[:, lo:hi], self.zk[:, lo:hi] = chain_variant(
                self.ck[:, lo:hi], self.sk[:, lo:hi], self.zk[:, lo:hi], p.cur_bits, self.variant)
            self.cv[:, lo:hi], self.sv[:, lo:hi], self.zv[:, lo:hi] = chain_variant(
                self.cv[:, lo:hi], self.sv[:, lo:hi], self.zv[:, lo:hi], p.cur_bits, self.variant)
            self.bits[lo:hi] = p.cur_bits

    # -- Eq. 9 + softmax attention over all cached tokens ------------------------
    def decode_attention(self, q, sm_scale=None):
        """q: [n_stored, G, 128] fp32 (bf16-exact) queries of the G heads sharing each
        stored KV-head slice.  Returns fp32 [n_stored, G, 128].

        P = (Q Lambda) . dequant(K Lambda^-1)^T (Eq. 9), softmax over all N cached tokens
        (the one just appended included), times dequant(V); everything in float64."""
        n = self.p.n_tokens
        q = np.asarray(q, dtype=np.float32)
        scale = 1.0 / np.sqrt(float(HEAD_DIM)) if not sm_scale else float(sm_scale)
        out = np.empty(q.shape, dtype=np.float32)
        for s in range(self.S):
            qs = q[s].astype(np.float64) * self.lam[s].astype(np.float64)[None, :]
            kh = dequantize(self.ck[s, :n], self.sk[s, :n], self.zk[s, :n])      # [n,128]
            vh = dequantize(self.cv[s, :n], self.sv[s, :n], self.zv[s, :n])
            sc = scale * (qs @ kh.T)                                             # [G,n]
            sc = sc - sc.max(axis=1, keepdims=True)
            pr = np.exp(sc)
            pr = pr / pr.sum(axis=1, keepdims=True)
            out[s] = (pr @ vh).astype(np.float32)
        return out

    # -- what the parity tests compare --------------------------------------------
    def export_slice(self, s, is_value):
        n = self.p.n_tokens
        if is_value:
            return self.cv[s, :n].copy(), self.sv[s, :n].copy(), self.zv[s, :n].copy(), self.bits[:n].copy()
        return self.ck[s, :n].copy(), self.sk[s, :n].copy(), self.zk[s, :n].copy(), self.bits[:n].copy()


# --------------------------------------------------------------------------
# Sec. 3.2: block-wise bit allocation (Eq. 6-8) and the sensitivity stand-in
# --------------------------------------------------------------------------
def allocate_bits_brute_force(sensitivity, mem_bytes, budget_bytes):
    """Eq. 6-8 by exhaustive search: one choice per block, minimal summed sensitivity subject to the
    summed memory <= budget.  Returns (choice index per block, cost) or (None, inf) if nothing fits.
    Ties: less memory first, then the lexicographically smallest choice vector.  Small inputs only."""
    import itertools
    sens = np.asarray(sensitivity, dtype=np.float64)
    mem = np.asarray(mem_bytes, dtype=np.int64)
    layers, c = sens.shape
    best = (np.inf, np.inf, None)
    for combo in itertools.product(range(c), repeat=layers):
        m = int(sum(mem[i, combo[i]] for i in range(layers)))
        if m > budget_bytes:
            continue
        s = float(sum(sens[i, combo[i]] for i in range(layers)))
        if (s, m, combo) < best:
            best = (s, m, combo)
    return (None, np.inf) if best[2] is None else (list(best[2]), best[0])


def quantization_sensitivity(k, v, bits: int):
    """Stand-in for Eq. 5 without the gradient factor (it needs the model): ||K - Q_b(K)||_1 +
    ||V - Q_b(V)||_1 with the per-token group quantizer of Eq. 1-2 at ``bits``."""
    total = 0.0
    for x in (k, v):
        x = np.asarray(x, dtype=np.float32)
        c, s, z = quantize_asym(x, bits)
        total += float(np.abs(dequantize(c, s, z) - x).sum())
    return total


# --------------------------------------------------------------------------
# Sec. 3.3: calibration of Lambda with positional interpolation (Eq. 10-12)
# --------------------------------------------------------------------------
def rope_interpolated(x_pre, positions, pos_scale: float = 1.0, theta: float = 10000.0):
    """Eq. 12 (Eq. 11 when pos_scale = 1): rotate channel pairs (i, i + d/2) of x_pre [n, ..., d] by the angle
    pos_scale * m * theta^(-2i/d) of each token's position m.  float64."""
    x = np.asarray(x_pre, dtype=np.float64)
    d = x.shape[-1]
    half = d // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * pos_scale * inv_freq[None, :]
    shape = (x.shape[0],) + (1,) * (x.ndim - 2) + (half,)
    c, s = np.cos(ang).reshape(shape), np.sin(ang).reshape(shape)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x1 * s + x2 * c], axis=-1)


def calibrate_lambda(k_pre, pos_scale: float = 1.0, theta: float = 10000.0, alpha: float = 0.5, floor: float = 1e-5):
    """Eq. 10 on Keys rotated per Eq. 12.  k_pre: [n_tokens, n_seq, kv_heads, d], token t at position t.
    lambda[h, i] = max(max_{t, seq} |K_rot[t, seq, h, i]|, floor)^alpha (absolute maxima, as in the
    channel-equalization scheme the section builds on)."""
    k = np.asarray(k_pre, dtype=np.float64)
    rot = rope_interpolated(k, np.arange(k.shape[0]), pos_scale, theta)
    amax = np.abs(rot).max(axis=(0, 1))
    return np.maximum(amax, floor) ** alpha


# --------------------------------------------------------------------------
# Sec. 4.1.1: alpha of Eq. 10 by grid search on the attention reconstruction loss
# --------------------------------------------------------------------------
def causal_self_attention(q, k, v, group: int):
    """softmax(Q K^T / sqrt(d)) V with a causal mask, per sequence and head, in float64.
    q: [n, n_seq, kv_heads * group, d]; k, v: [n, n_seq, kv_heads, d]; query head h reads KV head h // group
    (grouped-query attention); token t attends to tokens 0..t.  Returns [n, n_seq, kv_heads * group, d]."""
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    n, n_seq, q_heads, d = q.shape
    out = np.empty_like(q)
    mask = np.tril(np.ones((n, n), dtype=bool))
    for b in range(n_seq):
        for h in range(q_heads):
            sc = (q[:, b, h] @ k[:, b, h // group].T) / np.sqrt(float(d))
            sc = np.where(mask, sc, -np.inf)
            sc = sc - sc.max(axis=1, keepdims=True)
            pr = np.exp(sc)
            pr = pr / pr.sum(axis=1, keepdims=True)
            out[:, b, h] = pr @ v[:, b, h // group]
    return out


def quantize_progressively(x, bits: int):
    """What the cache holds for a token that has reached ``bits``: Eq. 1-2 at 16 bit on fp32 values, then
    the Eq. 3 chain down to ``bits``; returned dequantized (float64)."""
    c16, s16, z = quantize_asym(np.asarray(x, dtype=np.float32), 16)
    c, s = chain_to(c16, s16, bits)
    return dequantize(c, s, z)


def attention_reconstruction_losses(k_pre, q_pre, v, group: int, bits: int, alphas, pos_scale: float = 1.0,
                                    theta: float = 10000.0, floor: float = 1e-5):
    """Loss of the self-attention operator for each alpha of the grid (Sec. 4.1.1), on one block's calibration
    tensors: k_pre, v [n, n_seq, kv_heads, d] and q_pre [n, n_seq, kv_heads * group, d], Keys and Queries
    before RoPE, token t at position t.

    Keys and Queries are rotated with the interpolated RoPE of Eq. 12; lambda(alpha) follows Eq. 10 on the
    rotated Keys; the quantized operator is Eq. 9, (Q Lambda) . Q_b(K Lambda^-1)^T, with K Lambda^-1 formed
    in fp32 from the fp32 lambda the cache would be configured with, K and V both quantized the way the cache
    holds ``bits``-bit tokens.  The loss is the mean squared difference between the causal self-attention
    output of the unquantized tensors and that of the quantized ones, over all tokens, sequences, heads and
    channels.  Returns a float64 array, one loss per alpha."""
    k_pre, q_pre, v = (np.asarray(a, dtype=np.float64) for a in (k_pre, q_pre, v))
    n = k_pre.shape[0]
    pos = np.arange(n)
    k_rot = rope_interpolated(k_pre, pos, pos_scale, theta)
    q_rot = rope_interpolated(q_pre, pos, pos_scale, theta)
    amax = np.maximum(np.abs(k_rot).max(axis=(0, 1)), floor)          # [kv_heads, d]
    ref = causal_self_attention(q_rot, k_rot, v, group)
    v_hat = quantize_progressively(v, bits)
    k32 = k_rot.astype(np.float32)
    losses = []
    for alpha in alphas:
        lam = (amax ** float(alpha)).astype(np.float32)              # Eq. 10
        inv = (np.float32(1.0) / lam).astype(np.float32)
        k_hat = quantize_progressively((k32 * inv[None, None]).astype(np.float32), bits)
        q_eq = q_rot * np.repeat(lam.astype(np.float64), group, axis=0)[None, None]
        got = causal_self_attention(q_eq, k_hat, v_hat, group)
        losses.append(float(np.mean((got - ref) ** 2)))
    return np.asarray(losses, dtype=np.float64)


def alpha_grid(n_grid: int = 20):
    """The search grid over [0, 1]: n_grid equally spaced values starting at 0, alpha_j = j / n_grid (the
    convention of the grid search the section cites; alpha = 1 itself is not visited)."""
    return np.arange(n_grid, dtype=np.float64) / float(n_grid)


def grid_search_alpha(k_pre, q_pre, v, group: int, bits: int, n_grid: int = 20, **kw):
    """Sec. 4.1.1: the alpha of the grid with the smallest reconstruction loss (the first one on ties).
    Returns (alpha, losses)."""
    alphas = alpha_grid(n_grid)
    losses = attention_reconstruction_losses(k_pre, q_pre, v, group, bits, alphas, **kw)
    return float(alphas[int(np.argmin(losses))]), losses
