"""Pins for the oracle's quantizer (Eq. 1-2), the Equivalent Right Shift (Eq. 3, App. D) and the
canonical packing.  None of these re-type the oracle's own formula: they use closed forms, exact
rational arithmetic, exhaustive enumeration or hand-computed cases."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import pmkvq_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- Eq. 3 ----
def test_eq3_constants_match_paper():
    for b, mult, add, shift, sf in _rows("eq3_constants.txt"):
        b = int(b)
        assert O.shift_multiplier(b) == int(mult) == 2 ** (2 * b) - 2 ** b + 1
        # the oracle's step on the all-zero code and on the maximum code shows addend and shift
        assert int(O.shift_reduce(np.array([0]), b)[0]) == (int(mult) * int(add)) >> int(shift) == 0
        s2 = np.float32(0.375)
        assert O.reduce_scale(s2, b) == np.float32(float(s2) * int(sf))


@pytest.mark.parametrize("b", [8, 4, 2])
def test_eq3_exhaustive_is_nearest_integer_division(b):
    """App. D: Eq. 3 equals rounding X_2b / (2^b + 1) to the nearest integer (no ties exist
    because 2^b + 1 is odd), for every 2b-bit input."""
    x = np.arange(1 << (2 * b), dtype=np.uint32)
    got = O.shift_reduce(x, b).astype(np.int64)
    d = (1 << b) + 1
    want = np.array([int(Fraction(int(v), d) + Fraction(1, 2)) for v in x.tolist()]) if b < 8 else \
        (2 * x.astype(np.int64) + d) // (2 * d)
    assert np.array_equal(got, want)
    # Euclidean-division form of the proof: q if r <= 2^(b-1) else q + 1
    q, r = np.divmod(x.astype(np.int64), d)
    assert np.array_equal(got, q + (r > (1 << (b - 1))))
    assert got[0] == 0 and got[-1] == (1 << b) - 1          # end points map to end points
    assert np.all(np.diff(got) >= 0)                          # monotone


def test_eq3_identity_and_4to2_table():
    for b in (8, 4, 2):
        assert O.shift_multiplier(b) * (2 ** b + 1) == 2 ** (3 * b) + 1
    # 4 -> 2 bit: every 4-bit level to the nearest of {0, 5, 10, 15} / 5
    assert O.shift_reduce(np.arange(16), 2).tolist() == [0, 0, 0, 1, 1, 1, 1, 1, 2, 2, 2, 2, 2, 3, 3, 3]


def _exact_quant(xs, bits):
    """Eq. 1-2 in exact rational arithmetic with the proof's rounding interval [X-1/2, X+1/2)."""
    z, m = min(xs), max(xs)
    s = Fraction(m - z, (1 << bits) - 1)
    return [int((Fraction(x - z) / s + Fraction(1, 2)).__floor__()) for x in xs]


@pytest.mark.parametrize("b", [8, 4, 2])
def test_theorem_progressive_equals_direct_in_exact_arithmetic(b):
    """Theorem of App. D: shifting the exact 2b-bit quantization gives the exact b-bit one."""
    rng = np.random.default_rng(b)
    for _ in range(40):
        xs = [Fraction(int(v), 64) for v in rng.integers(-2000, 2000, size=24)]
        if min(xs) == max(xs):
            continue
        c2b = np.array(_exact_quant(xs, 2 * b))
        assert O.shift_reduce(c2b, b).tolist() == _exact_quant(xs, b)


def test_chain_scale_matches_direct_scale():
    """S_b = (2^b+1) S_2b reproduces (max - Z)/(2^b - 1) (App. D) up to the fp32 roundings."""
    rng = np.random.default_rng(0)
    x = rng.standard_normal((64, 128)).astype(np.float32)
    c16, s16, z = O.quantize_asym(x, 16)
    for bits in (8, 4, 2):
        c, s = O.chain_to(c16, s16, bits)
        direct = (x.max(-1).astype(np.float64) - z) / ((1 << bits) - 1)
        assert np.allclose(s, direct, rtol=4 * 2.0 ** -24, atol=0)
        assert c.max() <= (1 << bits) - 1
        # post-chain reconstruction error bounded by S_b / 2 (+ the INT16 half step)
        err = np.abs(O.dequantize(c, s, z) - x)
        assert np.all(err <= (s[:, None].astype(np.float64) / 2 + s16[:, None] / 2) * (1 + 1e-5))


# --------------------------------------------------------------- Eq. 1-2 ----
def test_quantizer_hand_cases():
    # group [0, 1, 2, 3] at 2 bit: Z = 0, S = 1, codes = values
    c, s, z = O.quantize_asym(np.array([[0.0, 1.0, 2.0, 3.0]], np.float32), 2)
    assert c.tolist() == [[0, 1, 2, 3]] and s[0] == 1.0 and z[0] == 0.0
    # [-1, 0, 0.5, 1] at 2 bit: Z = -1, S = 2/3; (x-Z)/S = 0, 1.5, 2.25, 3 -> 0, 2 (tie to even), 2, 3
    c, s, z = O.quantize_asym(np.array([[-1.0, 0.0, 0.5, 1.0]], np.float32), 2)
    assert z[0] == -1.0 and s[0] == np.float32(2.0) / np.float32(3.0)
    assert c.tolist() == [[0, 2, 2, 3]]
    # ties go to even: values 0.5 and 2.5 steps above Z with S = 1
    c, s, z = O.quantize_asym(np.array([[0.0, 0.5, 2.5, 3.0]], np.float32), 2)
    assert c.tolist() == [[0, 0, 2, 3]]
    # constant group: S = 0, codes 0, dequantizes to Z
    c, s, z = O.quantize_asym(np.full((1, 8), 1.25, np.float32), 16)
    assert s[0] == 0 and z[0] == 1.25 and not c.any()
    assert np.all(O.dequantize(c, s, z) == 1.25)


@pytest.mark.parametrize("bits", [16, 8, 4, 2])
def test_quantizer_invariants(bits):
    rng = np.random.default_rng(bits)
    x = (rng.standard_normal((200, 128)) * rng.uniform(0.1, 30, (200, 1))).astype(np.float32)
    c, s, z = O.quantize_asym(x, bits)
    qmax = (1 << bits) - 1
    assert np.array_equal(z, x.min(-1)) and c.min() >= 0 and c.max() <= qmax
    assert np.all(c[np.arange(200), x.argmin(-1)] == 0)
    assert np.all(c[np.arange(200), x.argmax(-1)] == qmax)
    # Eq. 2 in float64 agrees with the fp32 scale to one rounding
    assert np.allclose(s, (x.max(-1).astype(np.float64) - z) / qmax, rtol=2.0 ** -23, atol=0)
    # round-trip error <= S/2 (the bound the method states); the slack covers the three fp32 roundings of the
    # recipe (x - Z, the division, S itself), each at most 2^-24 of the group's range
    err = np.abs(O.dequantize(c, s, z) - x.astype(np.float64))
    rng_ = (x.max(-1).astype(np.float64) - z)[:, None]
    assert np.all(err <= s[:, None].astype(np.float64) / 2 + 3 * 2.0 ** -24 * rng_)


def test_quantizer_matches_exact_rational_on_non_ties():
    """Codes from the fp32 recipe equal exact-arithmetic rounding wherever the exact value is
    not within 0.05 of a rounding boundary (the fp32 sub / div / scale roundings move a 16-bit code's
    pre-rounding value by at most ~3 * 65535 * 2^-24 = 0.012)."""
    rng = np.random.default_rng(5)
    x = rng.standard_normal((8, 128)).astype(np.float32)
    c, s, z = O.quantize_asym(x, 16)
    for g in range(8):
        xs = [Fraction(float(v)) for v in x[g]]
        zf, mf = min(xs), max(xs)
        sf = (mf - zf) / 65535
        for i, v in enumerate(xs):
            t = (v - zf) / sf
            frac = t - t.__floor__()
            if abs(frac - Fraction(1, 2)) > Fraction(1, 20):
                assert int(c[g, i]) == int((t + Fraction(1, 2)).__floor__())


# ------------------------------------------------------------- variants ----
def test_ablation_shift_variants():
    """Sec. 4.4.1: Direct keeps the upper b bits with S*(2^b+1); Modified maps the mean of the
    levels sharing the upper bits: S*2^b and Z + (S_b - S_2b)/2."""
    c4 = np.arange(16, dtype=np.uint16)
    s, z = np.float32(0.5), np.float32(-1.0)
    cd, sd, zd = O.direct_right_shift(c4, s, z, 2)
    assert cd.tolist() == [v >> 2 for v in range(16)] and sd == np.float32(2.5) and zd == z
    cm, sm, zm = O.modified_right_shift(c4, s, z, 2)
    assert cm.tolist() == cd.tolist() and sm == np.float32(2.0) and zm == np.float32(-1.0 + 0.75)
    # modified: dequantized level = mean of the four 4-bit levels that share the upper 2 bits
    lv4 = s * np.arange(16) + z
    for q in range(4):
        assert np.isclose(sm * q + zm, lv4[4 * q: 4 * q + 4].mean())


def test_shift_variant_chains_and_error_ordering():
    """Chains of the three shrinking strategies (Sec. 4.4.1).  Direct / Modified codes are the upper
    bits of the INT16 code; Modified dequantizes to the centre of the merged bin; on N(0,1) groups the
    mean squared reconstruction error after 16 -> 2 orders as Equivalent < Modified < Direct, the
    mechanics behind the accuracy ordering of Table 4."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal((512, 128)).astype(np.float32)
    c16, s16, z16 = O.quantize_asym(x, 16)
    mse = {}
    for variant in (O.SHIFT_EQUIVALENT, O.SHIFT_DIRECT, O.SHIFT_MODIFIED):
        for bits in (8, 4, 2):
            c, s, z = O.chain_variant(c16, s16, z16, bits, variant)
            assert c.max() <= (1 << bits) - 1
            if variant != O.SHIFT_EQUIVALENT:
                assert np.array_equal(c, c16 >> (16 - bits))
            if variant == O.SHIFT_MODIFIED:     # level = centre of the 2^(16-bits) fine levels it replaces
                k = 1 << (16 - bits)
                centre = s16.astype(np.float64) * (k - 1) / 2 + z16
                assert np.allclose(z, centre, rtol=1e-5, atol=1e-6)
                assert np.allclose(s, s16.astype(np.float64) * k, rtol=1e-6)
            if variant == O.SHIFT_EQUIVALENT:
                c_ref, s_ref = O.chain_to(c16, s16, bits)
                assert np.array_equal(c, c_ref) and np.array_equal(s, s_ref) and np.array_equal(z, z16)
        err = np.abs(O.dequantize(c, s, z) - x)            # c, s, z: the 2-bit end of the chain
        step = s.astype(np.float64)[:, None]
        if variant == O.SHIFT_DIRECT:
            # bins of a quarter of the range, levels a third apart: off by up to 3/4 of a step at the ends
            assert (err <= step * 0.75 * 1.001 + s16[:, None]).all() and (err > step * 0.6).any()
        else:
            assert (err <= step * 0.5 * 1.001 + s16[:, None]).all()
        mse[variant] = float(np.mean(err ** 2))
    assert mse[O.SHIFT_EQUIVALENT] < mse[O.SHIFT_DIRECT] and mse[O.SHIFT_MODIFIED] < mse[O.SHIFT_DIRECT]


# -------------------------------------------------------------- packing ----
def test_canonical_packing_hand_and_roundtrip():
    codes = np.zeros(128, np.uint16)
    codes[:8] = [1, 2, 3, 0, 3, 3, 0, 1]
    p2 = O.pack_canonical(codes, 2)
    assert p2.shape == (32,) and p2[0] == (1 | 2 << 2 | 3 << 4 | 0 << 6) and p2[1] == (3 | 3 << 2 | 0 << 4 | 1 << 6)
    codes4 = np.zeros(128, np.uint16); codes4[:4] = [0xA, 0x1, 0xF, 0x3]
    p4 = O.pack_canonical(codes4, 4)
    assert p4.shape == (64,) and p4[0] == 0x1A and p4[1] == 0x3F
    c16 = np.zeros(128, np.uint16); c16[0] = 0xBEEF
    p16 = O.pack_canonical(c16, 16)
    assert p16.shape == (256,) and p16[0] == 0xEF and p16[1] == 0xBE
    rng = np.random.default_rng(1)
    for bits in (16, 8, 4, 2):
        c = rng.integers(0, 1 << bits, size=(5, 128)).astype(np.uint16)
        assert np.array_equal(O.unpack_canonical(O.pack_canonical(c, bits), bits), c)
        assert O.pack_canonical(c, bits).shape == (5, 16 * bits)
