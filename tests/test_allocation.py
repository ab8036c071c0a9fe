"""Block-wise bit allocation (Sec. 3.2, Eq. 6-8): the library's exact dynamic program against the
exhaustive definition in the oracle, plus the limits the formulation fixes.  Host only."""
import numpy as np
import pytest

from oracle import pmkvq_oracle as O
from paper_2505_18610_b200 import binding as B
from paper_2505_18610_b200 import synth


def _mem(layers, widths, n_tokens=4096, n_slices=8):
    return np.array([[2 * n_slices * n_tokens * O.tokbytes(b) for b in widths] for _ in range(layers)], dtype=np.uint64)


def test_hand_case():
    # two blocks, widths {2,4}: memory 10/20 each, budget 30 -> exactly one block may take 4 bits: the one that gains more
    sens = np.array([[5.0, 1.0], [9.0, 2.0]])
    mem = np.array([[10, 20], [10, 20]], dtype=np.uint64)
    fbit, cost = B.allocate_bits([2, 4], sens, mem, 30)
    assert fbit == [2, 4] and cost == 5.0 + 2.0
    assert B.allocate_bits([2, 4], sens, mem, 40) == ([4, 4], 3.0)
    assert B.allocate_bits([2, 4], sens, mem, 20) == ([2, 2], 14.0)
    with pytest.raises(B.PmkvqError):
        B.allocate_bits([2, 4], sens, mem, 19)
    # the same hand-computed answers pin the exhaustive oracle the other tests compare against
    assert O.allocate_bits_brute_force(sens, mem, 30) == ([0, 1], 7.0)
    assert O.allocate_bits_brute_force(sens, mem, 40) == ([1, 1], 3.0)
    assert O.allocate_bits_brute_force(sens, mem, 20) == ([0, 0], 14.0)
    assert O.allocate_bits_brute_force(sens, mem, 19) == (None, np.inf)


def test_sensitivity_of_hand_made_tokens():
    """The oracle's sensitivity (L1 error of the per-token quantizer) on tokens whose codes can be written down:
    a token with values {0, 1, 2, 3} (times any scale) is exact at 2 bit, one with {0, 1.5, 3} loses 0.5 on
    its middle value at 2 bit (code 1 or 2, S = 1) and nothing at 4 bit (S = 0.2, code 7.5 -> tie, error 0.1)."""
    exact = np.tile(np.array([0.0, 1.0, 2.0, 3.0], np.float32), 32)[None, :] * 0.25
    assert O.quantization_sensitivity(exact, exact, 2) == 0.0
    tok = np.zeros((1, 128), np.float32); tok[0, 1] = 1.5; tok[0, 2] = 3.0
    assert abs(O.quantization_sensitivity(tok, np.zeros_like(tok), 2) - 0.5) < 1e-6
    # 4 bit: S = 3 / 15 = 0.2, 1.5 / 0.2 = 7.5 rounds to 8 (half to even) -> 1.6: error 0.1
    assert abs(O.quantization_sensitivity(tok, np.zeros_like(tok), 4) - 0.1) < 1e-6
    # errors add over K and V and over tokens
    both = O.quantization_sensitivity(np.concatenate([tok, tok]), tok, 2)
    assert abs(both - 1.5) < 1e-6


@pytest.mark.parametrize("seed", range(6))
def test_matches_exhaustive_search(seed):
    rng = np.random.default_rng(seed)
    layers = int(rng.integers(2, 9))
    widths = [[2, 4], [4, 8], [2, 4, 8]][seed % 3]
    # sensitivities fall with the width (more bits, less error) but differ a lot between blocks (Fig. 3)
    base = rng.uniform(0.5, 20.0, size=(layers, 1))
    sens = base * np.array([[4.0 ** -i for i in range(len(widths))]]) * rng.uniform(0.8, 1.2, size=(layers, len(widths)))
    mem = _mem(layers, widths) if seed % 2 == 0 else rng.integers(1, 40, size=(layers, len(widths))).astype(np.uint64) * 64
    lo, hi = int(mem.min(axis=1).sum()), int(mem.max(axis=1).sum())
    for budget in (lo, (lo + hi) // 2, (2 * lo + hi) // 3, hi, 2 * hi):
        want_idx, want_cost = O.allocate_bits_brute_force(sens, mem, budget)
        fbit, cost = B.allocate_bits(widths, sens, mem, budget)
        assert abs(cost - want_cost) <= 1e-9 * max(1.0, abs(want_cost))
        used = sum(int(mem[i, widths.index(fbit[i])]) for i in range(layers))
        assert used <= budget
        assert abs(sum(sens[i, widths.index(fbit[i])] for i in range(layers)) - want_cost) <= 1e-9 * max(1.0, want_cost)


def test_limits_and_monotonicity_on_synthetic_sensitivities():
    """Sensitivities from the quantizer's own error on synthetic K/V (Eq. 5 without the gradient factor):
    unbounded budget -> every block takes the widest choice; budget at the floor -> the narrowest;
    the optimum never gets worse when the budget grows; the 'average 3 bits' budget of the 2/4-bit
    schedule gives exactly half of the blocks 4 bits when all blocks have the same shape."""
    layers, widths = 8, [2, 4]
    sens = np.zeros((layers, 2))
    for l in range(layers):
        k, v = synth.make_kv(5, l, 0, 64, 1, 2, 0, 4, 15.0 + 3 * l)
        for j, b in enumerate(widths):
            sens[l, j] = O.quantization_sensitivity(k.float().numpy(), v.float().numpy(), b)
    assert (sens[:, 0] > sens[:, 1]).all()
    mem = _mem(layers, widths)
    lo, hi = int(mem[:, 0].sum()), int(mem[:, 1].sum())
    assert B.allocate_bits(widths, sens, mem, 10 * hi)[0] == [4] * layers
    assert B.allocate_bits(widths, sens, mem, lo)[0] == [2] * layers
    costs = [B.allocate_bits(widths, sens, mem, b)[1] for b in np.linspace(lo, hi, 9).astype(np.int64)]
    assert all(a >= b - 1e-9 for a, b in zip(costs, costs[1:]))
    fbit, _ = B.allocate_bits(widths, sens, mem, (lo + hi) // 2)
    assert sorted(fbit) == [2] * 4 + [4] * 4
    gain = sens[:, 0] - sens[:, 1]
    assert {i for i, b in enumerate(fbit) if b == 4} == set(np.argsort(-gain)[:4].tolist())
