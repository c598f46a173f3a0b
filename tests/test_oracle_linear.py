"""Pins of the oracle's linear layer (Section 2: f^(i)(x^(i)) = x^(i) W^(i), BF16 in and out): hand-computed
values, ties, the single rounding from the exact sum, identity and scaling laws, and the two oracles against
each other."""
import numpy as np
import pytest

from util import bf16_bits, bf16_value


def _b(vals):
    return bf16_bits(np.asarray(vals, dtype=np.float64))


def _val(bits) -> float:
    return float(bf16_value(np.asarray([bits], np.uint16))[0])


@pytest.fixture
def rng():
    return np.random.default_rng(20241107)


def _both(corc, norc):
    return [("c", corc.linear_bf16), ("np", norc.linear_bf16)]


def test_hand_computed(corc, norc):
    x = _b([[1.0, 2.0, 3.0], [0.0, -1.0, 0.5]])
    w = _b([[1.0, 1.0, 1.0], [0.5, -1.0, 2.0]])          # [E = 2][K = 3]
    for name, f in _both(corc, norc):
        y = f(x, w)
        assert y.tolist() == [[0x40C0, 0x4090], [0xBF00, 0x4000]], name   # 6, 4.5; -0.5, 2


def test_ties_go_to_even(corc, norc):
    """Near 256 the BF16 spacing is 2: 257 lies between 256 (even) and 258, 259 between 258 and 260 (even)."""
    x = _b([[1.0, 1.0]])
    for name, f in _both(corc, norc):
        assert f(x, _b([[256.0, 1.0]]))[0, 0] == 0x4380, name     # 256
        assert f(x, _b([[258.0, 1.0]]))[0, 0] == 0x4382, name     # 260
        assert f(x, _b([[256.0, 3.0]]))[0, 0] == 0x4382, name     # 259 -> 260
        assert f(x, _b([[-256.0, -1.0]]))[0, 0] == 0xC380, name   # sign symmetric


def test_one_rounding_from_the_exact_sum(corc, norc):
    """1 + 2^-8 + 2^-30 is just above the midpoint of 1 and 1 + 2^-7: the exact sum rounds UP.  Rounding to
    binary32 first would land on the midpoint and then go to even (1.0): the oracle must not do that."""
    x = _b([[1.0, 1.0, 1.0]])
    w = _b([[1.0, 2.0 ** -8, 2.0 ** -30]])
    for name, f in _both(corc, norc):
        assert f(x, w)[0, 0] == 0x3F81, name
    twice = np.float32(1.0 + 2.0 ** -8 + 2.0 ** -30)
    assert int(bf16_bits(np.asarray([twice]))[0]) == 0x3F80                      # the double rounding this pin excludes


def test_identity_weight_passes_bf16_through(corc, norc, rng):
    K = 24
    x = rng.integers(0, 1 << 16, size=(7, K)).astype(np.uint16)
    x[(x & 0x7F80) == 0x7F80] = 0x3F80                            # no Inf / NaN
    x[(x & 0x7F80) == 0] = 0                                      # no subnormals (a product with 1 is exact anyway)
    w = np.zeros((K, K), np.uint16)
    w[np.arange(K), np.arange(K)] = 0x3F80
    for name, f in _both(corc, norc):
        y = f(x, w)
        assert np.array_equal(y & 0x7FFF, x & 0x7FFF), name       # value preserved (a -0 sum is +0)
        nz = (x & 0x7FFF) != 0
        assert np.array_equal(y[nz], x[nz]), name


def test_power_of_two_scaling_commutes(corc, norc, rng):
    T, K, E = 5, 40, 9
    x = _b(rng.normal(0, 1, (T, K)))
    w = _b(rng.normal(0, 1, (E, K)))
    x4 = ((x.astype(np.int32) + (2 << 7)) & 0xFFFF).astype(np.uint16)   # exponent + 2: every value times 4
    for name, f in _both(corc, norc):
        y, y4 = f(x, w), f(x4, w)
        assert np.array_equal(y4.astype(np.int32), y.astype(np.int32) + (2 << 7)), name


@pytest.mark.parametrize("T,K,E", [(3, 8, 8), (17, 72, 40), (33, 200, 24), (4, 1000, 16)])
def test_c_and_numpy_agree(corc, norc, rng, T, K, E):
    x = _b(rng.normal(0, 1, (T, K)))
    w = _b(rng.normal(0, 0.05, (E, K)))
    a, b = corc.linear_bf16(x, w), norc.linear_bf16(x, w)
    assert np.array_equal(a, b)
    # and against exact rational arithmetic on a few entries
    from fractions import Fraction
    for (t, j) in [(0, 0), (T - 1, E - 1), (T // 2, E // 3)]:
        exact = sum(Fraction(_val(x[t, c])) * Fraction(_val(w[j, c])) for c in range(K))
        got = Fraction(_val(a[t, j]))
        lo, hi = Fraction(_val(int(a[t, j]) - 1)), Fraction(_val(int(a[t, j]) + 1))
        if got < 0:
            lo, hi = hi, lo
        assert abs(exact - got) <= min(abs(exact - lo), abs(exact - hi)), (t, j)
