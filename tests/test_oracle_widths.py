"""Pins for the oracle at code widths other than 4 bits (Section 4 / Figure 3): closed-form bit count, brute-force nearest level, a bit stream written out with
Python integers, the error bound of a symmetric quantiser, and the two oracles against each other."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle_np
from util import bf16_bits as f32_to_bf16_bits, bf16_value


def bf16_bits_to_f32(bits):
    return bf16_value(bits).astype(np.float32)

WIDTHS = [2, 3, 5, 6, 7, 8]


@pytest.mark.parametrize("bits", WIDTHS + [4])
def test_bits_per_value_closed_form(corc, bits):
    """b + (16 - b) k / E bits per value when the code stream needs no padding (Section 4's count with
    4 replaced by b)."""
    for E, k, T in [(256, 4, 64), (5120, 80, 128), (8192, 128, 16), (4608, 72, 128)]:
        assert (T * (E - k) * bits) % 128 == 0
        P = corc.payload_bytes(T, E, k, bits)
        assert P == oracle_np.payload_bytes(T, E, k, bits)
        assert Fraction(8 * P, T * E) == bits + Fraction((16 - bits) * k, E)


@pytest.mark.parametrize("bits", WIDTHS)
def test_nearest_level_bruteforce(corc, bits):
    """The code is the integer of [-2^(b-1), 2^(b-1)-1] nearest to fl(x * inv_s), ties to the even one
    (exact comparison in rationals over every candidate)."""
    rng = np.random.default_rng(bits)
    lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    xs = f32_to_bf16_bits(rng.normal(0, 3, 300).astype(np.float32))
    # add exact half-way points and out-of-range values
    extra = np.array([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, hi + 0.5, lo - 0.5, 1e6, -1e6, 0.0], np.float32)
    xs = np.concatenate([xs, f32_to_bf16_bits(extra)])
    for inv_s in (np.float32(1.0), np.float32(0.37), np.float32(7.0)):
        for xb in xs:
            x = bf16_bits_to_f32(np.array([xb], np.uint16))[0]
            u = np.float32(x) * inv_s                      # one binary32 rounding
            uf = Fraction(float(u))
            best = min(range(lo, hi + 1), key=lambda q: (abs(uf - q), q % 2))
            assert corc.quantize_one(int(xb), float(inv_s), bits) == best, (bits, x, inv_s)


@pytest.mark.parametrize("bits", WIDTHS + [4])
def test_bit_stream_written_with_python_integers(corc, norc, bits):
    """Code p occupies bits [p b, p b + b) of a little-endian stream: the same bytes as one big integer
    sum(u_p << (p b)) written least significant byte first."""
    T, E = 5, 24
    hp = np.array([3, 17], np.int32)
    k, L = len(hp), E - len(hp)
    rng = np.random.default_rng(100 + bits)
    y = f32_to_bf16_bits(rng.normal(0, 2, (T, E)).astype(np.float32))
    inv = np.full(E, 1.0, np.float32)
    payload = corc.quantize_pack(y, hp, inv, bits)
    lp = corc.lp_index(E, hp)
    big = 0
    for t in range(T):
        for c in range(L):
            q = corc.quantize_one(int(y[t, lp[c]]), 1.0, bits)
            big |= (q & ((1 << bits) - 1)) << ((t * L + c) * bits)
    nb = corc.lp_bytes(T, E, k, bits)
    assert payload[:nb].tobytes() == big.to_bytes(nb, "little")
    assert payload[nb:].view(np.uint16).reshape(T, k).tolist() == y[:, hp].tolist()
    assert np.array_equal(payload, norc.quantize_pack(y, hp, inv, bits))


@pytest.mark.parametrize("bits", WIDTHS)
def test_round_trip_error_bound_and_sum(corc, norc, bits):
    """Inside the calibrated range a symmetric quantiser is off by at most half a step; the reduced sum is
    the sum of code * step over the devices (binary64, exact products)."""
    N, T, E = 3, 9, 40
    hp = np.array([0, 7, 13, 39], np.int32)
    rng = np.random.default_rng(7 * bits)
    R = (rng.uniform(1.0, 8.0, (N, E))).astype(np.float32)
    s, inv = corc.params(R, bits)
    s2, inv2 = norc.params(R, bits)
    assert np.array_equal(s, s2) and np.array_equal(inv, inv2)
    assert np.array_equal(s, (R / np.float32((1 << bits) - 1)).astype(np.float32))
    ys, pls = [], []
    for i in range(N):
        # values within the representable part of the range: |x| <= (2^(b-1) - 1) s
        lim = ((1 << (bits - 1)) - 1) * s[i]
        x = (rng.uniform(-1, 1, (T, E)) * lim[None, :]).astype(np.float32)
        yb = f32_to_bf16_bits(x)
        ys.append(yb)
        pls.append(corc.quantize_pack(yb, hp, inv[i], bits))
        assert np.array_equal(pls[-1], norc.quantize_pack(yb, hp, inv[i], bits))
        codes, hpv = norc.unpack(pls[-1], T, E, len(hp), bits)
        lp = corc.lp_index(E, hp)
        xr = bf16_bits_to_f32(yb)[:, lp].astype(np.float64)
        err = np.abs(codes.astype(np.float64) * s[i, lp][None, :] - xr)
        # half a step, plus the rounding of the product x * fl(1/s) (a few ulps of the code magnitude)
        assert (err <= 0.5 * s[i, lp][None, :] * (1 + 1e-5) + 1e-6 * np.abs(xr)).all()
    ref, chain = corc.dequant_reduce(pls, T, E, hp, s, bits=bits)
    ref_np = norc.dequant_reduce(pls, T, E, hp, s, bits)
    assert np.array_equal(ref, ref_np)
    assert np.allclose(chain, ref, rtol=1e-6, atol=1e-6)
    sel = bf16_bits_to_f32(np.stack([y[:, hp] for y in ys])).astype(np.float64).sum(axis=0)
    assert np.array_equal(ref[:, hp], sel)


@pytest.mark.parametrize("bits", WIDTHS)
def test_c_and_numpy_oracles_agree_on_random_inputs(corc, norc, bits):
    rng = np.random.default_rng(bits + 40)
    T, E = 33, 96
    hp = np.sort(rng.permutation(E)[:8]).astype(np.int32)
    y = f32_to_bf16_bits((rng.normal(0, 1, (T, E)) * rng.lognormal(0, 1, E)[None, :]).astype(np.float32))
    R = (2 * np.abs(bf16_bits_to_f32(y)).max(axis=0)).astype(np.float32)
    s, inv = corc.params(R, bits)
    a = corc.quantize_pack(y, hp, inv, bits)
    b = norc.quantize_pack(y, hp, inv, bits)
    assert np.array_equal(a, b)
    ref, _ = corc.dequant_reduce([a, a], T, E, hp, np.stack([s, s]), bits=bits)
    assert np.array_equal(ref, norc.dequant_reduce([a, a], T, E, hp, np.stack([s, s]), bits))
