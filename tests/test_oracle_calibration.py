"""Pins of the oracle's calibration (paper Section 3, Eq. (1)-(2), gamma = 0.01,
first-sequence initialisation, R = 2 max(-m, M), R-bar = sum_i R^(i))."""
import numpy as np
import pytest

from util import bf16_bits, bf16_value


def _data(seed, n_seq, S, E, scale=3.0):
    rng = np.random.default_rng(seed)
    return bf16_bits(rng.standard_normal((n_seq, S, E)) * scale)


@pytest.mark.parametrize("which", ["c", "np"])
def test_single_sequence_is_min_max(corc, norc, which):
    orc = corc if which == "c" else norc
    y = _data(1, 1, 37, 50)
    m, M, cnt = orc.calibrate(None, None, 0, y, 0.01)
    v = bf16_value(y[0])
    assert cnt == 1
    assert np.array_equal(m.astype(np.float64), v.min(axis=0))     # library min/max
    assert np.array_equal(M.astype(np.float64), v.max(axis=0))
    R, Rbar = orc.ranges(m[None], M[None])
    assert np.array_equal(R[0].astype(np.float64), 2 * np.abs(v).max(axis=0))
    assert np.array_equal(Rbar, R[0])                              # N = 1: R-bar = R


@pytest.mark.parametrize("which", ["c", "np"])
def test_ema_closed_form(corc, norc, which):
    """m_n = (1-g)^(n-1) mn_1 + g sum_{t>=2} (1-g)^(n-t) mn_t, evaluated in float64."""
    orc = corc if which == "c" else norc
    n, g = 40, 0.01
    y = _data(2, n, 16, 24)
    m, M, cnt = orc.calibrate(None, None, 0, y, g)
    v = bf16_value(y.reshape(-1, 24)).reshape(n, 16, 24)
    mn, mx = v.min(axis=1), v.max(axis=1)
    g64 = float(np.float32(g))
    w = np.array([(1 - g64) ** (n - 1)] + [g64 * (1 - g64) ** (n - t) for t in range(2, n + 1)])
    assert cnt == n
    np.testing.assert_allclose(m, (w[:, None] * mn).sum(0), rtol=1e-5)
    np.testing.assert_allclose(M, (w[:, None] * mx).sum(0), rtol=1e-5)
    assert np.all(m <= M)


@pytest.mark.parametrize("which", ["c", "np"])
def test_gamma_extremes_and_batching(corc, norc, which):
    orc = corc if which == "c" else norc
    y = _data(3, 6, 8, 12)
    v = bf16_value(y.reshape(-1, 12)).reshape(6, 8, 12)
    m1, M1, _ = orc.calibrate(None, None, 0, y, 1.0)          # gamma = 1: last sequence
    assert np.array_equal(m1.astype(np.float64), v[-1].min(0))
    assert np.array_equal(M1.astype(np.float64), v[-1].max(0))
    m0, M0, _ = orc.calibrate(None, None, 0, y, 0.0)          # gamma = 0: first sequence
    assert np.array_equal(m0.astype(np.float64), v[0].min(0))
    assert np.array_equal(M0.astype(np.float64), v[0].max(0))
    # one call with 6 sequences == 6 calls with one
    ma, Ma, ca = orc.calibrate(None, None, 0, y, 0.01)
    mb, Mb, cb = None, None, 0
    for q in range(6):
        mb, Mb, cb = orc.calibrate(mb, Mb, cb, y[q:q + 1], 0.01)
    assert ca == cb == 6
    assert np.array_equal(ma.view(np.uint32), mb.view(np.uint32))
    assert np.array_equal(Ma.view(np.uint32), Mb.view(np.uint32))


@pytest.mark.parametrize("which", ["c", "np"])
def test_constant_input_is_a_fixed_point(corc, norc, which):
    orc = corc if which == "c" else norc
    y = np.broadcast_to(bf16_bits([3.0, -123.5, 0.7])[None, None, :], (50, 4, 3)).copy()
    m, M, _ = orc.calibrate(None, None, 0, y, 0.01)
    c = bf16_value(bf16_bits([3.0, -123.5, 0.7]))
    np.testing.assert_allclose(m, c, rtol=2e-6)
    np.testing.assert_allclose(M, c, rtol=2e-6)


@pytest.mark.parametrize("which", ["c", "np"])
def test_signed_zero_min_max_order_independent(corc, norc, which):
    """-0 < +0 so that the result does not depend on row order."""
    orc = corc if which == "c" else norc
    a = np.array([[[0x0000], [0x8000]]], np.uint16)
    b = a[:, ::-1].copy()
    for y in (a, b):
        m, M, _ = orc.calibrate(None, None, 0, y, 0.01)
        assert m.view(np.uint32)[0] == 0x80000000 and M.view(np.uint32)[0] == 0


def test_ranges_formula(corc, norc):
    m = np.array([[-1.0, 2.0, -5.0, -0.5], [-3.0, 0.25, -1.0, -0.5]], np.float32)
    M = np.array([[4.0, 3.0, 1.0, 0.5], [2.0, 0.5, 7.0, 0.5]], np.float32)
    for orc in (corc, norc):
        R, Rbar = orc.ranges(m, M)
        assert R.tolist() == [[8.0, 6.0, 10.0, 1.0], [6.0, 1.0, 14.0, 1.0]]
        assert Rbar.tolist() == [14.0, 7.0, 24.0, 2.0]


def test_rbar_sum_is_ascending_float32(corc, norc):
    """The aggregate is the float32 chain over devices in ascending order (not float64, not pairwise)."""
    R_half = np.array([[2.0 ** 24], [1.0], [1.0], [1.0]], np.float32) / 2   # R = 2 * max(-m, M)
    m = -R_half
    M = R_half
    for orc in (corc, norc):
        R, Rbar = orc.ranges(m, M)
        assert R[:, 0].tolist() == [2.0 ** 24, 1.0, 1.0, 1.0]
        assert Rbar[0] == np.float32(2.0 ** 24)          # each +1 is absorbed in ascending order
