"""Pins of the oracle's Int4 quantiser (paper Section 3: symmetric Int4 from the
calibrated range) against definitions that are not the oracle's own code:
nearest-level brute force in exact arithmetic, literal tie values, saturation,
the half-step error bound and scale invariance."""
import numpy as np
import pytest

from util import bf16_bits, bf16_value, finite_bf16_patterns, read_golden

SCALES = [1.0, 0.37, 3.0e-3, 17.25, 2.0 ** -10, 1.0 / 3.0, 123.456]


def _codes_all_patterns(orc, inv_s, which):
    pats = finite_bf16_patterns()
    n = pats.size
    E = 256
    T = (n + E - 1) // E
    y = np.zeros(T * E, np.uint16)
    y[:n] = pats
    y = y.reshape(T, E)
    inv = np.full(E, inv_s, np.float32)
    hp = np.zeros(0, np.int32)
    payload = orc.quantize_pack(y, hp, inv)
    from oracle import oracle_np
    codes, _ = oracle_np.unpack(payload, T, E, 0)
    return pats, codes.reshape(-1)[:n].astype(np.int64)


@pytest.mark.parametrize("s", SCALES)
@pytest.mark.parametrize("which", ["c", "np"])
def test_nearest_level_bruteforce_all_bf16(corc, norc, s, which):
    """Every finite BF16 input lands on a level that is nearest in exact
    arithmetic (up to the rounding slack of the two float32 operations), and
    exact ties go to the even code."""
    orc = corc if which == "c" else norc
    s32 = np.float32(s)
    inv_s = np.float32(1.0) / s32
    pats, q = _codes_all_patterns(orc, inv_s, which)
    x = bf16_value(pats)                                   # float64, exact
    finite = np.isfinite(x)
    levels = np.arange(-8, 8, dtype=np.float64) * np.float64(s32)      # exact products
    d = np.abs(x[:, None] - levels[None, :])
    d[~finite] = 0
    best = d.min(axis=1)
    with np.errstate(invalid="ignore"):
        got = np.abs(x - q * np.float64(s32))
    slack = 2.0 ** -20 * np.float64(s32)        # rounding of 1/s and of the product, in units of s
    assert np.all(got[finite] <= best[finite] + slack), "a code is not the nearest level"
    assert q.min() >= -8 and q.max() <= 7
    # infinities saturate
    assert q[np.isposinf(x)].tolist() == [7]
    assert q[np.isneginf(x)].tolist() == [-8]
    # inside the representable span the error never exceeds half a step (+ slack)
    inside = finite & (x >= -8.5 * np.float64(s32)) & (x <= 7.5 * np.float64(s32))
    assert np.all(got[inside] <= np.float64(s32) * (0.5 + 2.0 ** -20))
    # exact ties (only possible when x/s is exact: s a power of two) go to the even code
    if float(np.log2(s32)).is_integer():
        r = x / np.float64(s32)
        with np.errstate(invalid="ignore"):
            tie = finite & (np.abs(r) < 7.4) & (np.abs(r - np.floor(r) - 0.5) == 0)
        assert tie.sum() == 14          # +-0.5 .. +-6.5
        assert np.all(q[tie] % 2 == 0)
        assert np.all(np.abs(q[tie] - r[tie]) == 0.5)
    # beyond it the code saturates
    assert np.all(q[finite & (x > 7.5 * np.float64(s32) * (1 + 1e-6))] == 7)
    assert np.all(q[finite & (x < -8.5 * np.float64(s32) * (1 + 1e-6))] == -8)


@pytest.mark.parametrize("which", ["c", "np"])
def test_ties_to_even_golden(corc, norc, which):
    rows = read_golden("int4_ties.txt")
    vals = np.array([float(r[0]) for r in rows], np.float32)
    want = np.array([int(r[1]) for r in rows])
    bits = bf16_bits(vals)
    assert np.array_equal(bf16_value(bits), vals.astype(np.float64)), "fixture values must be exact BF16"
    if which == "c":
        got = np.array([corc.quantize_one(int(b), 1.0) for b in bits])
    else:
        got = norc.quantize_codes(bits[None, :], np.ones(len(bits), np.float32))[0].astype(int)
    assert got.tolist() == want.tolist()


def test_monotone_in_x(corc):
    """The code is a non-decreasing function of the input (clamp and rounding are monotone)."""
    pats = finite_bf16_patterns()
    x = bf16_value(pats)
    order = np.argsort(x, kind="stable")
    for s in (0.37, 5.5):
        inv_s = np.float32(1.0) / np.float32(s)
        _, q = _codes_all_patterns(corc, inv_s, "c")
        assert np.all(np.diff(q[order]) >= 0)


def test_scale_invariance(corc):
    """Scaling inputs and step by the same power of two changes no code."""
    rng = np.random.default_rng(5)
    x = bf16_bits(rng.standard_normal(4096) * 3.0)
    s = np.float32(0.61)
    base = np.array([corc.quantize_one(int(b), float(np.float32(1.0) / s)) for b in x])
    for a in (-6, 3, 11):
        xs = bf16_bits(bf16_value(x) * 2.0 ** a)
        sa = np.float32(s * np.float32(2.0 ** a))
        got = np.array([corc.quantize_one(int(b), float(np.float32(1.0) / sa)) for b in xs])
        assert np.array_equal(got, base)


def test_two_roundings_not_fused(corc, norc):
    """The product x * inv_s is rounded to float32 BEFORE the integer rounding.
    Searched pairs where a fused multiply-round would give another code: the
    float32 product sits exactly on a half-integer although the exact product
    does not."""
    found = 0
    rng = np.random.default_rng(11)
    pats = finite_bf16_patterns()
    xs = pats[(bf16_value(pats) > 0.9) & (bf16_value(pats) < 1.2)]
    for _ in range(200000):
        if found >= 20:
            break
        xb = int(xs[rng.integers(len(xs))])
        x = float(bf16_value(np.array([xb], np.uint16))[0])
        half = rng.integers(0, 7) + 0.5
        inv_s = np.float32(half / x)
        for d in (-1, 0, 1):
            cand = np.nextafter(inv_s, np.float32(np.inf if d > 0 else -np.inf)) if d else inv_s
            exact = np.float64(x) * np.float64(cand)          # exact: 8-bit x 24-bit significands
            u32 = np.float32(exact)                           # one rounding to float32
            if float(u32) == half and exact != half:
                # float32 product is a tie -> even neighbour; exact product is not a tie
                want = int(half - 0.5) if int(half - 0.5) % 2 == 0 else int(half + 0.5)
                fused = int(half + 0.5) if exact > half else int(half - 0.5)
                if want != fused:
                    assert corc.quantize_one(xb, float(cand)) == want
                    got_np = int(norc.quantize_codes(np.array([[xb]], np.uint16), np.array([cand], np.float32))[0, 0])
                    assert got_np == want
                    found += 1
    assert found >= 5, "search found too few discriminating pairs"
    # the literal example: x = 1.0078125, inv_s = 0.4961240589618683 -> product rounds to 0.5 -> code 0
    xb = int(bf16_bits(np.array([1.0078125]))[0])
    assert corc.quantize_one(xb, float(np.float32(0.4961240589618683))) == 0


def test_params_grid(corc, norc):
    """Step = range / 15 so that the range [-R/2, R/2] spans codes -7.5 .. 7.5;
    a zero range is floored and gives finite parameters and zero codes."""
    R = np.array([15.0, 30.0, 0.0, 1e-30, 7.5], np.float32)
    for orc in (corc, norc):
        s, inv = orc.params(R)
        assert s[0] == 1.0 and inv[0] == 1.0
        assert s[1] == 2.0 and inv[1] == 0.5
        assert s[2] == np.float32(2.0 ** -23) and inv[2] == np.float32(2.0 ** 23)
        assert s[3] == np.float32(2.0 ** -23)
        assert s[4] == 0.5 and inv[4] == 2.0
        assert np.all(np.isfinite(inv))
    # the edge of the calibrated range maps to the outermost codes
    s, inv = corc.params(np.array([2.0 * 3.3], np.float32))
    assert corc.quantize_one(int(bf16_bits([3.3])[0]), float(inv[0])) == 7
    assert corc.quantize_one(int(bf16_bits([-3.3])[0]), float(inv[0])) in (-8, -7)
    assert corc.quantize_one(0, float(np.float32(2.0 ** 23))) == 0
