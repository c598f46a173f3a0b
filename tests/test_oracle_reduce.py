"""Pins of the oracle's dequantise-and-sum (paper Figure 2 caption and Section 5:
all-gather followed by a local reduction) and of the Irwin-Hall shape of the
aggregated quantisation error (paper Section 1)."""
import math

import numpy as np
import pytest
import torch

from util import bf16_bits, bf16_value


def _setup(seed, N, T, E, k, scale=2.0):
    rng = np.random.default_rng(seed)
    ys = [bf16_bits(rng.standard_normal((T, E)) * scale) for _ in range(N)]
    hp = np.sort(rng.permutation(E)[:k]).astype(np.int32)
    s = rng.uniform(0.2, 0.9, (N, E)).astype(np.float32)
    inv = (np.float32(1.0) / s).astype(np.float32)
    return ys, hp, s, inv


@pytest.mark.parametrize("which", ["c", "np"])
def test_all_selected_is_a_plain_sum_reduce(corc, norc, which):
    """k = E: the synchronisation is the textbook all-reduce-sum of the BF16 inputs."""
    N, T, E = 5, 9, 24
    ys, _, s, inv = _setup(1, N, T, E, 0)
    hp = np.arange(E, dtype=np.int32)
    pl = [corc.quantize_pack(y, hp, inv[i]) for i, y in enumerate(ys)]
    want = torch.stack([torch.from_numpy(bf16_value(y)) for y in ys]).sum(0).numpy()   # float64 library sum
    if which == "c":
        ref, chain = corc.dequant_reduce(pl, T, E, hp, s)
        np.testing.assert_allclose(chain, want, rtol=1e-6, atol=1e-6)
    else:
        ref = norc.dequant_reduce(pl, T, E, hp, s)
    np.testing.assert_allclose(ref, want, rtol=1e-15, atol=1e-15)


@pytest.mark.parametrize("which", ["c", "np"])
def test_single_shard_is_code_times_step(corc, norc, which):
    T, E, k = 6, 40, 3
    ys, hp, s, inv = _setup(2, 1, T, E, k)
    p = corc.quantize_pack(ys[0], hp, inv[0])
    ref = corc.dequant_reduce([p], T, E, hp, s)[0] if which == "c" else norc.dequant_reduce([p], T, E, hp, s)
    for t in range(T):
        for j in range(E):
            if j in hp:
                assert ref[t, j] == bf16_value(ys[0][t, j:j + 1])[0]
            else:
                q = corc.quantize_one(int(ys[0][t, j]), float(inv[0, j]))
                assert ref[t, j] == q * float(s[0, j])


def test_equal_steps_give_integer_sum(corc, norc):
    N, T, E = 7, 5, 16
    ys, _, _, _ = _setup(3, N, T, E, 0)
    s = np.full((N, E), 0.375, np.float32)
    inv = (np.float32(1) / s).astype(np.float32)
    hp = np.zeros(0, np.int32)
    pl = [corc.quantize_pack(y, hp, inv[i]) for i, y in enumerate(ys)]
    qsum = sum(norc.unpack(p, T, E, 0)[0].astype(np.int64) for p in pl)
    ref, chain = corc.dequant_reduce(pl, T, E, hp, s)
    assert np.array_equal(ref, qsum * 0.375)
    assert np.array_equal(chain.astype(np.float64), qsum * 0.375)       # exact in float32 too
    assert np.array_equal(norc.dequant_reduce(pl, T, E, hp, s), qsum * 0.375)


def test_end_to_end_error_bound(corc):
    """|sum_i D(C(y_i)) - sum_i y_i| <= sum_i s_i / 2 for unclipped low-precision
    features and == 0 for the selected ones (Section 2: f ~ D(C(f)))."""
    N, T, E, k = 4, 32, 64, 5
    ys, hp, s, inv = _setup(4, N, T, E, k, scale=1.0)
    pl = [corc.quantize_pack(y, hp, inv[i]) for i, y in enumerate(ys)]
    ref, _ = corc.dequant_reduce(pl, T, E, hp, s)
    exact = sum(bf16_value(y) for y in ys)
    vals = np.stack([bf16_value(y) for y in ys])
    unclipped = np.all((vals >= -8.5 * s[:, None, :]) & (vals <= 7.5 * s[:, None, :]), axis=0)
    bound = 0.5 * s.sum(0)[None, :] * (1 + 1e-5)
    lp = np.ones(E, bool)
    lp[hp] = False
    err = np.abs(ref - exact)
    assert np.all(err[:, lp][unclipped[:, lp]] <= np.broadcast_to(bound, err.shape)[:, lp][unclipped[:, lp]])
    assert np.all(err[:, hp] == 0)
    assert unclipped.mean() > 0.5


def _irwin_hall_cdf(x, n):
    x = np.asarray(x, np.float64)
    out = np.zeros_like(x)
    for kk in range(n + 1):
        out += (-1) ** kk * math.comb(n, kk) * np.where(x >= kk, (x - kk) ** n, 0.0)
    return np.clip(out / math.factorial(n), 0, 1)


@pytest.mark.parametrize("N", [1, 2, 4, 8, 16])
def test_aggregated_error_is_irwin_hall(corc, norc, N):
    """The sum of N independent quantisation errors (in steps), shifted by N/2,
    follows Irwin-Hall(N): mean N/2, variance N/12, excess kurtosis -1.2/N, and
    its empirical CDF matches the closed form."""
    n = 400_000
    rng = np.random.default_rng(100 + N)
    s = np.float32(0.37)
    inv = np.float32(1.0) / s
    E = 1000
    T = n // E
    tot = np.zeros((T, E))
    exact = np.zeros((T, E))
    pl = []
    hp = np.zeros(0, np.int32)
    for i in range(N):
        y = bf16_bits(rng.uniform(-7 * float(s), 7 * float(s), (T, E)))
        exact += bf16_value(y)
        pl.append(corc.quantize_pack(y, hp, np.full(E, inv, np.float32)))
    ref, _ = corc.dequant_reduce(pl, T, E, hp, np.full((N, E), s, np.float32))
    e = ((exact - ref) / float(s) + N / 2).reshape(-1)
    assert abs(e.mean() - N / 2) < 4 * math.sqrt(N / 12 / e.size) + 2e-3
    assert abs(e.var() * 12 / N - 1) < 0.02
    kurt = ((e - e.mean()) ** 4).mean() / e.var() ** 2 - 3
    assert abs(kurt - (-1.2 / N)) < 0.05
    xs = np.sort(e)
    emp = (np.arange(xs.size) + 0.5) / xs.size
    ks = np.abs(emp - _irwin_hall_cdf(xs, N)).max()
    assert ks < 0.01, ks


def test_bias_is_added_after_the_sum(corc, norc):
    """Section 2: f(x) = sum_i f_i(x_i) + b.  The reference with a bias is the reference without it plus b,
    exactly (binary64); the chain adds b last; a zero bias changes no value; with every feature selected
    and one device the output is y + b computed by the library."""
    rng = np.random.default_rng(12)
    N, T, E = 3, 7, 48
    hp = np.array([1, 5, 20, 47], np.int32)
    y = [bf16_bits((rng.normal(0, 2, (T, E))).astype(np.float32)) for _ in range(N)]
    R = np.stack([2 * np.abs(bf16_value(v)).max(axis=0) for v in y]).astype(np.float32)
    s, inv = corc.params(R)
    pls = [corc.quantize_pack(y[i], hp, inv[i]) for i in range(N)]
    bias = rng.normal(0, 3, E).astype(np.float32)
    ref0, chain0 = corc.dequant_reduce(pls, T, E, hp, s)
    ref1, chain1 = corc.dequant_reduce(pls, T, E, hp, s, bias=bias)
    assert np.array_equal(ref1, ref0 + bias.astype(np.float64)[None, :])
    assert np.array_equal(chain1, (chain0 + bias[None, :]).astype(np.float32))
    assert np.array_equal(norc.dequant_reduce(pls, T, E, hp, s, 4, bias), ref1)
    refz, chainz = corc.dequant_reduce(pls, T, E, hp, s, bias=np.zeros(E, np.float32))
    assert np.array_equal(refz, ref0) and np.array_equal(chainz + 0.0, chain0 + 0.0)
    # every feature selected, one device: the payload is y itself
    allhp = np.arange(E, dtype=np.int32)
    p1 = corc.quantize_pack(y[0], allhp, inv[0])
    ref, chain = corc.dequant_reduce([p1], T, E, allhp, s[:1], bias=bias)
    assert np.array_equal(ref, bf16_value(y[0]) + bias.astype(np.float64)[None, :])
    assert np.array_equal(chain, (bf16_value(y[0]).astype(np.float32) + bias[None, :]).astype(np.float32))
