"""Pins of the oracle's payload (paper Section 4 bit count; Figure 2: selected
features stay BF16): hand-derived bytes, the bits/value accounting, round trip,
exact pass-through of the selected features, and the k = 0 / k = E special cases."""
import numpy as np
import pytest

from util import bf16_bits, finite_bf16_patterns, read_golden


def _slot_order_by_definition(E, hp):
    """The payload's slot order, spelled out independently of the oracle: slot c holds feature c unless
    c is selected; selected features below L are filled in order with unselected ones from L upwards."""
    L = E - len(hp)
    sel = set(hp)
    spare = [j for j in range(L, E) if j not in sel]
    out = []
    for c in range(L):
        out.append(c if c not in sel else spare.pop(0))
    assert not spare
    return out


@pytest.mark.parametrize("E,hp", [(8, [1, 6]), (8, []), (8, [6, 7]), (8, [0, 1]), (16, [0, 3, 9, 15]),
                                  (16, list(range(8))), (16, list(range(8, 16))), (12, [11]), (5, [0, 1, 2, 3, 4])])
def test_slot_order_definition(corc, norc, E, hp):
    want = _slot_order_by_definition(E, hp)
    assert corc.lp_index(E, hp).tolist() == want
    assert norc.lp_index(E, np.array(hp, np.int64)).tolist() == want
    # a permutation of the unselected features; most features keep their own index as slot
    assert sorted(want) == [j for j in range(E) if j not in hp]
    assert all(want[c] == c for c in range(len(want)) if c not in hp)


def _orcs(corc, norc):
    return [("c", corc), ("np", norc)]


def test_pack_small_golden(corc, norc):
    rows = read_golden("pack_small.txt")
    x = np.array([[int(h, 16) for h in r[1:]] for r in rows if r[0] == "x"], np.uint16)
    want = np.array([int(h, 16) for r in rows if r[0] == "p" for h in r[1:]], np.uint8)
    hp = np.array([1, 6], np.int32)
    s, inv = corc.params(np.full(8, 15.0, np.float32))
    assert np.all(s == 1.0)
    for _, orc in _orcs(corc, norc):
        got = orc.quantize_pack(x, hp, inv)
        assert got.tolist() == want.tolist()
        assert orc.payload_bytes(2, 8, 2) == 24


def test_bits_per_value_golden(corc, norc):
    """bits/value = 4 + 12k/E with k = floor(E/64): below 4.2 as the paper states."""
    for name, E, k, bits, bound in read_golden("bits_per_value.txt"):
        E, k, bits, bound = int(E), int(k), float(bits), float(bound)
        assert corc.default_k(E) == k == norc.default_k(E)
        for T in (64, 2048):        # T(E-k)/2 a multiple of 16: no padding
            for _, orc in _orcs(corc, norc):
                got = 8.0 * orc.payload_bytes(T, E, k) / (T * E)
                assert got == pytest.approx(bits, abs=1e-12)
                assert got < bound
                assert got == pytest.approx(4 + 12 * k / E, abs=1e-12)


@pytest.mark.parametrize("T,E,k", [(1, 8, 0), (3, 65, 1), (17, 130, 2), (5, 33, 33), (16, 256, 4), (7, 253, 0)])
def test_payload_size_closed_form(corc, norc, T, E, k):
    nib = T * (E - k)
    lp = -(-((nib + 1) // 2) // 16) * 16
    for _, orc in _orcs(corc, norc):
        assert orc.payload_bytes(T, E, k) == lp + 2 * T * k
    # padding never costs more than 128 bits per call
    assert 8 * corc.payload_bytes(T, E, k) - (4 * nib + 16 * T * k) < 128 + 4


@pytest.mark.parametrize("T,E,k", [(1, 8, 0), (3, 65, 1), (17, 130, 2), (16, 256, 4), (7, 253, 9), (2, 31, 30)])
def test_roundtrip_and_padding(corc, norc, T, E, k):
    rng = np.random.default_rng(T * 1000 + E)
    y = bf16_bits(rng.standard_normal((T, E)) * 4)
    hp = np.sort(rng.permutation(E)[:k]).astype(np.int32)
    inv = (1.0 / rng.uniform(0.2, 2.0, E)).astype(np.float32)
    lp_cols = _slot_order_by_definition(E, hp.tolist())
    for _, orc in _orcs(corc, norc):
        p = orc.quantize_pack(y, hp, inv)
        codes, hpv = norc.unpack(p, T, E, k)
        want = np.array([[corc.quantize_one(int(y[t, j]), float(inv[j])) for j in lp_cols] for t in range(T)])
        assert np.array_equal(codes, want.reshape(T, E - k))
        assert np.array_equal(hpv, y[:, hp])
        nb = corc.lp_bytes(T, E, k)
        used = (T * (E - k) + 1) // 2
        assert not p[used:nb].any(), "padding must be zero"
        if (T * (E - k)) % 2:
            assert p[used - 1] >> 4 == 0, "unused high nibble must be zero"


def test_selected_features_pass_every_pattern(corc, norc):
    """k = E: every BF16 pattern (NaN payloads, signed zeros, subnormals) is
    transported unchanged and the payload is the input itself: 16 bits/value."""
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16).reshape(256, 256)
    hp = np.arange(256, dtype=np.int32)
    inv = np.ones(256, np.float32)
    for _, orc in _orcs(corc, norc):
        p = orc.quantize_pack(pats, hp, inv)
        assert p.size == 2 * 65536
        assert np.array_equal(p.view(np.uint16).reshape(256, 256), pats)


def test_k0_is_plain_int4(corc, norc):
    """k = 0 is the paper's "Int4" baseline: exactly 4 bits per value."""
    rng = np.random.default_rng(3)
    y = bf16_bits(rng.standard_normal((32, 64)))
    inv = np.full(64, 2.0, np.float32)
    for _, orc in _orcs(corc, norc):
        p = orc.quantize_pack(y, np.zeros(0, np.int32), inv)
        assert p.size * 8 == 4 * 32 * 64
