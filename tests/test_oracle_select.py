"""Pins of the oracle's feature selection (paper Section 3: top-k features by
aggregated range R-bar, one set for all devices; Section 4: k = floor(E/64))."""
import numpy as np
import pytest


def _brute(Rbar, k):
    """Definition by counting: feature j is selected iff fewer than k features beat it."""
    E = len(Rbar)
    sel = []
    for j in range(E):
        beats = sum(1 for a in range(E) if Rbar[a] > Rbar[j] or (Rbar[a] == Rbar[j] and a < j))
        if beats < k:
            sel.append(j)
    return sel


@pytest.mark.parametrize("E,k", [(8, 0), (8, 3), (64, 1), (100, 7), (256, 4), (33, 33)])
def test_topk_bruteforce(corc, norc, E, k):
    rng = np.random.default_rng(E + k)
    Rbar = rng.lognormal(0, 1, E).astype(np.float32)
    want = _brute(Rbar, k)
    for orc in (corc, norc):
        got = orc.select(Rbar, k)
        assert got.tolist() == want
        assert got.tolist() == sorted(got.tolist())
    if k:
        assert set(want) == set(np.argsort(-Rbar, kind="stable")[:k].tolist())     # library sort


def test_ties_lower_index_wins(corc, norc):
    Rbar = np.array([1, 5, 5, 5, 0, 5, 2, 0], np.float32)
    for orc in (corc, norc):
        assert orc.select(Rbar, 2).tolist() == [1, 2]
        assert orc.select(Rbar, 3).tolist() == [1, 2, 3]
        assert orc.select(Rbar, 5).tolist() == [1, 2, 3, 5, 6]
        assert orc.select(np.zeros(6, np.float32), 2).tolist() == [0, 1]


def test_permuting_features_permutes_the_set(corc):
    rng = np.random.default_rng(9)
    Rbar = rng.lognormal(0, 1, 128).astype(np.float32)
    perm = rng.permutation(128)
    a = set(corc.select(Rbar, 6).tolist())
    b = set(corc.select(Rbar[perm], 6).tolist())
    assert {int(perm[j]) for j in b} == a


def test_planted_outliers_recovered_on_tiny_config(corc):
    """Config 'tiny': the four x50 columns have the largest aggregated ranges."""
    from paper_2411_07942_b200 import synth

    w = synth.WORKLOADS["tiny"]
    ms, Ms = [], []
    for i in range(w.n_shards):
        m, M, _ = corc.calibrate(None, None, 0, synth.calibration_np(w, i), 0.01)
        ms.append(m)
        Ms.append(M)
    R, Rbar = corc.ranges(np.stack(ms), np.stack(Ms))
    got = corc.select(Rbar, corc.default_k(w.features))
    assert got.tolist() == _brute(Rbar, 4)
    planted = sorted(w.fixed_outliers)
    margin = np.sort(Rbar[planted])[0] / np.sort(np.delete(Rbar, planted))[-1]
    if margin > 1.5:
        assert got.tolist() == planted
