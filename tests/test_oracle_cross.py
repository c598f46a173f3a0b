"""The two independently written CPU statements (scalar C, NumPy) agree bit for
bit on the whole path, including odd shapes, clustered and empty index sets."""
import numpy as np
import pytest

from paper_2411_07942_b200 import synth


def _run(orc, w, ys, cal, k, is_c):
    ms, Ms = [], []
    for i in range(w.n_shards):
        m, M, _ = orc.calibrate(None, None, 0, cal[i], 0.01)
        ms.append(m)
        Ms.append(M)
    m, M = np.stack(ms), np.stack(Ms)
    R, Rbar = orc.ranges(m, M)
    hp = orc.select(Rbar, k)
    s, inv = orc.params(R)
    pl = [orc.quantize_pack(ys[i], hp, inv[i]) for i in range(w.n_shards)]
    T, E = ys[0].shape
    ref = orc.dequant_reduce(pl, T, E, hp, s)
    ref = ref[0] if is_c else ref
    return m, M, R, Rbar, hp, s, inv, pl, ref


@pytest.mark.parametrize("name,T,E,k", [("tiny", 16, 256, 4), ("tiny", 3, 65, 1), ("tiny", 17, 130, 0),
                                        ("tiny", 5, 253, 9), ("tiny", 1, 64, 64)])
def test_c_and_numpy_agree(corc, norc, name, T, E, k):
    base = synth.WORKLOADS[name]
    w = synth.Workload(base.name, base.n_shards, T, E, base.sd, 2, 50.0, 50.0, 3, 8, 7 + E)
    ys = [synth.activations_np(w, i, T) for i in range(w.n_shards)]
    cal = [synth.calibration_np(w, i) for i in range(w.n_shards)]
    a = _run(corc, w, ys, cal, k, True)
    b = _run(norc, w, ys, cal, k, False)
    for x, y in zip(a[:7], b[:7]):
        x, y = np.asarray(x), np.asarray(y)
        assert x.shape == y.shape
        assert np.array_equal(x.view(np.uint32) if x.dtype == np.float32 else x,
                              y.view(np.uint32) if y.dtype == np.float32 else y)
    for pa, pb in zip(a[7], b[7]):
        assert np.array_equal(pa, pb)
    np.testing.assert_allclose(a[8], b[8], rtol=1e-15, atol=0)
