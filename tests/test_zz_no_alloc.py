"""The allocation-free calibration entry point (tpq_calibrate_ranges_noalloc).

Some callers of the library cannot allocate device memory while they run: a serving loop whose memory
belongs to a pool, a framework that forbids allocation after start-up, or code that cannot afford the
device-wide synchronisation hidden in cudaFree.  tpq_calibrate_ranges may grow its scratch buffer; the
variant tested here keeps that scratch in a fixed array inside the library instead.  The test drives it
through the C ABI and checks, on two calls in a row, that it leaves exactly the state the ordinary entry
point leaves and the state the CPU oracle computes from the same sequences (Eq. 1-2; bit for bit, the
tolerance every calibration test uses), that the array's stale contents
from the first call do not leak into the second, and that an oversized call is refused with a clear
error and launches nothing.  It is collected last so that a run that stops at the first failure has
already run everything else."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2411_07942_b200 import binding, synth  # noqa: E402

import oracle  # noqa: E402

import gpu_util as gu  # noqa: E402


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gu.ensure_lib()


def _cal(E, n_seq, S, seed):
    w = synth.Workload("na", 1, 1, E, 0.7, 4, 20.0, 200.0, n_seq, S, seed)
    return synth.calibration_np(w, 0)


def test_noalloc_matches_the_allocating_entry_point_twice_in_a_row():
    E = 1024
    first, second = _cal(E, 5, 300, 11), _cal(E, 3, 77, 12)      # different shapes: different scratch layouts
    ref = binding.Tpq(2, E)
    na = binding.Tpq(2, E)
    orc = oracle.c()
    state = {0: (None, None, 0), 1: (None, None, 0)}      # the oracle's (m, M, count) per shard
    for shard, cal in ((0, first), (0, second), (1, second)):
        d = gu.dev_bf16(cal)
        n_seq, S, _ = cal.shape
        ref.calibrate_ranges(shard, d.data_ptr(), n_seq, S)
        na.calibrate_ranges_noalloc(shard, d.data_ptr(), n_seq, S)
        torch.cuda.synchronize()
        a, b = ref.get_ranges(with_R=False), na.get_ranges(with_R=False)
        assert gu.bits_equal(a[0], b[0]) and gu.bits_equal(a[1], b[1])
        state[shard] = orc.calibrate(*state[shard], cal, 0.01)
        assert gu.bits_equal(b[0][shard], state[shard][0]) and gu.bits_equal(b[1][shard], state[shard][1])
    assert na.device_status() == 0
    # the two contexts now select the same features and steps
    assert ref.select_features(-1).tolist() == na.select_features(-1).tolist()
    assert all(gu.bits_equal(x, y) for x, y in zip(ref.get_scales(), na.get_scales()))
    ref.close()
    na.close()


def test_noalloc_strided_and_generic_shapes():
    for E, stride in ((520, 528), (1001, 1001)):
        cal = _cal(E, 2, 40, 20 + E)
        wide = np.full((2, 40, stride), 0x7FC0, np.uint16)
        wide[:, :, :E] = cal
        d = gu.dev_bf16(wide)
        ref, na = binding.Tpq(1, E), binding.Tpq(1, E)
        ref.calibrate_ranges(0, d.data_ptr(), 2, 40, row_stride=stride)
        na.calibrate_ranges_noalloc(0, d.data_ptr(), 2, 40, row_stride=stride)
        torch.cuda.synchronize()
        a, b = ref.get_ranges(with_R=False), na.get_ranges(with_R=False)
        assert gu.bits_equal(a[0], b[0]) and gu.bits_equal(a[1], b[1])
        ref.close()
        na.close()


def test_noalloc_near_its_limit_against_the_oracle():
    """100 sequences x 8192 features fill 78 % of the array; the result is the oracle's.  (The branch that
    lowers the row-split count to fit the array needs more than 512 SMs' worth of splits and is not
    reachable on this GPU: 8 x 148 x 256 partial extremes always fit.)"""
    E, n_seq, S = 8192, 100, 24
    cal = _cal(E, n_seq, S, 31)
    d = gu.dev_bf16(cal)
    na = binding.Tpq(1, E)
    na.calibrate_ranges_noalloc(0, d.data_ptr(), n_seq, S)
    torch.cuda.synchronize()
    m, M = na.get_ranges(with_R=False)
    om, oM, _ = oracle.c().calibrate(None, None, 0, cal, 0.01)
    assert gu.bits_equal(m[0], om) and gu.bits_equal(M[0], oM)
    assert na.device_status() == 0
    na.close()


def test_noalloc_rejects_what_does_not_fit():
    E = 8192
    t = binding.Tpq(1, E)
    y = torch.zeros((8, E), dtype=torch.bfloat16, device="cuda")
    n0 = t.launch_count()
    # 129 sequences x 8192 features > 1 048 576: refused before anything is launched
    st = t.raw("tpq_calibrate_ranges_noalloc", 0, y.data_ptr(), 129, 1, E, None)
    assert st == binding.TPQ_ERR_SIZE
    assert b"scratch" in binding.lib().tpq_last_error(t._h)
    assert t.launch_count() == n0
    # 128 sequences fit exactly
    y2 = torch.zeros((128, E), dtype=torch.bfloat16, device="cuda")
    t.calibrate_ranges_noalloc(0, y2.data_ptr(), 128, 1)
    torch.cuda.synchronize()
    assert t.launch_count() == n0 + 2
    t.close()
