"""Host-side failure injection through the C ABI: every bad call returns a status
code, launches nothing and leaves the context usable.  No GPU fault is provoked."""
import ctypes

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2411_07942_b200 import binding  # noqa: E402

import gpu_util as gu  # noqa: E402


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gu.ensure_lib()


def _ready_ctx(N=2, E=64, k=8):
    t = binding.Tpq(N, E)
    M = np.ones((N, E), np.float32)
    t.set_ranges(-M, M, np.ones(N, np.int64))
    t.set_features(list(range(k)))
    return t


def test_state_errors():
    t = binding.Tpq(2, 64)
    y = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    n0 = t.launch_count()
    assert t.raw("tpq_quantize_pack", 0, y.data_ptr(), 4, 64, buf.data_ptr(), 4096, None) == binding.TPQ_ERR_BAD_STATE
    assert t.raw("tpq_select_features", -1, None, None) == binding.TPQ_ERR_BAD_STATE      # nothing calibrated
    t.calibrate_ranges(0, y.data_ptr(), 1, 4)
    assert t.raw("tpq_select_features", -1, None, None) == binding.TPQ_ERR_BAD_STATE      # shard 1 missing
    assert t.payload_bytes(4) == 0 and t.num_selected() == -1
    assert t.raw("tpq_get_scales", None, None) == binding.TPQ_ERR_BAD_STATE
    assert t.launch_count() == n0 + 2          # only the calibration launched (extremes + fold)
    assert binding.lib().tpq_last_error(t._h) != b""
    t.close()


def test_argument_errors_launch_nothing():
    t = _ready_ctx()
    y = torch.zeros((4, 72), dtype=torch.bfloat16, device="cuda")
    P = t.payload_bytes(4)
    buf = torch.zeros(P + 64, dtype=torch.uint8, device="cuda")
    out = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    n0 = t.launch_count()
    E = binding
    q = lambda *a: t.raw("tpq_quantize_pack", *a)  # noqa: E731
    assert q(2, y.data_ptr(), 4, 64, buf.data_ptr(), P, None) == E.TPQ_ERR_INVALID_ARG          # shard
    assert q(-1, y.data_ptr(), 4, 64, buf.data_ptr(), P, None) == E.TPQ_ERR_INVALID_ARG
    assert q(0, y.data_ptr(), -1, 64, buf.data_ptr(), P, None) == E.TPQ_ERR_INVALID_ARG         # T < 0
    assert q(0, None, 4, 64, buf.data_ptr(), P, None) == E.TPQ_ERR_INVALID_ARG                  # NULL
    assert q(0, y.data_ptr(), 4, 56, buf.data_ptr(), P, None) == E.TPQ_ERR_INVALID_ARG          # stride < E
    assert q(0, y.data_ptr() + 2, 4, 64, buf.data_ptr(), P, None) == E.TPQ_ERR_ALIGN
    assert q(0, y.data_ptr(), 4, 64, buf.data_ptr() + 4, P, None) == E.TPQ_ERR_ALIGN
    assert q(0, y.data_ptr(), 4, 64, buf.data_ptr(), P - 1, None) == E.TPQ_ERR_SIZE
    assert q(0, y.data_ptr(), 0, 64, buf.data_ptr(), 0, None) == E.TPQ_OK                       # T = 0: no-op
    ptrs = (ctypes.c_void_p * 2)(buf.data_ptr(), buf.data_ptr())
    d = lambda *a: t.raw("tpq_dequant_reduce", *a)  # noqa: E731
    assert d(ptrs, 1, 4, out.data_ptr(), 1, 64, None) == E.TPQ_ERR_INVALID_ARG                  # n_payloads != N
    assert d(ptrs, 2, 4, out.data_ptr(), 7, 64, None) == E.TPQ_ERR_INVALID_ARG                  # dtype
    assert d(ptrs, 2, 4, out.data_ptr(), 1, 60, None) == E.TPQ_ERR_INVALID_ARG                  # stride < E
    assert d(ptrs, 2, 4, out.data_ptr() + 4, 1, 64, None) == E.TPQ_ERR_ALIGN
    bad = (ctypes.c_void_p * 2)(buf.data_ptr(), None)
    assert d(bad, 2, 4, out.data_ptr(), 1, 64, None) == E.TPQ_ERR_INVALID_ARG
    assert d(ptrs, 2, 0, out.data_ptr(), 1, 64, None) == E.TPQ_OK
    c = lambda *a: t.raw("tpq_calibrate_ranges", *a)  # noqa: E731
    assert c(5, y.data_ptr(), 1, 4, 64, None) == E.TPQ_ERR_INVALID_ARG
    assert c(0, y.data_ptr(), -1, 4, 64, None) == E.TPQ_ERR_INVALID_ARG
    assert c(0, y.data_ptr(), 1, 0, 64, None) == E.TPQ_ERR_INVALID_ARG
    assert c(0, y.data_ptr(), 1, 4, 8, None) == E.TPQ_ERR_INVALID_ARG
    assert c(0, y.data_ptr(), 0, 4, 64, None) == E.TPQ_OK
    assert t.raw("tpq_select_features", 65, None, None) == E.TPQ_ERR_INVALID_ARG
    idx = (ctypes.c_int32 * 3)(5, 5, 9)
    assert t.raw("tpq_set_features", idx, 3) == E.TPQ_ERR_INVALID_ARG                           # not ascending
    idx = (ctypes.c_int32 * 2)(5, 64)
    assert t.raw("tpq_set_features", idx, 2) == E.TPQ_ERR_INVALID_ARG                           # out of range
    assert t.raw("tpq_set_option", 9, 0) == E.TPQ_ERR_INVALID_ARG
    assert t.raw("tpq_set_state", b"garbage-garbage-garbage-garbage-garbage", 38) == E.TPQ_ERR_INVALID_ARG
    assert t.launch_count() == n0
    # forced tiled path on a shape that does not admit it
    t2 = binding.Tpq(1, 65)
    M = np.ones((1, 65), np.float32)
    t2.set_ranges(-M, M, np.ones(1, np.int64))
    t2.set_features([3])
    t2.set_option(binding.TPQ_OPT_KERNEL_PATH, binding.PATH_TILED)
    y2 = torch.zeros((2, 72), dtype=torch.bfloat16, device="cuda")
    assert t2.raw("tpq_quantize_pack", 0, y2.data_ptr(), 2, 72, buf.data_ptr(), P, None) == E.TPQ_ERR_INVALID_ARG
    t2.close()
    # the context still works after all of that
    t.quantize_pack(0, y.data_ptr(), 4, buf.data_ptr(), P, row_stride=72)
    torch.cuda.synchronize()
    assert t.device_status() == 0
    t.close()


def test_comm_report_matches_formulas():
    t = _ready_ctx(N=8, E=4608, k=72)
    r = t.comm_bytes(64)
    assert r.payload_bytes == 154368
    assert r.quantized_allgather_send == 7 * 154368
    assert r.bf16_allgather_send == 7 * 2 * 64 * 4608
    assert r.bf16_ring_allreduce_send == 2 * 7 * 2 * 64 * 4608 // 8
    assert r.bits_per_value == pytest.approx(4.1875) and r.bits_per_value_formula == pytest.approx(4.1875)
    t.close()
