"""ctypes front end of libtpq.so: the same names as include/tpq.h, argument
marshalling only.  Every step of the method runs in the library's CUDA kernels.

torch is used by callers for device memory and streams; this module only needs
``tensor.data_ptr()`` values and raw stream handles.  There is no CPU fallback:
if the library cannot be loaded the import of :func:`lib` raises.
"""
from __future__ import annotations

import ctypes
from ctypes import POINTER, byref, c_char_p, c_double, c_float, c_int, c_int32, c_int64, c_size_t, c_void_p
from pathlib import Path

import numpy as np

TPQ_OK = 0
TPQ_ERR_INVALID_ARG, TPQ_ERR_BAD_STATE, TPQ_ERR_SIZE, TPQ_ERR_ALIGN = 1, 2, 3, 4
TPQ_ERR_CUDA, TPQ_ERR_NOMEM, TPQ_ERR_TIMEOUT = 5, 6, 7
TPQ_OUT_BF16, TPQ_OUT_FP32 = 0, 1
TPQ_OPT_KERNEL_PATH = 0
TPQ_OPT_DEQUANT_KERNEL = 1
DQ_AUTO, DQ_ROWS, DQ_TENSOR_PANELS, DQ_COPY_PANELS = 0, 1, 2, 3
PATH_AUTO, PATH_GENERIC, PATH_TILED = 0, 1, 2

_LIB_PATH = Path(__file__).resolve().parent / "libtpq.so"


class CommReport(ctypes.Structure):
    _fields_ = [("payload_bytes", c_int64), ("quantized_allgather_send", c_int64),
                ("bf16_allgather_send", c_int64), ("bf16_ring_allreduce_send", c_int64),
                ("bits_per_value", c_double), ("bits_per_value_formula", c_double)]


# name -> (restype, argtypes); one entry per declaration in include/tpq.h
SIGNATURES = {
    "tpq_create": (c_int, [POINTER(c_void_p), c_int, c_int, c_int, c_float]),
    "tpq_destroy": (c_int, [c_void_p]),
    "tpq_set_option": (c_int, [c_void_p, c_int, c_int]),
    "tpq_calibrate_ranges": (c_int, [c_void_p, c_int, c_void_p, c_int64, c_int64, c_int64, c_void_p]),
    "tpq_calibrate_ranges_noalloc": (c_int, [c_void_p, c_int, c_void_p, c_int64, c_int64, c_int64, c_void_p]),
    "tpq_select_features": (c_int, [c_void_p, c_int, POINTER(c_int32), POINTER(c_int)]),
    "tpq_set_features": (c_int, [c_void_p, POINTER(c_int32), c_int]),
    "tpq_set_ranges": (c_int, [c_void_p, POINTER(c_float), POINTER(c_float), POINTER(c_int64)]),
    "tpq_get_ranges": (c_int, [c_void_p, POINTER(c_float), POINTER(c_float), POINTER(c_float), POINTER(c_float)]),
    "tpq_get_scales": (c_int, [c_void_p, POINTER(c_float), POINTER(c_float)]),
    "tpq_num_selected": (c_int, [c_void_p]),
    "tpq_get_features": (c_int, [c_void_p, POINTER(c_int32)]),
    "tpq_get_slot_order": (c_int, [c_void_p, POINTER(c_int32)]),
    "tpq_payload_bytes": (c_size_t, [c_void_p, c_int64]),
    "tpq_payload_bytes_for": (c_size_t, [c_int64, c_int64, c_int64]),
    "tpq_payload_bytes_for_bits": (c_size_t, [c_int64, c_int64, c_int64, c_int]),
    "tpq_comm_bytes": (c_int, [c_void_p, c_int64, POINTER(CommReport)]),
    "tpq_quantize_pack": (c_int, [c_void_p, c_int, c_void_p, c_int64, c_int64, c_void_p, c_size_t, c_void_p]),
    "tpq_quantize_pack_batch": (c_int, [c_void_p, c_int, c_int, POINTER(c_void_p), c_int64, c_int64, POINTER(c_void_p),
                                        c_size_t, c_void_p]),
    "tpq_dequant_reduce": (c_int, [c_void_p, POINTER(c_void_p), c_int, c_int64, c_void_p, c_int, c_int64, c_void_p]),
    "tpq_dequant_reduce_bias": (c_int, [c_void_p, POINTER(c_void_p), c_int, c_int64, c_void_p, c_int, c_int64, c_void_p,
                                        c_void_p]),
    "tpq_permute_weight": (c_int, [c_void_p, c_void_p, c_int64, c_void_p, c_void_p]),
    "tpq_linear_quantize_pack": (c_int, [c_void_p, c_int, c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_size_t, c_void_p,
                                         c_void_p]),
    "tpq_quantize_pack_push": (c_int, [c_void_p, c_int, c_void_p, c_int64, c_int64, POINTER(c_void_p), POINTER(c_void_p),
                                       c_int, c_size_t, ctypes.c_uint32, c_void_p]),
    "tpq_dequant_reduce_arrivals": (c_int, [c_void_p, POINTER(c_void_p), c_int, c_int64, c_void_p, c_int, c_int64, c_void_p,
                                            c_void_p, ctypes.c_uint32, ctypes.c_uint64, c_void_p]),
    "tpq_wait_arrivals": (c_int, [c_void_p, c_void_p, c_int, ctypes.c_uint32, ctypes.c_uint64, c_void_p]),
    "tpq_get_state": (c_int, [c_void_p, c_void_p, POINTER(c_size_t)]),
    "tpq_set_state": (c_int, [c_void_p, c_void_p, c_size_t]),
    "tpq_device_status": (c_int, [c_void_p]),
    "tpq_launch_count": (c_int64, [c_void_p]),
    "tpq_status_string": (c_char_p, [c_int]),
    "tpq_last_error": (c_char_p, [c_void_p]),
    "tpq_version": (c_char_p, []),
}

_lib = None


def lib() -> ctypes.CDLL:
    """Load libtpq.so (built in-tree by ``paper_2411_07942_b200.build``); raises if absent."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2411_07942_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(str(_LIB_PATH))
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


class TpqError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"tpq status {status} ({lib().tpq_status_string(status).decode()}): {message}")
        self.status = status


def _fp(a: np.ndarray):
    return a.ctypes.data_as(POINTER(c_float))


class Tpq:
    """One context (N shards, E features).  Methods mirror the C entry points one to one."""

    def __init__(self, n_shards: int, n_features: int, bits: int = 4, gamma: float = 0.01):
        self._h = c_void_p()
        st = lib().tpq_create(byref(self._h), n_shards, n_features, bits, gamma)
        if st != TPQ_OK:
            self._h = c_void_p()
            raise TpqError(st, "tpq_create failed")
        self.N, self.E, self.bits = n_shards, n_features, bits

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            lib().tpq_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != TPQ_OK:
            raise TpqError(st, lib().tpq_last_error(self._h).decode())

    # raw status-returning calls (for error-path tests)
    def raw(self, name: str, *args) -> int:
        return getattr(lib(), name)(self._h, *args)

    def set_option(self, opt: int, value: int):
        self._check(lib().tpq_set_option(self._h, opt, value))

    def calibrate_ranges(self, shard: int, y_ptr: int, n_seq: int, S: int, row_stride: int | None = None,
                         stream: int = 0):
        self._check(lib().tpq_calibrate_ranges(self._h, shard, y_ptr, n_seq, S,
                                               self.E if row_stride is None else row_stride, stream))

    def calibrate_ranges_noalloc(self, shard: int, y_ptr: int, n_seq: int, S: int, row_stride: int | None = None,
                                 stream: int = 0):
        """tpq_calibrate_ranges for callers that must not allocate: the scratch is a fixed 4 MiB array
        inside the library (n_seq * E <= 1 048 576 per call); see include/tpq.h."""
        self._check(lib().tpq_calibrate_ranges_noalloc(self._h, shard, y_ptr, n_seq, S,
                                                       self.E if row_stride is None else row_stride, stream))

    def select_features(self, k: int = -1) -> np.ndarray:
        out = np.zeros(self.E, np.int32)
        kk = c_int(0)
        self._check(lib().tpq_select_features(self._h, k, out.ctypes.data_as(POINTER(c_int32)), byref(kk)))
        return out[: kk.value].copy()

    def set_features(self, hp_idx):
        hp = np.ascontiguousarray(hp_idx, dtype=np.int32)
        self._check(lib().tpq_set_features(self._h, hp.ctypes.data_as(POINTER(c_int32)), hp.size))

    def set_ranges(self, m: np.ndarray, M: np.ndarray, counts):
        m = np.ascontiguousarray(m, dtype=np.float32)
        M = np.ascontiguousarray(M, dtype=np.float32)
        cnt = np.ascontiguousarray(counts, dtype=np.int64)
        assert m.shape == (self.N, self.E) and M.shape == (self.N, self.E) and cnt.shape == (self.N,)
        self._check(lib().tpq_set_ranges(self._h, _fp(m), _fp(M), cnt.ctypes.data_as(POINTER(c_int64))))

    def get_ranges(self, with_R: bool = True):
        m = np.empty((self.N, self.E), np.float32)
        M = np.empty((self.N, self.E), np.float32)
        if not with_R:
            self._check(lib().tpq_get_ranges(self._h, _fp(m), _fp(M), None, None))
            return m, M
        R = np.empty((self.N, self.E), np.float32)
        Rbar = np.empty(self.E, np.float32)
        self._check(lib().tpq_get_ranges(self._h, _fp(m), _fp(M), _fp(R), _fp(Rbar)))
        return m, M, R, Rbar

    def get_scales(self):
        s = np.empty((self.N, self.E), np.float32)
        inv = np.empty((self.N, self.E), np.float32)
        self._check(lib().tpq_get_scales(self._h, _fp(s), _fp(inv)))
        return s, inv

    def num_selected(self) -> int:
        return int(lib().tpq_num_selected(self._h))

    def get_features(self) -> np.ndarray:
        k = max(self.num_selected(), 0)
        out = np.zeros(max(k, 1), np.int32)
        self._check(lib().tpq_get_features(self._h, out.ctypes.data_as(POINTER(c_int32))))
        return out[:k].copy()

    def get_slot_order(self) -> np.ndarray:
        """Feature carried by each code slot of a token (length E - k)."""
        L = self.E - max(self.num_selected(), 0)
        out = np.zeros(max(L, 1), np.int32)
        self._check(lib().tpq_get_slot_order(self._h, out.ctypes.data_as(POINTER(c_int32))))
        return out[:L].copy()

    def payload_bytes(self, T: int) -> int:
        return int(lib().tpq_payload_bytes(self._h, T))

    def comm_bytes(self, T: int) -> CommReport:
        r = CommReport()
        self._check(lib().tpq_comm_bytes(self._h, T, byref(r)))
        return r

    def quantize_pack(self, shard: int, y_ptr: int, T: int, payload_ptr: int, payload_capacity: int,
                      row_stride: int | None = None, stream: int = 0):
        self._check(lib().tpq_quantize_pack(self._h, shard, y_ptr, T, self.E if row_stride is None else row_stride,
                                            payload_ptr, payload_capacity, stream))

    def quantize_pack_batch(self, first_shard: int, y_ptrs, T: int, payload_ptrs, payload_capacity: int,
                            row_stride: int | None = None, stream: int = 0):
        n = len(y_ptrs)
        assert len(payload_ptrs) == n
        ya = y_ptrs if isinstance(y_ptrs, ctypes.Array) else (c_void_p * n)(*y_ptrs)
        pa = payload_ptrs if isinstance(payload_ptrs, ctypes.Array) else (c_void_p * n)(*payload_ptrs)
        self._check(lib().tpq_quantize_pack_batch(self._h, first_shard, n, ya, T,
                                                  self.E if row_stride is None else row_stride, pa,
                                                  payload_capacity, stream))

    def dequant_reduce(self, payload_ptrs, T: int, out_ptr: int, out_dtype: int = TPQ_OUT_BF16,
                       out_row_stride: int | None = None, stream: int = 0, bias_ptr: int | None = None,
                       arrived_ptr: int | None = None, epoch: int = 0, timeout_ns: int = 0):
        arr = payload_ptrs if isinstance(payload_ptrs, ctypes.Array) else (c_void_p * len(payload_ptrs))(*payload_ptrs)
        stride = self.E if out_row_stride is None else out_row_stride
        if arrived_ptr is not None:
            self._check(lib().tpq_dequant_reduce_arrivals(self._h, arr, len(payload_ptrs), T, out_ptr, out_dtype, stride,
                                                          bias_ptr, arrived_ptr, epoch & 0xFFFFFFFF, timeout_ns, stream))
        elif bias_ptr is None:
            self._check(lib().tpq_dequant_reduce(self._h, arr, len(payload_ptrs), T, out_ptr, out_dtype, stride, stream))
        else:
            self._check(lib().tpq_dequant_reduce_bias(self._h, arr, len(payload_ptrs), T, out_ptr, out_dtype, stride,
                                                      bias_ptr, stream))

    def permute_weight(self, w_ptr: int, K: int, w_slots_ptr: int, stream: int = 0):
        self._check(lib().tpq_permute_weight(self._h, w_ptr, K, w_slots_ptr, stream))

    def linear_quantize_pack(self, shard: int, x_ptr: int, w_slots_ptr: int, T: int, K: int, payload_ptr: int,
                             payload_capacity: int, y_slots_ptr: int | None = None, stream: int = 0):
        self._check(lib().tpq_linear_quantize_pack(self._h, shard, x_ptr, w_slots_ptr, T, K, payload_ptr, payload_capacity,
                                                   y_slots_ptr, stream))

    def quantize_pack_push(self, shard: int, y_ptr: int, T: int, dst_ptrs, arrived_ptrs, dst_capacity: int, epoch: int,
                           row_stride: int | None = None, stream: int = 0):
        n = len(dst_ptrs)
        assert len(arrived_ptrs) == n
        da = dst_ptrs if isinstance(dst_ptrs, ctypes.Array) else (c_void_p * n)(*dst_ptrs)
        aa = arrived_ptrs if isinstance(arrived_ptrs, ctypes.Array) else (c_void_p * n)(*arrived_ptrs)
        self._check(lib().tpq_quantize_pack_push(self._h, shard, y_ptr, T, self.E if row_stride is None else row_stride,
                                                 da, aa, n, dst_capacity, epoch & 0xFFFFFFFF, stream))

    def wait_arrivals(self, arrived_ptr: int, n: int, epoch: int, timeout_ns: int = 0, stream: int = 0):
        self._check(lib().tpq_wait_arrivals(self._h, arrived_ptr, n, epoch & 0xFFFFFFFF, timeout_ns, stream))

    def get_state(self) -> bytes:
        n = c_size_t(0)
        self._check(lib().tpq_get_state(self._h, None, byref(n)))
        buf = ctypes.create_string_buffer(n.value)
        self._check(lib().tpq_get_state(self._h, buf, byref(n)))
        return buf.raw[: n.value]

    def set_state(self, blob: bytes):
        self._check(lib().tpq_set_state(self._h, blob, len(blob)))

    def device_status(self) -> int:
        return int(lib().tpq_device_status(self._h))

    def launch_count(self) -> int:
        return int(lib().tpq_launch_count(self._h))


def payload_bytes_for(T: int, E: int, k: int, bits: int = 4) -> int:
    if bits == 4:
        return int(lib().tpq_payload_bytes_for(T, E, k))
    return int(lib().tpq_payload_bytes_for_bits(T, E, k, bits))
